// CPU oracle for the Dynamic Communication Thresholding (DCT) compression path.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
// CUDA library is compared against.  It shares no code with the CUDA path and
// must never be called from it: only the test-suite, the smoke check and the
// benchmark's CPU-baseline leg may load it.
//
// Everything here follows the two algorithm boxes of the paper in their own
// order and notation:
//   Algorithm 1 (DCT-DP):  W = W_grad + E_grad;  tau = order statistic of |W|;
//                          M = I(|W| >= tau);  W_hat = W .* M;  E = W - W_hat.
//   Algorithm 2 (DCT-MP):  per sample i, tau_i = order statistic of |X_act,i|,
//                          m_i = I(|X_act,i| >= tau_i); the same mask M packs
//                          X_act (forward) and X_grad (backward).
//
// Readings where the paper is silent (also listed in the design notes):
//   * Order of magnitudes: key(x) = bit pattern of x with the sign bit cleared,
//     compared as an unsigned integer.  For every non-NaN x this is the order of
//     |x| with -0 == +0.
//   * The caller passes the survivor target k (k-th LARGEST magnitude), which
//     removes the paper's ambiguity about the direction of eta.
//   * Ties at the threshold: DP with no tie budget keeps every |w| >= tau
//     (Algorithm 1, mask step, literally); with a tie budget at most that many
//     elements equal to tau pass, lowest index first.  MP keeps exactly k per
//     row, lowest column first among equals.
//   * Capacity: survivors beyond the output capacity are treated as not sent,
//     so they stay in the residual and  sent + E' == W  still holds.
//   * W - W_hat is +0.0 where sent (w - w) and w itself elsewhere (w - 0).
//
// Parity status: every function below is pinned by tests that do not reuse its
// own formula (brute-force rank counting, library top-k / kthvalue, closed-form
// Gaussian quantiles, hand-worked fixtures, conservation invariants).  Nothing
// in this file is "parity unpinned".
//
// Arithmetic: one IEEE-754 binary32 addition, round-to-nearest-even, denormals
// kept (build without -ffast-math).  Everything else is integer work or a copy.

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <utility>
#include <vector>

namespace {

inline uint32_t bits_of(float x) {
    uint32_t u;
    std::memcpy(&u, &x, sizeof u);
    return u;
}

inline float float_of(uint32_t u) {
    float x;
    std::memcpy(&x, &u, sizeof x);
    return x;
}

// |x| as an unsigned integer: the total order used for every comparison.
inline uint32_t key_f32(float x) { return bits_of(x) & 0x7FFFFFFFu; }
inline uint16_t key_bf16(uint16_t x) { return static_cast<uint16_t>(x & 0x7FFFu); }

// Algorithm 1, "Error Feedback" step: W = W_grad + E_grad (one fp32 add).
inline float error_feedback(const float* grad, const float* residual, uint64_t i) {
    if (residual == nullptr) return grad[i];
    volatile float w = grad[i] + residual[i];  // volatile: no contraction, no excess precision
    return w;
}

}  // namespace

extern "C" {

// Algorithm 1, threshold steps: sort |W| and read the order statistic.
// tau is the k-th largest magnitude (1 <= k <= n).  n_gt / n_eq count the
// elements strictly above / exactly at tau, so n_gt < k <= n_gt + n_eq.
// full_sort != 0: literal full sort of the copy ("copy and sort").
// full_sort == 0: std::nth_element on the copy (same order statistic; used for
//                 sizes where a full sort is needlessly slow; the tests check
//                 that both agree).
int oracle_dp_select(const float* grad, const float* residual, uint64_t n, uint64_t k,
                     int full_sort, float* tau_out, uint64_t* n_gt_out, uint64_t* n_eq_out) {
    if (grad == nullptr || n == 0 || k == 0 || k > n) return 1;
    std::vector<uint32_t> keys(n);
    for (uint64_t i = 0; i < n; ++i) keys[i] = key_f32(error_feedback(grad, residual, i));

    uint32_t tau_key;
    if (full_sort) {
        std::vector<uint32_t> sorted(keys);
        std::sort(sorted.begin(), sorted.end());  // ascending: w_1 <= ... <= w_n
        tau_key = sorted[n - k];                  // k-th largest
    } else {
        std::vector<uint32_t> copy(keys);
        std::nth_element(copy.begin(), copy.begin() + (n - k), copy.end());
        tau_key = copy[n - k];
    }

    uint64_t n_gt = 0, n_eq = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (keys[i] > tau_key) ++n_gt;
        else if (keys[i] == tau_key) ++n_eq;
    }
    *tau_out = float_of(tau_key);
    if (n_gt_out) *n_gt_out = n_gt;
    if (n_eq_out) *n_eq_out = n_eq;
    return 0;
}

// Algorithm 1, error feedback + mask + compressed gradient + error steps, for a
// given tau.  One sequential pass in index order.
//   has_budget == 0: M = I(|W| >= tau).
//   has_budget != 0: elements with |w| == tau pass only while fewer than
//                    tie_budget of them have been seen (lowest index first).
// Survivors are written as (idx, val) in ascending index order while there is
// room; survivors without room stay in the residual.
int oracle_dp_compress(const float* grad, float* residual, uint64_t n, float tau,
                       int has_budget, uint64_t tie_budget,
                       int32_t* idx_out, float* val_out, uint64_t capacity,
                       uint64_t* count_out, uint64_t* needed_out) {
    if (grad == nullptr || residual == nullptr || n == 0) return 1;
    const uint32_t tau_key = key_f32(tau);
    uint64_t out = 0, needed = 0, eq_seen = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const float w = error_feedback(grad, residual, i);
        const uint32_t kw = key_f32(w);
        bool pass = kw > tau_key;
        if (kw == tau_key) {
            pass = !has_budget || eq_seen < tie_budget;
            ++eq_seen;
        }
        if (pass) ++needed;
        if (pass && out < capacity) {
            idx_out[out] = static_cast<int32_t>(i);
            val_out[out] = w;
            residual[i] = 0.0f;  // w - w
            ++out;
        } else {
            residual[i] = w;     // w - 0
        }
    }
    *count_out = out;
    *needed_out = needed;
    return 0;
}

}  // extern "C"

namespace {

// Algorithm 2, forward pass for one row: order the row by magnitude, read
// tau_i at the k-th largest, keep exactly k columns (ties: lower column).
template <typename T, typename KeyFn>
void mp_forward_row(const T* x, uint32_t d, uint32_t k, KeyFn key,
                    int16_t* cols, T* vals, T* tau) {
    std::vector<std::pair<uint32_t, uint32_t>> order(d);  // (key, column)
    for (uint32_t j = 0; j < d; ++j) order[j] = {key(x[j]), j};
    // descending magnitude; stable => lower column first among equal magnitudes
    std::stable_sort(order.begin(), order.end(),
                     [](const auto& a, const auto& b) { return a.first > b.first; });
    const uint32_t tau_col = order[k - 1].second;
    std::vector<uint32_t> kept(k);
    for (uint32_t s = 0; s < k; ++s) kept[s] = order[s].second;
    std::sort(kept.begin(), kept.end());
    for (uint32_t s = 0; s < k; ++s) {
        cols[s] = static_cast<int16_t>(kept[s]);
        vals[s] = x[kept[s]];  // bit copy, sign kept
    }
    if (tau) {
        T t = x[tau_col];
        // tau_i is a magnitude: clear the sign bit
        if constexpr (sizeof(T) == 4) {
            uint32_t u;
            std::memcpy(&u, &t, 4);
            u &= 0x7FFFFFFFu;
            std::memcpy(&t, &u, 4);
        } else {
            uint16_t u;
            std::memcpy(&u, &t, 2);
            u &= 0x7FFFu;
            std::memcpy(&t, &u, 2);
        }
        *tau = t;
    }
}

template <typename T, typename KeyFn>
int mp_forward(const T* x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, KeyFn key,
               int16_t* cols, T* vals, T* tau) {
    if (x == nullptr || d == 0 || k == 0 || k > d || d > 32768u || ld < d) return 1;
    for (uint32_t i = 0; i < rows; ++i)
        mp_forward_row(x + static_cast<uint64_t>(i) * ld, d, k, key,
                       cols + static_cast<uint64_t>(i) * k, vals + static_cast<uint64_t>(i) * k,
                       tau ? tau + i : nullptr);
    return 0;
}

// Algorithm 2, backward pass: X_grad .* M, packed in the slot order of the mask.
template <typename T>
int mp_backward(const T* gx, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                const int16_t* cols, T* gvals) {
    if (gx == nullptr || cols == nullptr || d == 0 || k == 0 || k > d || ld < d) return 1;
    for (uint32_t i = 0; i < rows; ++i)
        for (uint32_t s = 0; s < k; ++s) {
            const uint32_t c = static_cast<uint16_t>(cols[static_cast<uint64_t>(i) * k + s]);
            if (c >= d) return 2;
            gvals[static_cast<uint64_t>(i) * k + s] = gx[static_cast<uint64_t>(i) * ld + c];
        }
    return 0;
}

}  // namespace

extern "C" {

// Receiving end of "Send W_hat" (Algorithm 1): the sparse vector goes back into a dense one, either on
// its own (dense = W_hat) or added to what is already there (a server summing several trainers).
int oracle_dp_decompress(const int32_t* idx, const float* val, uint64_t count, float* dense, uint64_t n,
                         int accumulate) {
    if (dense == nullptr || n == 0) return 1;
    if (!accumulate)
        for (uint64_t i = 0; i < n; ++i) dense[i] = 0.0f;
    for (uint64_t j = 0; j < count; ++j) {
        if (idx[j] < 0 || static_cast<uint64_t>(idx[j]) >= n) return 2;
        if (accumulate) {
            volatile float s = dense[idx[j]] + val[j];
            dense[idx[j]] = s;
        } else {
            dense[idx[j]] = val[j];
        }
    }
    return 0;
}

}  // extern "C"

namespace {
// Receiving end of Algorithm 2's sends: X .* M rebuilt from the mask columns and the packed values.
template <typename T>
int mp_unpack(const int16_t* cols, const T* vals, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, T* dense) {
    if (cols == nullptr || vals == nullptr || dense == nullptr || d == 0 || k == 0 || k > d || ld < d) return 1;
    for (uint32_t i = 0; i < rows; ++i) {
        for (uint32_t j = 0; j < d; ++j) dense[static_cast<uint64_t>(i) * ld + j] = T(0);
        for (uint32_t s = 0; s < k; ++s) {
            const uint32_t c = static_cast<uint16_t>(cols[static_cast<uint64_t>(i) * k + s]);
            if (c >= d) return 2;
            dense[static_cast<uint64_t>(i) * ld + c] = vals[static_cast<uint64_t>(i) * k + s];
        }
    }
    return 0;
}
}  // namespace

extern "C" {

int oracle_mp_unpack_f32(const int16_t* cols, const float* vals, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                         float* dense) {
    return mp_unpack<float>(cols, vals, rows, d, ld, k, dense);
}
int oracle_mp_unpack_bf16(const int16_t* cols, const uint16_t* vals, uint32_t rows, uint32_t d, uint32_t ld,
                          uint32_t k, uint16_t* dense) {
    return mp_unpack<uint16_t>(cols, vals, rows, d, ld, k, dense);
}

int oracle_mp_fwd_f32(const float* x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                      int16_t* cols, float* vals, float* tau) {
    return mp_forward<float>(x, rows, d, ld, k, [](float v) { return key_f32(v); }, cols, vals, tau);
}

// bf16 values travel as their 16-bit patterns.
int oracle_mp_fwd_bf16(const uint16_t* x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                       int16_t* cols, uint16_t* vals, uint16_t* tau) {
    return mp_forward<uint16_t>(x, rows, d, ld, k,
                                [](uint16_t v) { return static_cast<uint32_t>(key_bf16(v)); },
                                cols, vals, tau);
}

int oracle_mp_bwd_f32(const float* gx, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                      const int16_t* cols, float* gvals) {
    return mp_backward<float>(gx, rows, d, ld, k, cols, gvals);
}

int oracle_mp_bwd_bf16(const uint16_t* gx, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                       const int16_t* cols, uint16_t* gvals) {
    return mp_backward<uint16_t>(gx, rows, d, ld, k, cols, gvals);
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Threshold diagnostics (the quantities behind the paper's two threshold plots)
// ---------------------------------------------------------------------------
namespace {

// tau_i for one row and one sparsity level: the row's magnitudes sorted in
// descending order, read at position k (Algorithm 2, threshold step).
template <typename T, typename KeyFn>
uint32_t row_threshold_key(const T* x, uint32_t d, uint32_t k, KeyFn key) {
    std::vector<uint32_t> mags(d);
    for (uint32_t j = 0; j < d; ++j) mags[j] = key(x[j]);
    std::sort(mags.begin(), mags.end(), [](uint32_t a, uint32_t b) { return a > b; });
    return mags[k - 1];
}

inline double value_of_key(float, uint32_t k) { return static_cast<double>(float_of(k)); }
inline double value_of_key(uint16_t, uint32_t k) { return static_cast<double>(float_of(k << 16)); }

// Sec. 2.2 (the plot of the mean threshold): mean_out[q] = (1/B) sum_i tau_i at
// sparsity level q, with tau_i the ks[q]-th largest magnitude of row i.  The
// sum runs over the rows in order, in binary64; nothing is sparsified.
template <typename T, typename KeyFn, typename FromKey>
int mp_threshold_mean(const T* x, uint32_t rows, uint32_t d, uint32_t ld, const uint32_t* ks, uint32_t m,
                      KeyFn key, FromKey from_key, double* mean_out, T* tau_out) {
    if (x == nullptr || ks == nullptr || mean_out == nullptr || rows == 0 || d == 0 || ld < d) return 1;
    for (uint32_t q = 0; q < m; ++q) {
        if (ks[q] == 0 || ks[q] > d) return 1;
        double sum = 0.0;
        for (uint32_t i = 0; i < rows; ++i) {
            const uint32_t tk = row_threshold_key(x + static_cast<uint64_t>(i) * ld, d, ks[q], key);
            if (tau_out) tau_out[static_cast<uint64_t>(q) * rows + i] = from_key(tk);
            volatile double s = sum + value_of_key(T(), tk);
            sum = s;
        }
        mean_out[q] = sum / static_cast<double>(rows);
    }
    return 0;
}

}  // namespace

extern "C" {

// Sec. 2.1 (the plot of the top-K threshold at several sparsity levels): the
// order statistic of Algorithm 1 read at several positions of ONE sorted copy.
int oracle_dp_select_multi(const float* grad, const float* residual, uint64_t n, const uint64_t* ks, uint32_t m,
                           float* tau_out, uint64_t* n_gt_out, uint64_t* n_eq_out) {
    if (grad == nullptr || ks == nullptr || n == 0) return 1;
    std::vector<uint32_t> sorted(n);
    for (uint64_t i = 0; i < n; ++i) sorted[i] = key_f32(error_feedback(grad, residual, i));
    std::sort(sorted.begin(), sorted.end());      // ascending: w_1 <= ... <= w_n
    for (uint32_t q = 0; q < m; ++q) {
        if (ks[q] == 0 || ks[q] > n) return 1;
        const uint32_t tau_key = sorted[n - ks[q]];
        uint64_t n_gt = 0, n_eq = 0;
        for (uint64_t i = 0; i < n; ++i) {
            if (sorted[i] > tau_key) ++n_gt;
            else if (sorted[i] == tau_key) ++n_eq;
        }
        tau_out[q] = float_of(tau_key);
        if (n_gt_out) n_gt_out[q] = n_gt;
        if (n_eq_out) n_eq_out[q] = n_eq;
    }
    return 0;
}

int oracle_mp_threshold_mean_f32(const float* x, uint32_t rows, uint32_t d, uint32_t ld, const uint32_t* ks,
                                 uint32_t m, double* mean_out, float* tau_out) {
    return mp_threshold_mean<float>(x, rows, d, ld, ks, m, [](float v) { return key_f32(v); },
                                    [](uint32_t k) { return float_of(k); }, mean_out, tau_out);
}
int oracle_mp_threshold_mean_bf16(const uint16_t* x, uint32_t rows, uint32_t d, uint32_t ld, const uint32_t* ks,
                                  uint32_t m, double* mean_out, uint16_t* tau_out) {
    return mp_threshold_mean<uint16_t>(x, rows, d, ld, ks, m,
                                       [](uint16_t v) { return static_cast<uint32_t>(key_bf16(v)); },
                                       [](uint32_t k) { return static_cast<uint16_t>(k); }, mean_out, tau_out);
}

// Guard for a reused threshold (Sec. 2.1, threshold life-span): 1 if the survivor
// count exceeds k * num / den, 2 if it is below k * den / num, 0 otherwise
// (num / den >= 1; exact integer comparison).  The rule is the library's, not
// the paper's; the oracle states it so that the device kernel has a definition.
int oracle_dp_drift_flag(uint64_t needed, uint64_t k, uint32_t num, uint32_t den) {
    const unsigned __int128 a = static_cast<unsigned __int128>(needed) * den, b = static_cast<unsigned __int128>(k) * num;
    const unsigned __int128 c = static_cast<unsigned __int128>(needed) * num, e = static_cast<unsigned __int128>(k) * den;
    if (a > b) return 1;
    if (c < e) return 2;
    return 0;
}

}  // extern "C"
