// Threshold diagnostics: the quantities the paper plots to motivate the method.
//
//   dct_threshold_select_multi  top-k thresholds of one gradient vector at several sparsity levels
//                               (Sec. 2.1: the threshold at 75 / 90 / 95 % sparsity over the iterations)
//   dct_mp_threshold_mean       (1/B) sum_i tau_i at several sparsity levels, nothing sparsified
//                               (Sec. 2.2: the mean threshold with and without DCT-MP)
//   dct_dp_drift_check          survivor count against the target while tau is reused (Sec. 2.1, life-span L)
//
// The multi-quantile select is the most-significant-digit-first radix select of dct_threshold_select
// (digits of 11/10/10 bits over the 31 magnitude bits) carried out for m ranks in the same three
// passes: the histogram of the leading digit is common to all ranks; the second and third pass keep
// one histogram per rank, each restricted to the prefix that rank has chosen so far.
#include "common.cuh"
#include "mp_warp.cuh"
#include "row_select.cuh"

namespace dct {
namespace {

constexpr int kMaxQ = static_cast<int>(DCT_DIAG_MAX_QUANTILES);
constexpr int kDiagThreads = 512;
constexpr int kDiagVecs = 4;
constexpr uint32_t kDiagChunk = kDiagThreads * kDiagVecs * 4;   // 8192 elements per CTA iteration
constexpr int kDiagBins = 2048;
constexpr int kDiagPasses = 3;

__host__ __device__ constexpr int diag_shift(int p) { return p == 0 ? 20 : (p == 1 ? 10 : 0); }
__host__ __device__ constexpr int diag_bits(int p) { return p == 0 ? 11 : 10; }

struct RankState {
    uint32_t prefix;      // digits chosen so far (right-aligned)
    uint32_t k_rem;       // rank still to be located inside the prefix bucket
    uint64_t n_gt;        // elements known to be above the bucket
    uint32_t hist[kDiagPasses][kDiagBins];   // hist[0] is used by rank 0 only (the leading digit is shared)
};
struct MultiWorkspace {
    uint32_t done[kDiagPasses];
    uint32_t pad;
    RankState rank[kMaxQ];
};
struct Ranks {
    uint32_t k[kMaxQ];
};

__global__ void multi_init_kernel(MultiWorkspace* ws, int m, dct_result_t* results) {
    uint32_t* words = reinterpret_cast<uint32_t*>(ws);
    const uint32_t n_words = sizeof(MultiWorkspace) / 4;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += gridDim.x * blockDim.x) words[i] = 0;
    if (blockIdx.x == 0 && threadIdx.x < static_cast<uint32_t>(m)) {
        dct_result_t* r = results + threadIdx.x;
        r->status = DCT_OK;
        r->reserved = 0;
        r->count = 0;
        r->needed = 0;
        r->n_gt = 0;
        r->n_eq = 0;
    }
}
// k_rem is written after the clearing kernel has finished (a separate launch keeps the two apart)
__global__ void multi_seed_kernel(MultiWorkspace* ws, Ranks ks, int m) {
    if (threadIdx.x < static_cast<uint32_t>(m)) ws->rank[threadIdx.x].k_rem = ks.k[threadIdx.x];
}

// The last CTA of a pass: the digit that holds rank k_rem, counted from the top of `hist`.
template <int kPass>
__device__ __forceinline__ void multi_finish(RankState* st, const uint32_t* hist, uint32_t* s_scan, float* tau_out,
                                             dct_result_t* result) {
    constexpr int bits = diag_bits(kPass);
    const uint32_t prefix = kPass == 0 ? 0u : st->prefix;
    const uint32_t k_rem = st->k_rem;
    // thread t owns bins top-down: bin(t, q) = kDiagBins-1 - (4t + q), q = 0..3
    uint32_t c[4], own = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        c[q] = __ldcg(&hist[kDiagBins - 1 - (4 * threadIdx.x + q)]);
        own += c[q];
    }
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    uint32_t incl = own;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= static_cast<uint32_t>(o)) incl += t;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    uint32_t above = incl - own;
    for (uint32_t v = 0; v < warp; ++v) above += s_scan[v];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (above < k_rem && k_rem <= above + c[q]) {
            const uint32_t digit = kDiagBins - 1 - (4 * threadIdx.x + q);
            const uint32_t new_prefix = (prefix << bits) | digit;
            const uint64_t n_gt = st->n_gt + above;
            st->prefix = new_prefix;
            st->k_rem = k_rem - above;
            st->n_gt = n_gt;
            if (kPass == kDiagPasses - 1) {
                *tau_out = __uint_as_float(new_prefix);
                result->n_gt = n_gt;
                result->n_eq = c[q];
            }
        }
        above += c[q];
    }
    __syncthreads();      // s_scan is reused for the next rank
}

template <int kPass, bool kVectorised>
__global__ void __launch_bounds__(kDiagThreads)
multi_pass_kernel(const float* __restrict__ grad, const float* __restrict__ residual, uint32_t n, MultiWorkspace* ws,
                  int m, float* __restrict__ tau_out, dct_result_t* __restrict__ results) {
    constexpr int shift = diag_shift(kPass);
    constexpr int bits = diag_bits(kPass);
    constexpr uint32_t digit_mask = (1u << bits) - 1u;
    constexpr int kHists = kPass == 0 ? 1 : kMaxQ;
    __shared__ uint32_t sh[kHists][kDiagBins];
    __shared__ uint32_t s_scan[kDiagThreads / 32];
    __shared__ uint32_t s_last;
    const int hists = kPass == 0 ? 1 : m;

    for (int b = threadIdx.x; b < hists * kDiagBins; b += kDiagThreads) (&sh[0][0])[b] = 0;
    // Ranks whose prefixes are equal so far share one histogram (that of the first of them): an element then
    // matches at most one histogram, and a pass costs one shared-memory atomic per matching element, not one
    // instruction per rank.  owner[q] = the rank whose histogram rank q reads; prefix[q] = 0xFFFFFFFF (matches
    // nothing) for q >= m and for ranks that are not owners.
    uint32_t prefix[kMaxQ];
    int owner[kMaxQ];
#pragma unroll
    for (int q = 0; q < kMaxQ; ++q) {
        prefix[q] = (kPass != 0 && q < m) ? ws->rank[q].prefix : 0xFFFFFFFFu;
        owner[q] = q;
    }
#pragma unroll
    for (int q = 1; q < kMaxQ; ++q) {
#pragma unroll
        for (int p = q - 1; p >= 0; --p)
            if (kPass != 0 && q < m && prefix[p] == prefix[q] && owner[p] == p) owner[q] = p;
    }
#pragma unroll
    for (int q = 0; q < kMaxQ; ++q)
        if (owner[q] != q) prefix[q] = 0xFFFFFFFFu;
    __syncthreads();

    auto consume = [&](uint32_t key) {
        const uint32_t digit = (key >> shift) & digit_mask;
        if (kPass == 0) {
            atomicAdd(&sh[0][digit], 1u);
        } else {
            const uint32_t upper = key >> (shift + bits);
            int hit = -1;
#pragma unroll
            for (int q = 0; q < kMaxQ; ++q)
                if (upper == prefix[q]) hit = q;
            if (hit >= 0) atomicAdd(&(&sh[0][0])[(hit % kHists) * kDiagBins + digit], 1u);
        }
    };

    const uint32_t num_chunks = (n + kDiagChunk - 1) / kDiagChunk;
    for (uint32_t chunk = blockIdx.x; chunk < num_chunks; chunk += gridDim.x) {
        const uint32_t base = chunk * kDiagChunk;
        if (kVectorised && base + kDiagChunk <= n) {
            float4 g4[kDiagVecs], e4[kDiagVecs];
#pragma unroll
            for (int j = 0; j < kDiagVecs; ++j) {
                const uint32_t off = base + (j * kDiagThreads + threadIdx.x) * 4;
                g4[j] = ld_readonly_f4(grad + off);
                e4[j] = residual ? ld_readonly_f4(residual + off) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const bool add = residual != nullptr;
#pragma unroll
            for (int j = 0; j < kDiagVecs; ++j) {
                consume(key_f32(add ? __fadd_rn(g4[j].x, e4[j].x) : g4[j].x));
                consume(key_f32(add ? __fadd_rn(g4[j].y, e4[j].y) : g4[j].y));
                consume(key_f32(add ? __fadd_rn(g4[j].z, e4[j].z) : g4[j].z));
                consume(key_f32(add ? __fadd_rn(g4[j].w, e4[j].w) : g4[j].w));
            }
        } else {
            for (uint32_t i = base + threadIdx.x; i < n && i < base + kDiagChunk; i += kDiagThreads)
                consume(key_f32(residual ? __fadd_rn(grad[i], residual[i]) : grad[i]));
        }
    }
    __syncthreads();

#pragma unroll
    for (int q = 0; q < kHists; ++q) {
        if (q >= hists || (kPass != 0 && owner[q] != q)) continue;      // (counted in its owner's histogram)
        uint32_t* hist = ws->rank[q].hist[kPass];
        for (int b = threadIdx.x; b < kDiagBins; b += kDiagThreads) {
            const uint32_t c = sh[q][b];
            if (c) atomicAdd(&hist[b], c);
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(&ws->done[kPass], 1u) == gridDim.x - 1) ? 1u : 0u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
#pragma unroll
    for (int q = 0; q < kMaxQ; ++q)
        if (q < m)
            multi_finish<kPass>(&ws->rank[q], ws->rank[kPass == 0 ? 0 : owner[q]].hist[kPass], s_scan, tau_out + q,
                                results + q);
}

// ------------------------------------------------------------------------------------------------
// mean of the per-row thresholds
// ------------------------------------------------------------------------------------------------
struct RowRanks {
    uint32_t k[kMaxQ];
};

// One CTA per row at a time; the row is read once into shared memory and selected m times.
template <typename T>
__global__ void mp_row_thresholds_kernel(const T* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, RowRanks ks,
                                         int m, T* __restrict__ tau_out, bool rows_aligned16) {
    using Tr = ElemTraits<T>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    T* row_s = reinterpret_cast<T*>(smem_raw);
    __shared__ uint32_t s_hist[256];
    __shared__ uint32_t s_sel[2];
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    for (uint32_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const T* xr = x + static_cast<size_t>(row) * ld;
        if (rows_aligned16) {
            constexpr uint32_t per16 = 16 / sizeof(T);
            const uint32_t nvec = d / per16;
            const int4* src = reinterpret_cast<const int4*>(xr);
            int4* dst = reinterpret_cast<int4*>(row_s);
            for (uint32_t v = tid; v < nvec; v += nt) dst[v] = __ldg(src + v);
            for (uint32_t j = nvec * per16 + tid; j < d; j += nt) row_s[j] = xr[j];
        } else {
            for (uint32_t j = tid; j < d; j += nt) row_s[j] = xr[j];
        }
        for (int q = 0; q < m; ++q) {
            uint32_t tau_key, take;
            cta_row_select<T>(row_s, d, ks.k[q], s_hist, s_sel, tau_key, take);
            if (tid == 0) tau_out[static_cast<size_t>(q) * rows + row] = Tr::from_key(tau_key);
        }
        __syncthreads();      // row_s is overwritten by the next row
    }
}

// mean_out[q] = (sum_i tau[q*rows + i]) / rows.  Fixed order: thread t adds the elements t, t + 1024, ... in
// ascending order, then the 1024 partial sums are added pairwise (stride 512, 256, ..., 1).
constexpr int kMeanThreads = 1024;
template <typename T>
__global__ void __launch_bounds__(kMeanThreads)
tau_mean_kernel(const T* __restrict__ tau, uint32_t rows, double* __restrict__ mean_out) {
    using Tr = ElemTraits<T>;
    __shared__ double s_part[kMeanThreads];
    const T* t = tau + static_cast<size_t>(blockIdx.x) * rows;
    double acc = 0.0;
    for (uint32_t i = threadIdx.x; i < rows; i += kMeanThreads) acc = __dadd_rn(acc, Tr::to_double(t[i]));
    s_part[threadIdx.x] = acc;
    __syncthreads();
    for (int s = kMeanThreads / 2; s > 0; s >>= 1) {
        if (threadIdx.x < static_cast<uint32_t>(s))
            s_part[threadIdx.x] = __dadd_rn(s_part[threadIdx.x], s_part[threadIdx.x + s]);
        __syncthreads();
    }
    if (threadIdx.x == 0) mean_out[blockIdx.x] = __ddiv_rn(s_part[0], static_cast<double>(rows));
}

template <typename T>
dct_status_t launch_threshold_mean(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, const RowRanks& ks, int m,
                                   double* mean_out, void* tau_out, cudaStream_t stream) {
    // Where the CTA-per-row forward kernels apply to every level, they find the thresholds (one launch per level,
    // nothing packed): 16384x4096 bf16, three levels: 0.31 -> 0.12 ms.  The general kernel below reads the row once
    // for all levels, but selects with 8-bit radix passes.
    {
        bool all = true;
        for (int q = 0; q < m && all; ++q) {
            bool handled = false;
            void* out = static_cast<T*>(tau_out) + static_cast<size_t>(q) * rows;
            const dct_status_t st = sizeof(T) == 2
                ? launch_tau_bf16_wide(x_act, rows, d, ld, ks.k[q], out, stream, &handled)
                : launch_tau_f32_wide(x_act, rows, d, ld, ks.k[q], out, stream, &handled);
            if (st != DCT_OK) return st;
            all = handled;              // (q == 0 decides for shapes; a later k outside the kernels' range starts over below)
        }
        if (all) {
            tau_mean_kernel<T><<<m, kMeanThreads, 0, stream>>>(static_cast<const T*>(tau_out), rows, mean_out);
            DCT_CUDA_TRY(cudaGetLastError());
            return DCT_OK;
        }
    }
    const size_t smem = ((static_cast<size_t>(d) * sizeof(T)) + 15) & ~static_cast<size_t>(15);
    auto kernel = mp_row_thresholds_kernel<T>;
    // (static shared memory counts against the 48 KiB a kernel gets without asking: ask well below that)
    if (smem > 32 * 1024) DCT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    const int threads = d <= 4096 ? 128 : (d <= 8192 ? 256 : (d <= 16384 ? 512 : 1024));
    int per_sm = 0;
    DCT_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem));
    if (per_sm < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t max_grid = static_cast<uint64_t>(sms) * per_sm;
    const uint32_t grid = static_cast<uint32_t>(rows < max_grid ? rows : max_grid);
    const bool rows_aligned16 = aligned_to(x_act, 16) && ((static_cast<size_t>(ld) * sizeof(T)) % 16 == 0);
    kernel<<<grid, threads, smem, stream>>>(static_cast<const T*>(x_act), rows, d, ld, ks, m, static_cast<T*>(tau_out),
                                            rows_aligned16);
    DCT_CUDA_TRY(cudaGetLastError());
    tau_mean_kernel<T><<<m, kMeanThreads, 0, stream>>>(static_cast<const T*>(tau_out), rows, mean_out);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

__global__ void drift_check_kernel(const dct_result_t* __restrict__ result, uint64_t k, uint32_t num, uint32_t den,
                                   uint32_t* __restrict__ flag_out) {
    // needed, k < 2^32 and num, den < 2^32: the products fit 64 bits
    const uint64_t needed = result->needed;
    uint32_t flag = 0;
    if (needed * den > k * num) flag = 1;
    else if (needed * num < k * den) flag = 2;
    *flag_out = flag;
}

}  // namespace
}  // namespace dct

using namespace dct;

extern "C" size_t dct_threshold_select_multi_workspace_bytes(uint64_t n, uint32_t m) {
    if (n == 0 || n > 0x7FFFFFFFull || m == 0 || m > DCT_DIAG_MAX_QUANTILES) return 0;
    return (sizeof(MultiWorkspace) + 255) & ~static_cast<size_t>(255);
}

extern "C" dct_status_t dct_threshold_select_multi(const float* grad, const float* residual, uint64_t n,
                                                   const uint64_t* ks, uint32_t m, float* tau_out,
                                                   dct_result_t* results, void* workspace, size_t workspace_bytes,
                                                   dct_stream_t stream_) {
    if (!grad || !ks || !tau_out || !results || n == 0 || n > 0x7FFFFFFFull || m == 0 || m > DCT_DIAG_MAX_QUANTILES)
        return DCT_ERR_INVALID_ARG;
    Ranks ranks{};
    for (uint32_t q = 0; q < m; ++q) {
        if (ks[q] == 0 || ks[q] > n) return DCT_ERR_INVALID_ARG;
        ranks.k[q] = static_cast<uint32_t>(ks[q]);
    }
    if (!aligned_to(grad, 4) || (residual && !aligned_to(residual, 4)) || !aligned_to(tau_out, 4) ||
        !aligned_to(results, 8))
        return DCT_ERR_INVALID_ARG;
    if (!workspace || !aligned_to(workspace, 256) ||
        workspace_bytes < dct_threshold_select_multi_workspace_bytes(n, m))
        return DCT_ERR_WORKSPACE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    auto* ws = static_cast<MultiWorkspace*>(workspace);
    const uint32_t n32 = static_cast<uint32_t>(n);
    const int im = static_cast<int>(m);
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t chunks = (n + kDiagChunk - 1) / kDiagChunk;
    const int grid = static_cast<int>(chunks < static_cast<uint64_t>(sms) * 2 ? chunks : sms * 2);
    const bool vec = aligned_to(grad, 16) && (!residual || aligned_to(residual, 16));

    multi_init_kernel<<<32, 1024, 0, stream>>>(ws, im, results);
    DCT_CUDA_TRY(cudaGetLastError());
    multi_seed_kernel<<<1, 32, 0, stream>>>(ws, ranks, im);
    DCT_CUDA_TRY(cudaGetLastError());
    if (vec) {
        multi_pass_kernel<0, true><<<grid, kDiagThreads, 0, stream>>>(grad, residual, n32, ws, im, tau_out, results);
        multi_pass_kernel<1, true><<<grid, kDiagThreads, 0, stream>>>(grad, residual, n32, ws, im, tau_out, results);
        multi_pass_kernel<2, true><<<grid, kDiagThreads, 0, stream>>>(grad, residual, n32, ws, im, tau_out, results);
    } else {
        multi_pass_kernel<0, false><<<grid, kDiagThreads, 0, stream>>>(grad, residual, n32, ws, im, tau_out, results);
        multi_pass_kernel<1, false><<<grid, kDiagThreads, 0, stream>>>(grad, residual, n32, ws, im, tau_out, results);
        multi_pass_kernel<2, false><<<grid, kDiagThreads, 0, stream>>>(grad, residual, n32, ws, im, tau_out, results);
    }
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

extern "C" dct_status_t dct_mp_threshold_mean(const void* x_act, dct_dtype_t dtype, uint32_t rows, uint32_t d,
                                              uint32_t ld, const uint32_t* ks, uint32_t m, double* mean_out,
                                              void* tau_out, dct_stream_t stream_) {
    if (!x_act || !ks || !mean_out || !tau_out || rows == 0 || d == 0 || ld < d || m == 0 ||
        m > DCT_DIAG_MAX_QUANTILES)
        return DCT_ERR_INVALID_ARG;
    if (dtype != DCT_F32 && dtype != DCT_BF16) return DCT_ERR_INVALID_ARG;
    if (d > 32768u) return DCT_ERR_UNSUPPORTED;
    RowRanks ranks{};
    for (uint32_t q = 0; q < m; ++q) {
        if (ks[q] == 0 || ks[q] > d) return DCT_ERR_INVALID_ARG;
        ranks.k[q] = ks[q];
    }
    const size_t es = dtype == DCT_F32 ? 4 : 2;
    if (!aligned_to(x_act, es) || !aligned_to(tau_out, es) || !aligned_to(mean_out, 8)) return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (dtype == DCT_F32)
        return launch_threshold_mean<float>(x_act, rows, d, ld, ranks, static_cast<int>(m), mean_out, tau_out, stream);
    return launch_threshold_mean<uint16_t>(x_act, rows, d, ld, ranks, static_cast<int>(m), mean_out, tau_out, stream);
}

extern "C" dct_status_t dct_dp_drift_check(const dct_result_t* compress_result, uint64_t k, uint32_t ratio_num,
                                           uint32_t ratio_den, uint32_t* flag_out, dct_stream_t stream_) {
    if (!compress_result || !flag_out || k == 0 || k > 0x7FFFFFFFull || ratio_den == 0 || ratio_num < ratio_den)
        return DCT_ERR_INVALID_ARG;
    if (!aligned_to(compress_result, 8) || !aligned_to(flag_out, 4)) return DCT_ERR_INVALID_ARG;
    drift_check_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream_)>>>(compress_result, k, ratio_num, ratio_den,
                                                                          flag_out);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}
