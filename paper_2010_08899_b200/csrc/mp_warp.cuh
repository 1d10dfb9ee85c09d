// Pieces shared by the warp-per-row forward kernels of DCT-MP (Algorithm 2): one warp finds the row
// threshold tau_i and packs the row (bf16: mp_pack.cu; fp32: mp_pack_f32.cu).
#pragma once
#include <type_traits>
#include <utility>

#include "common.cuh"

namespace dct {

constexpr int kFwdMaxWarps = 24;   // rows in flight per CTA (one CTA per SM; shared memory bounds it)
constexpr uint32_t kAbsMask2 = 0x7FFF7FFFu;
constexpr uint32_t kHistWords = 256u;       // one histogram of up to 256 bins per warp


__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t u) { return *reinterpret_cast<__nv_bfloat162*>(&u); }
__device__ __forceinline__ uint32_t as_u32(__nv_bfloat162 h) { return *reinterpret_cast<uint32_t*>(&h); }


__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ int dp4a_ss(uint32_t a, uint32_t b, int c) {     // signed 8-bit dot product + c
    int d;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
template <int kOffset> __device__ __forceinline__ uint4 lds128(uint32_t addr) {      // 128 bits at addr + kOffset
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+%5];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr), "n"(kOffset));
    return v;
}
// f(integral_constant<int, 0>) ... f(integral_constant<int, N - 1>): a loop whose index is a constant expression
template <typename F, int... Is> __device__ __forceinline__ void static_for_impl(F&& f, std::integer_sequence<int, Is...>) {
    (f(std::integral_constant<int, Is>{}), ...);
}
template <int N, typename F> __device__ __forceinline__ void static_for(F&& f) {
    static_for_impl(f, std::make_integer_sequence<int, N>{});
}
__device__ __forceinline__ uint32_t bfind(uint32_t x) {       // position of the highest set bit
    uint32_t d;
    asm("bfind.u32 %0, %1;" : "=r"(d) : "r"(x));
    return d;
}
// bit j set iff key(element j) >= low, for the 8 bf16 of one int4; exact for every bit pattern (low <= 0x8000).
// Per 16-bit half, bit 15 of ((x | 0x8000) - low) is set iff key(x) >= low, and no borrow crosses the halves.  A
// byte permutation picks the upper byte of every half with its sign bit replicated (0xFF = -1 or 0), and two
// signed dot products with the weights -2^j turn the eight bytes into the eight flags: 12 instructions.
__device__ __forceinline__ uint32_t mask8_ge_exact(uint4 v, uint32_t low) {
    const uint32_t low2 = low | (low << 16);
    const uint32_t t0 = (v.x | 0x80008000u) - low2;
    const uint32_t t1 = (v.y | 0x80008000u) - low2;
    const uint32_t t2 = (v.z | 0x80008000u) - low2;
    const uint32_t t3 = (v.w | 0x80008000u) - low2;
    const uint32_t a = prmt(t0, t1, 0xFDB9u);              // elements 0..3
    const uint32_t b = prmt(t2, t3, 0xFDB9u);              // elements 4..7
    return static_cast<uint32_t>(dp4a_ss(b, 0x80C0E0F0u, dp4a_ss(a, 0xF8FCFEFFu, 0)));
}

// upper halves of two fp32 words in one register: (hi16(b) << 16) | hi16(a)
__device__ __forceinline__ uint32_t upper_halves(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x7632); }
// Flags "upper 15 key bits >= low" of the 8 fp32 of one 32-byte piece, read as two 16-byte halves `first` and `second`
// (a lane reads the halves in either order; w_first / w_second are the dot-product weights -2^j of the four columns
// each half holds).  Exact for every bit pattern: per 16-bit half, bit 15 of ((x | 0x8000) - low) is set iff the
// key's upper bits are >= low; a byte permutation with sign replication and two signed dot products collect the
// eight flags, bit j = column j of the piece (see mask8_ge_exact in mp_warp.cuh).  low2 = low in both halves.
__device__ __forceinline__ uint32_t piece_flags(uint4 first, uint4 second, uint32_t low2, uint32_t w_first, uint32_t w_second) {
    const uint32_t t0 = (upper_halves(first.x, first.y) | 0x80008000u) - low2;
    const uint32_t t1 = (upper_halves(first.z, first.w) | 0x80008000u) - low2;
    const uint32_t t2 = (upper_halves(second.x, second.y) | 0x80008000u) - low2;
    const uint32_t t3 = (upper_halves(second.z, second.w) | 0x80008000u) - low2;
    return static_cast<uint32_t>(dp4a_ss(prmt(t2, t3, 0xFDB9u), w_second, dp4a_ss(prmt(t0, t1, 0xFDB9u), w_first, 0)));
}

// v = *(uint2*)shared_address if p (a predicated load: no branch)
__device__ __forceinline__ void lds64_if(uint2& v, uint32_t shared_address, bool p) {
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %3, 0;\n\t@q ld.shared.v2.u32 {%0, %1}, [%2];\n\t}"
                 : "+r"(v.x), "+r"(v.y) : "r"(shared_address), "r"(static_cast<uint32_t>(p)));
}

__device__ __forceinline__ uint32_t warp_inclusive_sum(uint32_t v) {
    const uint32_t lane = lane_id();
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= static_cast<uint32_t>(o)) v += t;
    }
    return v;
}

// hist holds 256 exponent bins.  Returns the exponent that holds rank k_rem
// (counting from exponent `top_exp` downwards) and reduces k_rem to the rank inside that exponent.
__device__ __forceinline__ uint32_t pick_exponent(const uint32_t* hist, uint32_t top_exp, uint32_t& k_rem) {
    const uint32_t lane = lane_id();
    for (int top = static_cast<int>(top_exp); top >= 0; top -= 32) {   // 32 exponents per step, highest first
        const int eb = top - static_cast<int>(lane);
        uint32_t c = 0;
        if (eb >= 0) {
            c = hist[eb];
        }
        const uint32_t inc = warp_inclusive_sum(c);
        const uint32_t hit = __ballot_sync(0xFFFFFFFFu, inc >= k_rem);
        if (hit) {
            const int src = __ffs(hit) - 1;
            k_rem -= __shfl_sync(0xFFFFFFFFu, inc - c, src);
            return static_cast<uint32_t>(top - src);
        }
        k_rem -= __shfl_sync(0xFFFFFFFFu, inc, 31);
    }
    return 0;
}
// hist[0..127] holds mantissa counts.  Returns the mantissa that holds rank k_rem from the top and the
// rank inside it (1-based: how many elements of that bin are still needed).
__device__ __forceinline__ uint32_t pick_mantissa(const uint32_t* hist, uint32_t k_rem, uint32_t& take) {
    const uint32_t lane = lane_id();
    // lane owns 4 bins, top-down: bin(lane, q) = 127 - (4 lane + q)
    const uint4 h = reinterpret_cast<const uint4*>(hist)[31 - lane];
    const uint32_t c[4] = {h.w, h.z, h.y, h.x};
    const uint32_t own = c[0] + c[1] + c[2] + c[3];
    uint32_t above = warp_inclusive_sum(own) - own, found = 0xFFFFFFFFu, found_take = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (above < k_rem && k_rem <= above + c[q]) {
            found = 127u - (4u * lane + q);
            found_take = k_rem - above;
        }
        above += c[q];
    }
    const uint32_t who = __ballot_sync(0xFFFFFFFFu, found != 0xFFFFFFFFu);
    const int src = who ? __ffs(who) - 1 : 0;
    take = __shfl_sync(0xFFFFFFFFu, found_take, src);
    return __shfl_sync(0xFFFFFFFFu, found, src) & 0x7Fu;
}

// General slow path for one row (rare): no usable bound, or very many elements tie at it.  tau_i is found
// bit by bit on the row itself, most significant first (the largest v with #{key >= v} >= k); then
// everything above tau_i and the first ties are written, in column order, straight from the row.
// Kept out of line so that the common path stays small in the instruction cache.
template <int E8>
__device__ __noinline__ void mp_row_slow_path(const unsigned char* span, uint32_t k, size_t out_base, uint32_t row,
                                              int16_t* __restrict__ cols_out, uint16_t* __restrict__ vals_out,
                                              int32_t* __restrict__ rows_out, uint16_t* __restrict__ tau_out) {
    constexpr uint32_t E = E8 * 8u;
    constexpr int kMaskWords = (E8 + 3) / 4;
    const uint32_t lane = lane_id();
    uint32_t tau_key = 0;
#pragma unroll 1
    for (int bit = 14; bit >= 0; --bit) {
        const uint32_t trial = tau_key | (1u << bit);
        uint32_t cnt = 0;
#pragma unroll 4
        for (int c = 0; c < E8; ++c)
            cnt += __popc(mask8_ge_exact(*reinterpret_cast<const uint4*>(span + c * 16), trial));
        if (__reduce_add_sync(0xFFFFFFFFu, cnt) >= k) tau_key = trial;
    }
    uint32_t gt_masks[kMaskWords], eq_masks[kMaskWords];
    uint32_t n_gt_mine = 0, n_eq_mine = 0;
#pragma unroll
    for (int i = 0; i < kMaskWords; ++i) gt_masks[i] = eq_masks[i] = 0;
#pragma unroll
    for (int c = 0; c < E8; ++c) {
        const uint4 v = *reinterpret_cast<const uint4*>(span + c * 16);
        const uint32_t gt = mask8_ge_exact(v, tau_key + 1u);
        const uint32_t eq = mask8_ge_exact(v, tau_key) & ~gt;
        gt_masks[c / 4] |= gt << (8 * (c % 4));
        eq_masks[c / 4] |= eq << (8 * (c % 4));
        n_gt_mine += __popc(gt);
        n_eq_mine += __popc(eq);
    }
    const uint32_t incl = warp_inclusive_sum(n_gt_mine);
    const uint32_t take = k - __shfl_sync(0xFFFFFFFFu, incl, 31);   // ties to keep, lowest columns first
    uint32_t g_at = incl - n_gt_mine;
    uint32_t e_at = warp_inclusive_sum(n_eq_mine) - n_eq_mine;
#pragma unroll
    for (int wd = 0; wd < kMaskWords; ++wd) {
        uint32_t m = gt_masks[wd] | eq_masks[wd];
        while (m) {
            const uint32_t bit = __ffs(m) - 1;
            m &= m - 1;
            const bool is_eq = (eq_masks[wd] >> bit) & 1u;
            if (!is_eq || e_at < take) {
                const uint32_t j = wd * 32 + bit;
                const size_t pos = out_base + g_at + (e_at < take ? e_at : take);
                cols_out[pos] = static_cast<int16_t>(lane * E + j);
                vals_out[pos] = *reinterpret_cast<const uint16_t*>(span + j * 2);
                if (rows_out) rows_out[pos] = static_cast<int32_t>(row);
            }
            g_at += is_eq ? 0u : 1u;
            e_at += is_eq ? 1u : 0u;
        }
    }
    if (lane == 0 && tau_out) tau_out[row] = static_cast<uint16_t>(tau_key);
}

// PL: candidates a lane holds in registers (5: k <= 112, rows of at most 1024 columns; 10: k <= 224; 20: k <= 448, with 4-element leaves for the
// exact bound, since 8-element leaves get loose as k approaches their number).
template <int PL> struct FwdVariant {
    static constexpr int kMaxWarps = PL <= 10 ? kFwdMaxWarps : 20;    // registers per thread grow with PL
    static constexpr bool kFineLeaves = PL > 10;
};


// Slot counts the tail of the sparse kernel is instantiated for besides PL itself: what rows mostly need when
// the guessed bound is accepted (k + a few dozen candidates rather than the k * 1.45 the exact bound may leave).
template <int PL> struct FwdTrips;
template <> struct FwdTrips<5> { static constexpr uint32_t kFew = 3, kSome = 4; };
template <> struct FwdTrips<10> { static constexpr uint32_t kFew = 8, kSome = 9; };
template <> struct FwdTrips<20> { static constexpr uint32_t kFew = 15, kSome = 17; };

// Warps per CTA when there are fewer rows than row slots on the device: the rows are spread over all SMs (fewer
// warps per CTA) instead of filling some SMs and leaving the others idle.
inline size_t warps_for_rows(size_t max_warps, uint32_t rows, int sms) {
    const size_t per_sm = (static_cast<size_t>(rows) + static_cast<size_t>(sms) - 1) / static_cast<size_t>(sms);
    return per_sm >= max_warps ? max_warps : (per_sm < 1 ? 1 : per_sm);
}

// Which sparse warp-per-row variant fits a shape: candidates per lane (5, 10 or 20), or 0 if none does.
// The exact bound (k-th largest leaf maximum) leaves k * r candidates, where r grows as k approaches the
// number of leaves L: measured 99th percentiles on post-ReLU rows with log-normal column scales are
// r = 1.43 / 1.53 / 1.67 / 1.84 / 2.14 at k/L = 0.4 / 0.5 / 0.6 / 0.7 / 0.8 and the bound degenerates beyond.
// 8-element leaves (L = d/8) serve 5 or 10 candidates per lane, 4-element leaves (L = d/4) serve 20.
inline int fwd_candidates_per_lane(uint32_t d, uint32_t k) {
    auto need = [](uint32_t k_, uint32_t leaves) -> uint32_t {      // candidates to provide room for, 0: bound too loose
        if (leaves == 0) return 0;
        const uint32_t pct = (100u * k_ + leaves - 1) / leaves;
        const uint32_t r = pct <= 40 ? 145 : pct <= 50 ? 155 : pct <= 60 ? 170 : pct <= 70 ? 190 : pct <= 80 ? 220 : 0;
        return r == 0 ? 0u : (k_ * r + 99u) / 100u;
    };
    const uint32_t n8 = need(k, d / 8), n4 = need(k, d / 4);
    if (n8 != 0 && n8 <= 160 && d <= 1024) return 5;
    if (n8 != 0 && n8 <= 320) return 10;
    if (n4 != 0 && n4 <= 640) return 20;
    return 0;
}

// Rows of 256 or 512 bf16 columns: the row stays in registers, several rows per warp (mp_pack_narrow.cu).
dct_status_t launch_fwd_bf16_narrow(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                    int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                    dct_result_t* result, cudaStream_t stream, bool* handled);

// The same for fp32 rows of 256 columns.
dct_status_t launch_fwd_f32_narrow(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                   int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                   dct_result_t* result, cudaStream_t stream, bool* handled);

// bf16, every lane looking after one contiguous span of the row (mp_pack_span.cu).
dct_status_t launch_fwd_bf16_span(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                  int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                  dct_result_t* result, cudaStream_t stream, bool* handled);

// The fp32 kernels live in their own translation unit.
dct_status_t launch_fwd_f32_warp(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                 int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                 dct_result_t* result, cudaStream_t stream, bool* handled);
// fp32 rows of 513..32768 columns, one CTA per row (mp_pack_f32_wide.cu).
dct_status_t launch_fwd_f32_wide(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                 int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                 dct_result_t* result, cudaStream_t stream, bool* handled);

// The per-row thresholds alone by the CTA-per-row kernels (mp_pack_span.cu, mp_pack_f32_wide.cu).
dct_status_t launch_tau_bf16_wide(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, void* tau_out,
                                  cudaStream_t stream, bool* handled);
dct_status_t launch_tau_f32_wide(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, void* tau_out,
                                 cudaStream_t stream, bool* handled);

}  // namespace dct
