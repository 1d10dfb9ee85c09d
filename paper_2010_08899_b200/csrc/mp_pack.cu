// dct_mp_topk_pack_fwd / dct_mp_pack_bwd: Algorithm 2 (DCT-MP).
//
// Forward.  Every kernel reads a row from HBM exactly once, finds the row threshold tau_i (k-th largest
// magnitude) on chip and writes the kept columns -- every key above tau_i plus the lowest-column ties --
// in ascending column order together with their values.  The int16 column list is the mask M.
//   * general kernel (this file): one CTA per row, any dtype / width / stride / k; tau_i by a radix select
//     over the row in shared memory (row_select.cuh).
//   * bf16, sparse k, rows up to 4096 columns on 16-byte boundaries (this file): one warp per row, the
//     candidates above a bound in registers.
//   * bf16, denser k (mp_pack_span.cu): one warp per row, every lane looking after a contiguous span of the row,
//     tau_i pinned between two bounds.
//   * bf16, rows of 256 / 512 columns: several rows per warp, rows in registers (mp_pack_narrow.cu).
//   * fp32, sparse k: one warp per row (mp_pack_f32.cu).
// dct_mp_topk_pack_fwd (end of this file) picks among them.
//
// Backward: a gather of X_grad through the column list, one warp per row.
#include "common.cuh"
#include "row_select.cuh"
#include "mp_warp.cuh"

namespace dct {
namespace {

constexpr int kMaxWarps = 32;

template <typename T>
__global__ void mp_topk_pack_fwd_kernel(const T* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                        int16_t* __restrict__ cols_out, T* __restrict__ vals_out,
                                        int32_t* __restrict__ rows_out, T* __restrict__ tau_out,
                                        dct_result_t* __restrict__ result, bool rows_aligned16) {
    using Tr = ElemTraits<T>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    T* row_s = reinterpret_cast<T*>(smem_raw);
    __shared__ uint32_t s_hist[256];
    __shared__ uint32_t s_sel[2];
    __shared__ uint32_t s_wcnt[kMaxWarps];   // (gt << 16) | eq per warp; both <= 32768 / warps... see below

    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    const uint32_t lane = tid & 31u, warp = tid >> 5, nwarps = nt >> 5;
    if (blockIdx.x == 0 && tid == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }
    // each warp owns a contiguous span of columns (multiple of 32) for the ordered emit
    const uint32_t span = ((d + nwarps * 32u - 1u) / (nwarps * 32u)) * 32u;

    for (uint32_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const T* xr = x + static_cast<size_t>(row) * ld;
        // ---- stage the row in shared memory (one HBM read) ---------------------------------
        if (rows_aligned16) {
            constexpr uint32_t per16 = 16 / sizeof(T);
            const uint32_t nvec = d / per16;
            const int4* src = reinterpret_cast<const int4*>(xr);
            int4* dst = reinterpret_cast<int4*>(row_s);
            for (uint32_t v = tid; v < nvec; v += nt) {
                int4 t;
                asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(t.x), "=r"(t.y), "=r"(t.z), "=r"(t.w) : "l"(src + v));
                dst[v] = t;
            }
            for (uint32_t j = nvec * per16 + tid; j < d; j += nt) row_s[j] = xr[j];
        } else {
            for (uint32_t j = tid; j < d; j += nt) row_s[j] = xr[j];
        }
        // ---- radix select of the k-th largest key ------------------------------------------
        uint32_t tau_key, take;      // take: ties (key == tau_key) to keep, lowest columns first
        cta_row_select<T>(row_s, d, k, s_hist, s_sel, tau_key, take);
        if (tid == 0 && tau_out) tau_out[row] = Tr::from_key(tau_key);

        // ---- ordered emit: count per warp, then write ----------------------------------------
        const uint32_t c0 = warp * span;
        const uint32_t c1 = (c0 + span < d) ? c0 + span : d;
        uint32_t n_gt = 0, n_eq = 0;
        for (uint32_t base = c0; base < c1; base += 32) {
            const uint32_t j = base + lane;
            const uint32_t key = (j < c1) ? Tr::key(row_s[j]) : 0u;
            n_gt += __popc(__ballot_sync(0xFFFFFFFFu, j < c1 && key > tau_key));
            n_eq += __popc(__ballot_sync(0xFFFFFFFFu, j < c1 && key == tau_key));
        }
        if (lane == 0) s_wcnt[warp] = (n_gt << 16) | n_eq;   // n_gt < k <= 32768 and n_eq <= 32768: see note
        __syncthreads();
        uint32_t g_run = 0, e_run = 0;
        for (uint32_t v = 0; v < warp; ++v) {
            const uint32_t t = s_wcnt[v];
            g_run += t >> 16;
            e_run += t & 0xFFFFu;
        }
        const size_t out_base = static_cast<size_t>(row) * k;
        for (uint32_t base = c0; base < c1; base += 32) {
            if (g_run + (e_run < take ? e_run : take) >= k) break;   // all k slots already written
            const uint32_t j = base + lane;
            const bool valid = j < c1;
            const T v = valid ? row_s[j] : T(0);
            const uint32_t key = Tr::key(v);
            const bool is_gt = valid && key > tau_key, is_eq = valid && key == tau_key;
            const uint32_t bg = __ballot_sync(0xFFFFFFFFu, is_gt), be = __ballot_sync(0xFFFFFFFFu, is_eq);
            const uint32_t lt = lanemask_lt();
            const uint32_t gt_before = g_run + __popc(bg & lt);
            const uint32_t eq_before = e_run + __popc(be & lt);
            if (is_gt || (is_eq && eq_before < take)) {
                const uint32_t pos = gt_before + (eq_before < take ? eq_before : take);
                cols_out[out_base + pos] = static_cast<int16_t>(j);
                vals_out[out_base + pos] = v;
                if (rows_out) rows_out[out_base + pos] = static_cast<int32_t>(row);
            }
            g_run += __popc(bg);
            e_run += __popc(be);
        }
        __syncthreads();   // row_s, s_hist, s_prefix are reused by the next row
    }
}

// One element of the gradient matrix through the read-only path without a line in L1: the kept columns of a row
// touch every 128-byte line about once, so an L1 line is never hit again (the backward pack alone: 24.8 -> 22.6 us
// at 16384 x 4096 bf16).  What reaches DRAM is the same with every flavour of load: whole 128-byte lines.
template <typename T> __device__ __forceinline__ T gather_load(const T* p) {
    if constexpr (sizeof(T) == 2) {
        uint16_t v;
        asm volatile("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(v) : "l"(p));
        return *reinterpret_cast<T*>(&v);
    } else {
        uint32_t v;
        asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
        return *reinterpret_cast<T*>(&v);
    }
}

// The result block is reset inside the kernel (no memset node, no reset kernel on the stream).  Thread 0 of CTA 0
// clears it and then publishes the launch's ticket in `reserved` (release); a warp that has met a bad column
// waits (bounded) for that ticket before it raises the status, so the reset can never wipe a report.
template <typename T>
__global__ void __launch_bounds__(256)
mp_pack_bwd_kernel(const T* __restrict__ gx, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                   const int16_t* __restrict__ cols, T* __restrict__ gvals, dct_result_t* __restrict__ result,
                   uint32_t ticket) {
    const uint32_t lane = lane_id();
    const uint32_t warps_per_cta = blockDim.x >> 5;
    bool bad = false;
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&result->reserved), "r"(ticket) : "memory");
    }
    for (uint64_t row = static_cast<uint64_t>(blockIdx.x) * warps_per_cta + (threadIdx.x >> 5); row < rows;
         row += static_cast<uint64_t>(gridDim.x) * warps_per_cta) {
        const T* gr = gx + row * ld;
        const int16_t* cr = cols + row * k;
        T* out = gvals + row * k;
        for (uint32_t s0 = 0; s0 < k; s0 += 128) {
            uint32_t c[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t s = s0 + u * 32 + lane;
                c[u] = (s < k) ? static_cast<uint16_t>(__ldg(cr + s)) : 0u;
            }
            T v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t s = s0 + u * 32 + lane;
                const bool ok = c[u] < d;
                if (s < k && !ok) bad = true;
                v[u] = (s < k && ok) ? gather_load(gr + c[u]) : T(0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t s = s0 + u * 32 + lane;
                if (s < k) out[s] = v[u];
            }
        }
    }
    if (bad && result) {
        for (uint32_t spin = 0; spin < (1u << 20); ++spin) {          // CTA 0 is dispatched first: normally no wait at all
            uint32_t seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(&result->reserved) : "memory");
            if (seen == ticket) break;
        }
        atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_BAD_MASK));
    }
}

// The same for small k (fewer kept columns than lanes): one THREAD per kept entry, the rows' entries taken as one list
// of rows * k -- with a warp per row only k of 32 lanes work (1572864 rows of 64 columns, k = 3: 0.215 ms).  A thread
// takes four entries blockDim apart per round; row and position inside the row advance by fixed steps, so only the first
// entry of a thread costs a division.
template <typename T>
__global__ void __launch_bounds__(256)
mp_pack_bwd_flat_kernel(const T* __restrict__ gx, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                        const int16_t* __restrict__ cols, T* __restrict__ gvals, dct_result_t* __restrict__ result,
                        uint32_t ticket) {
    bool bad = false;
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&result->reserved), "r"(ticket) : "memory");
    }
    const uint64_t total = static_cast<uint64_t>(rows) * k;
    const uint32_t step_q = blockDim.x / k, step_r = blockDim.x % k;                        // one step of blockDim entries
    const uint64_t round = static_cast<uint64_t>(gridDim.x) * blockDim.x * 4u;              // one round of the grid
    const uint64_t round_q = round / k;
    const uint32_t round_r = static_cast<uint32_t>(round % k);
    uint64_t e0 = static_cast<uint64_t>(blockIdx.x) * blockDim.x * 4u + threadIdx.x;
    uint64_t row0 = e0 / k;
    uint32_t s0 = static_cast<uint32_t>(e0 - row0 * k);
    for (; e0 < total; e0 += round) {
        uint32_t c[4];
        uint64_t row[4];
        uint64_t r = row0;
        uint32_t s = s0;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint64_t e = e0 + static_cast<uint64_t>(u) * blockDim.x;
            row[u] = r;
            c[u] = e < total ? static_cast<uint16_t>(__ldg(cols + e)) : 0u;
            r += step_q;
            s += step_r;
            if (s >= k) {
                s -= k;
                ++r;
            }
        }
        T v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint64_t e = e0 + static_cast<uint64_t>(u) * blockDim.x;
            const bool ok = c[u] < d;
            if (e < total && !ok) bad = true;
            v[u] = (e < total && ok) ? gather_load(gx + row[u] * ld + c[u]) : T(0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint64_t e = e0 + static_cast<uint64_t>(u) * blockDim.x;
            if (e < total) gvals[e] = v[u];
        }
        row0 += round_q;
        s0 += round_r;
        if (s0 >= k) {
            s0 -= k;
            ++row0;
        }
    }
    if (bad && result) {
        for (uint32_t spin = 0; spin < (1u << 20); ++spin) {          // CTA 0 is dispatched first: normally no wait at all
            uint32_t seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(&result->reserved) : "memory");
            if (seen == ticket) break;
        }
        atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_BAD_MASK));
    }
}

// ------------------------------------------------------------------------------------------
// bf16 fast path: one warp per row, d <= 8192 a multiple of 8 (held in a buffer of 256 * E8 columns), rows on 16-byte boundaries
// ------------------------------------------------------------------------------------------
// One bulk asynchronous copy brings a row into shared memory exactly as it lies in HBM; the next row is
// requested as soon as the candidates of the current one sit in registers.
//   A  a lower bound `low` for tau_i.  First guess: the previous row's tau_i minus a margin (thresholds of
//      neighbouring samples are close).  If that leaves fewer than k or too many candidates, the exact
//      bound takes over: the k-th largest of the maxima of the aligned 8-element (or 4-element) leaves --
//      at least k elements are >= it, and fewer than k leaves hold anything above it.
//   B  one pass over the row (lane l reads the 16-byte units l, l + 32, ...: conflict-free for every width)
//      writes one flag per column, key >= low, into a bit table in column order; a warp scan over the
//      per-lane counts gives the number of candidates before every table word.
//   C  the candidates (typically ~1.3 k) are dealt out evenly, in column order, ceil(n/32) to a lane, which
//      finds its first one by bisection over the running counts and walks the table from there.
//   D  exact k-th largest of the candidates: a 64-bin histogram just above the bound, else a radix select
//      (exponent byte, then mantissa).
//   E  the kept entries (key > tau_i, then the lowest-column ties) go, in column order, through k staging
//      slots to coalesced stores.
// If the candidates do not fit the registers (heavy ties at the bound, or k larger than the number of
// leaves), the row takes a slow general path: tau_i is found bit by bit by counting over the row, and the
// output is written straight from the row.
template <int E8> struct WarpRowLayout {
    static constexpr uint32_t E = E8 * 8u;                   // columns per lane of the buffer (256 * E8 columns in all)
    static constexpr uint32_t kSpanBytes = E * 2u;           // the row lies in shared memory as it does in HBM
    static constexpr uint32_t kRowBytes = 32u * kSpanBytes;
    static constexpr uint32_t kRowWords = 8u * E8;           // 32-bit candidate-mask words of a row (one bit per column)
    static constexpr uint32_t kMaskWords = (E8 + 3) / 4;     // mask words a lane looks after: lane l has words [l kMaskWords, (l+1) kMaskWords)
    static constexpr uint32_t kTableWords = 32u * kMaskWords;
    // per warp: row | scratch | mbarrier.  The scratch is used in turn, never at the same time, as the
    // leaf histogram, the candidate-mask and running-count tables, the select histogram and the k
    // staging slots of the output.
    __host__ __device__ static constexpr uint32_t scratch_words(uint32_t k) {
        uint32_t w = 2u * kTableWords > kHistWords ? 2u * kTableWords : kHistWords;
        return w > ((k + 3u) & ~3u) ? w : ((k + 3u) & ~3u);
    }
    __host__ __device__ static constexpr uint32_t warp_bytes(uint32_t k) {
        return kRowBytes + scratch_words(k) * 4u + 16u;
    }
};

// Warps of a CTA: as many row buffers as shared memory holds (wide rows leave fewer warps and therefore more
// registers for each of them), at most 32 with up to 10 candidates per lane (the kernel then fits 64 registers;
// 32 warps against 24 are worth 7 to 11 % on rows of 2048 and 1024 columns) and 24 with 20 per lane.
template <int E8, int PL> constexpr int fwd_bf16_max_warps() {
    constexpr int by_smem = static_cast<int>((220u * 1024u) / WarpRowLayout<E8>::warp_bytes(1));
    constexpr int by_regs = PL <= 10 ? 32 : 24;
    return by_smem < by_regs ? by_smem : by_regs;
}

template <int E8, int PL>
__global__ void __launch_bounds__(fwd_bf16_max_warps<E8, PL>() * 32)
mp_topk_fwd_bf16_warp_kernel(const uint16_t* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                             int16_t* __restrict__ cols_out, uint16_t* __restrict__ vals_out,
                             int32_t* __restrict__ rows_out, uint16_t* __restrict__ tau_out,
                             dct_result_t* __restrict__ result, bool few_slots) {
    using Lay = WarpRowLayout<E8>;
    constexpr int kMaskWords = Lay::kMaskWords;
    constexpr uint32_t kPerLane = PL, kRound = 32u * kPerLane;   // candidates a lane holds in registers at a time
    constexpr bool kFineLeaves = FwdVariant<PL>::kFineLeaves;
    constexpr int kLeaves = kFineLeaves ? 2 * E8 : E8;           // leaves per lane (4 or 8 elements each)
    constexpr uint32_t kGuessMargin = 32;  // keys (a quarter of a binade) below the previous tau_i
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned char* base = smem_raw + warp * Lay::warp_bytes(k);
    unsigned char* span = base + lane * Lay::kSpanBytes;
    uint32_t* scratch = reinterpret_cast<uint32_t*>(base + Lay::kRowBytes);
    uint32_t* mask_tab = scratch;                             // one bit per column (key >= bound), column order
    uint2* table = reinterpret_cast<uint2*>(scratch);        // per mask word: {mask, running count and link}, built after the bit table
    uint32_t* hist = scratch;                                 // histograms (before / after the tables are in use)
    uint32_t* stage = scratch;                                // the k kept entries, column order (last use)
    uint64_t* bar = reinterpret_cast<uint64_t*>(scratch + Lay::scratch_words(k));
    __shared__ uint32_t s_stop;
    __shared__ uint32_t s_next;                               // rows of this CTA handed out so far
    __shared__ uint32_t s_hint;                               // the latest bound any warp of this CTA guessed from a tau_i

    if (threadIdx.x == 0) {
        s_stop = 0;
        s_next = blockDim.x >> 5;
        s_hint = 0;
    }
    if (lane == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
        fence_proxy_async_all();
    }
    // A row of d <= D columns (d a multiple of 8) fills the first d columns of the buffer; the rest is zeroed
    // once and never written again: zeros lie below every bound and, being the last columns, lose every tie.
    const uint32_t row_bytes = d * 2u;
    for (uint32_t b = row_bytes + lane * 16u; b < Lay::kRowBytes; b += 512u)
        *reinterpret_cast<uint4*>(base + b) = make_uint4(0, 0, 0, 0);
    __syncthreads();
    // Everything above is set-up in shared memory; the kernel before this one on the stream (which may have
    // produced x or may still read the outputs) must have finished before anything below.
    chain_wait_previous();
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }

    // Rows are dealt out CTA by CTA (row mod grid = CTA): every SM gets the same number of rows to within one.
    // Inside the CTA a warp takes the CTA's next row whenever it lets go of one (a counter in shared memory): the
    // warps drift apart by up to a row's time, and the rows of the last, partly filled round go to the warps that
    // are ahead instead of to fixed ones.
    const uint32_t warp_global = blockIdx.x + gridDim.x * warp;             // this warp's first row
    auto request_row = [&](uint32_t r) {          // one bulk copy brings the whole row
        if (lane == 0) {
            mbar_arrive_expect_tx(bar, row_bytes);
            bulk_load(base, x + static_cast<size_t>(r) * ld, row_bytes, bar);
        }
    };
    // In the passes over the whole row lane l reads the 16-byte units l, l + 32, l + 64, ...: the 32 lanes of a
    // 128-bit load then touch 512 consecutive bytes (no bank conflict for any row width).
    const unsigned char* unit0 = base + lane * 16u;
    uint64_t next_row = 0;
    auto release_row = [&]() {               // the row buffer is no longer needed: request the next row
        __syncwarp();
        fence_proxy_async_smem();
        uint32_t j = 0;
        if (lane == 0) j = atomicAdd(&s_next, 1u);
        j = __shfl_sync(0xFFFFFFFFu, j, 0);
        next_row = blockIdx.x + static_cast<uint64_t>(gridDim.x) * j;
        if (next_row < rows) request_row(static_cast<uint32_t>(next_row));
    };
    if (warp_global < rows) request_row(warp_global);

    uint32_t use = 0;
    uint32_t guess_low = 0;                         // bound guessed from the previous row (0: none)
    for (uint64_t row64 = warp_global; row64 < rows; row64 = next_row, ++use) {
        const uint32_t row = static_cast<uint32_t>(row64);
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(bar, use & 1u, 1u << 24, &s_stop))) {
            s_stop = 1;
            if (lane == 0 && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
            return;
        }
        const size_t out_base = static_cast<size_t>(row) * k;

        // ---- A: a lower bound for tau_i --------------------------------------------------------------
        uint32_t row_max = 0x7FFFu;                  // only the exact bound computes the true maximum
        const bool have_bound = k <= 32u * kLeaves;  // otherwise there are fewer leaves than k
        auto exact_bound = [&]() -> uint32_t {
            // maxima of the leaves: the 8 elements of a 16-byte unit, or (fine leaves) its even and its odd
            // elements separately -- any partition of the row into at least k groups will do
            uint32_t leaf[kLeaves];
            uint32_t top = 0;
#pragma unroll
            for (int c = 0; c < E8; ++c) {
                const uint4 v = *reinterpret_cast<const uint4*>(unit0 + c * 512);
                const __nv_bfloat162 m2 = __hmax2(__hmax2(__habs2(as_bf162(v.x)), __habs2(as_bf162(v.y))),
                                                  __hmax2(__habs2(as_bf162(v.z)), __habs2(as_bf162(v.w))));
                const uint32_t m = as_u32(m2);
                if (kFineLeaves) {
                    leaf[2 * c] = m & 0xFFFFu;
                    leaf[2 * c + 1] = m >> 16;
                    top = max(top, max(leaf[2 * c], leaf[2 * c + 1]));
                } else {
                    leaf[c] = max(m & 0xFFFFu, m >> 16);
                    top = max(top, leaf[c]);
                }
            }
            row_max = __reduce_max_sync(0xFFFFFFFFu, top);
            if (!have_bound) return 0u;
            // One histogram pass over the leaf maxima in bins of 8 keys counted down from the row maximum
            // (bin 255 collects everything further away).  The bound is the lowest key of the bin in which
            // the count reaches k: at least k leaves, hence k elements, lie at or above it.
            reinterpret_cast<uint4*>(hist)[lane] = make_uint4(0, 0, 0, 0);
            reinterpret_cast<uint4*>(hist)[lane + 32] = make_uint4(0, 0, 0, 0);
            __syncwarp();
#pragma unroll
            for (int c = 0; c < kLeaves; ++c) {
                const uint32_t rel = (row_max - leaf[c]) >> 3;
                atomicAdd(&hist[rel < 255u ? rel : 255u], 1u);
            }
            __syncwarp();
            uint32_t need = k, bin = 255;
#pragma unroll 1
            for (uint32_t first = 0; first < 256; first += 32) {
                const uint32_t c = hist[first + lane];
                const uint32_t inc = warp_inclusive_sum(c);
                const uint32_t hit = __ballot_sync(0xFFFFFFFFu, inc >= need);
                if (hit) {
                    bin = first + (__ffs(hit) - 1);
                    break;
                }
                need -= __shfl_sync(0xFFFFFFFFu, inc, 31);
            }
            __syncwarp();
            const uint32_t span_keys = bin * 8u + 7u;
            return (bin < 255u && row_max > span_keys) ? row_max - span_keys : 0u;
        };

        // ---- B: candidate masks (key >= low), in column order ------------------------------------------
        uint32_t masks[kMaskWords];
        uint32_t n_mine = 0, incl = 0, n_cand = 0;
        auto build_masks = [&](uint32_t bound, bool probe) -> bool {
            // unit u = 32 c + lane covers columns 8 u .. 8 u + 7: its 8 flags are byte u of the mask table, which
            // therefore holds one bit per column, in column order
            unsigned char* tab8 = reinterpret_cast<unsigned char*>(mask_tab) + lane;
            {
                const uint32_t m0 = mask8_ge_exact(*reinterpret_cast<const uint4*>(unit0), bound);
                tab8[0] = static_cast<unsigned char>(m0);
                // A guessed bound is probed on the first unit of every lane (1 / E8 of the row): if that sample says
                // that the candidates will be far too few or far too many, the rest of the pass is not worth making
                // (rows whose scale differs from the previous row's).  Only a saving: the guess is checked exactly below.
                if (E8 >= 8 && probe) {
                    const uint32_t sample = __reduce_add_sync(0xFFFFFFFFu, __popc(m0)) * E8;
                    if (8u * sample < 5u * k || 5u * sample > 8u * kRound) {
                        n_cand = 0;
                        return false;
                    }
                }
            }
#pragma unroll
            for (int c = 1; c < E8; ++c)
                tab8[c * 32] = static_cast<unsigned char>(
                    mask8_ge_exact(*reinterpret_cast<const uint4*>(unit0 + c * 512), bound));
            __syncwarp();
            // the lane's own words: columns 32 kMaskWords lane onwards (words past the end of the row are empty)
            if (kMaskWords == 4) {
                const uint4 t = reinterpret_cast<const uint4*>(mask_tab)[lane];
                masks[0] = t.x; masks[1 % kMaskWords] = t.y; masks[2 % kMaskWords] = t.z; masks[3 % kMaskWords] = t.w;
            } else if (kMaskWords == 2) {
                const uint2 t = reinterpret_cast<const uint2*>(mask_tab)[lane];
                masks[0] = t.x; masks[1 % kMaskWords] = t.y;
            } else {
#pragma unroll
                for (int i = 0; i < kMaskWords; ++i) masks[i] = mask_tab[lane * kMaskWords + i];
            }
            if (Lay::kRowWords != Lay::kTableWords) {
#pragma unroll
                for (int i = 0; i < kMaskWords; ++i)
                    if (lane * kMaskWords + i >= Lay::kRowWords) masks[i] = 0u;
            }
            n_mine = 0;
#pragma unroll
            for (int i = 0; i < kMaskWords; ++i) n_mine += __popc(masks[i]);
            incl = warp_inclusive_sum(n_mine);
            n_cand = __shfl_sync(0xFFFFFFFFu, incl, 31);
            return true;
        };

        // Thresholds of neighbouring samples are close (the observation behind the paper's threshold
        // life-span, applied across rows): first try the previous row's tau_i minus a margin as the bound.
        // It is only a guess -- it is accepted if it leaves at least k and not too many candidates, and the
        // exact leaf bound takes over otherwise -- so the result never depends on it.
        uint32_t low = 0;
        // a warp that has no row behind it borrows the latest guess of its CTA
        if (guess_low == 0) guess_low = *reinterpret_cast<volatile uint32_t*>(&s_hint);
        bool use_guess = have_bound && guess_low != 0;
#pragma unroll 1
        while (true) {
            low = use_guess ? guess_low : exact_bound();
            const bool built = build_masks(low, use_guess);
            if (!use_guess || (built && n_cand >= k && n_cand <= kRound)) break;
            use_guess = false;
        }
        if (!have_bound || n_cand > kRound || low == 0) {
            mp_row_slow_path<E8>(span, k, out_base, row, cols_out, vals_out, rows_out, tau_out);
            release_row();
            continue;
        }

        // ---- candidates into registers, evenly -------------------------------------------------------
        // Every table word becomes an entry {mask, candidates before it << 16 | index of the next non-empty
        // word}.  A lane finds the word that holds its first candidate by bisection over the running counts and
        // walks on from there; the link takes it over any run of empty words in one step.
        uint32_t first_word;                                    // the row's first non-empty word
        {
            const uint32_t wbase = lane * kMaskWords;
            uint32_t my_first = Lay::kTableWords;               // the lane's first non-empty word
#pragma unroll
            for (int i = kMaskWords - 1; i >= 0; --i)
                if (masks[i]) my_first = wbase + i;
            // after the last non-empty word the link wraps to the first one: a walk that runs past its candidates
            // (unused slots) then still meets a non-empty word, and its result is discarded
            const uint32_t holders = __ballot_sync(0xFFFFFFFFu, n_mine != 0);
            const uint32_t later = holders & (0xFFFFFFFEu << lane);
            first_word = __shfl_sync(0xFFFFFFFFu, my_first, __ffs(holders) - 1);
            // (all lanes take part in the shuffle; the source lane is the next holder, or the first one to wrap)
            uint32_t link = __shfl_sync(0xFFFFFFFFu, my_first, __ffs(later ? later : holders) - 1);
            uint32_t next_of[kMaskWords];
#pragma unroll
            for (int i = kMaskWords - 1; i >= 0; --i) {
                next_of[i] = link;
                if (masks[i]) link = wbase + i;
            }
            uint32_t before = incl - n_mine;
            if (kMaskWords == 4) {
                uint32_t y[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    y[i] = (before << 16) | next_of[i % kMaskWords];
                    before += __popc(masks[i % kMaskWords]);
                }
                uint4* t4 = reinterpret_cast<uint4*>(table + wbase);
                t4[0] = make_uint4(masks[0], y[0], masks[1 % kMaskWords], y[1]);
                t4[1] = make_uint4(masks[2 % kMaskWords], y[2], masks[3 % kMaskWords], y[3]);
            } else {
#pragma unroll
                for (int i = 0; i < kMaskWords; ++i) {
                    table[wbase + i] = make_uint2(masks[i], (before << 16) | next_of[i]);
                    before += __popc(masks[i]);
                }
            }
        }
        __syncwarp();
        // The rest of the row's work runs over the slots a lane holds.  per_lane varies from row to row (2 or 3 for
        // k = 52 of 1024 columns, 4 or 5 for k = 102 of 2048), so for rows of up to 3072 columns the code is
        // instantiated for three slot counts and the row takes the smallest that fits: the loops below are unrolled
        // over exactly that many slots (4 to 11 % faster there).  The kernels for wider rows are larger and lose
        // more to the extra code than they gain (4096 columns: 16 % slower with three copies, 3 % with two).
        const uint32_t per_lane = (n_cand + 31u) >> 5;
        auto finish_row = [&](auto trips_tag) {
            constexpr uint32_t kTrips = decltype(trips_tag)::value;
            // Every lane takes per_lane = ceil(n_cand / 32) consecutive candidates (the last lanes fewer or none).  An unused
            // slot holds 0: its key is below the bound (low >= 1 here), so the select and the emit skip it unaided.
            uint32_t ent[kTrips];
            const uint32_t first = lane * per_lane;                 // rank of the lane's first candidate
            const uint32_t nvalid = first >= n_cand ? 0u : (n_cand - first < per_lane ? n_cand - first : per_lane);
            {
                uint32_t word = 0, m = 0, link = first_word;
                if (kMaskWords == 4) {
                    // the lane whose words hold rank `first`: the last one with (candidates before it) <= first, found
                    // by a binary search over the lanes' running counts (every lane takes part in the shuffles)
                    const uint32_t excl = incl - n_mine;
                    const uint32_t pc = __popc(masks[0]) | (__popc(masks[1 % kMaskWords]) << 8) | (__popc(masks[2 % kMaskWords]) << 16);
                    uint32_t owner = 0, owner_excl = 0;
#pragma unroll
                    for (int step = 16; step > 0; step >>= 1) {
                        const uint32_t v = __shfl_sync(0xFFFFFFFFu, excl, owner + step);
                        if (v <= first) {
                            owner += step;
                            owner_excl = v;
                        }
                    }
                    const uint32_t opc = __shfl_sync(0xFFFFFFFFu, pc, owner);
                    if (nvalid) {
                        const uint32_t r = first - owner_excl;          // rank inside the owner's four words
                        const uint32_t p0 = opc & 0xFFu, p01 = p0 + ((opc >> 8) & 0xFFu), p012 = p01 + (opc >> 16);
                        const uint32_t i = (r >= p0 ? 1u : 0u) + (r >= p01 ? 1u : 0u) + (r >= p012 ? 1u : 0u);
                        const uint2 e = table[owner * 4u + i];
                        word = owner * 4u + i;
                        m = e.x;
                        link = e.y & 0xFFFFu;
                        for (uint32_t skip = r - (i == 0 ? 0u : (i == 1 ? p0 : (i == 2 ? p01 : p012))); skip; --skip) m &= m - 1;
                    }
                } else if (nvalid) {
                    uint32_t lo = 0, hi = Lay::kTableWords - 1;         // largest word with (candidates before it) <= first
                    const uint32_t limit = (first + 1u) << 16;
                    while (lo < hi) {
                        const uint32_t mid = (lo + hi + 1) >> 1;
                        if (table[mid].y < limit) lo = mid; else hi = mid - 1;
                    }
                    const uint2 e = table[lo];
                    word = lo;
                    m = e.x;
                    link = e.y & 0xFFFFu;
                    for (uint32_t skip = first - (e.y >> 16); skip; --skip) m &= m - 1;
                }
                // `ahead` is the entry the walk moves to when the current word runs out; it is fetched when the walk
                // arrives at a word, long before it is needed
                uint2 ahead = table[link];
                const uint32_t table_addr = smem_addr(table);
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const bool advance = (m == 0);
                    m = advance ? ahead.x : m;
                    word = advance ? link : word;
                    link = advance ? (ahead.y & 0xFFFFu) : link;
                    lds64_if(ahead, table_addr + link * 8u, advance);
                    const uint32_t col = word * 32u + (__ffs(m) - 1);
                    m &= m - 1;
                    const uint32_t e = reinterpret_cast<const uint16_t*>(base)[col] | (col << 16);
                    ent[i] = static_cast<uint32_t>(i) < nvalid ? e : 0u;
                }
            }
            release_row();

            // ---- C: k-th largest of the candidates --------------------------------------------------
            uint32_t tau_key = 0, take = 0;
            bool found = false;
            {
                // tau_i is the (n_cand - k + 1)-th smallest candidate.  Usually it lies within 64 keys of the
                // bound: a 64-bin histogram of the candidates in [low, low + 64), walked from the bottom, finds it.
                const uint32_t drop = n_cand - k;                 // candidates to discard, smallest first
                // (everything beyond the window, unused slots included, goes to a bin of the lane's own: no branch)
                hist[lane] = 0;
                hist[lane + 32] = 0;
                hist[lane + 64] = 0;
                __syncwarp();
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t rel = (ent[i] & 0x7FFFu) - low;
                    atomicAdd(&hist[min(rel, 64u + lane)], 1u);
                }
                __syncwarp();
                const uint2 h = reinterpret_cast<const uint2*>(hist)[lane];   // lane owns bins 2 lane, 2 lane + 1
                const uint32_t own = h.x + h.y;
                const uint32_t before = warp_inclusive_sum(own) - own;
                uint32_t my_tau = 0xFFFFFFFFu, my_take = 0;
                if (before <= drop && drop < before + h.x) {
                    my_tau = low + 2u * lane;
                    my_take = h.x - (drop - before);
                } else if (before + h.x <= drop && drop < before + own) {
                    my_tau = low + 2u * lane + 1u;
                    my_take = h.y - (drop - before - h.x);
                }
                const uint32_t who = __ballot_sync(0xFFFFFFFFu, my_tau != 0xFFFFFFFFu);
                if (who) {
                    const int src = __ffs(who) - 1;
                    tau_key = __shfl_sync(0xFFFFFFFFu, my_tau, src);
                    take = __shfl_sync(0xFFFFFFFFu, my_take, src);
                    found = true;
                }
                __syncwarp();
            }
            if (!found) {
                // general case: radix select over the candidates, exponent byte then mantissa
                uint32_t k_rem = k;
                reinterpret_cast<uint4*>(hist)[lane] = make_uint4(0, 0, 0, 0);
                reinterpret_cast<uint4*>(hist)[lane + 32] = make_uint4(0, 0, 0, 0);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i)
                    if (static_cast<uint32_t>(i) < nvalid) atomicAdd(&hist[(ent[i] & 0x7FFFu) >> 7], 1u);
                __syncwarp();
                const uint32_t exp_bin = pick_exponent(hist, row_max >> 7, k_rem);
                __syncwarp();
                reinterpret_cast<uint4*>(hist)[lane] = make_uint4(0, 0, 0, 0);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t key = ent[i] & 0x7FFFu;
                    if (static_cast<uint32_t>(i) < nvalid && (key >> 7) == exp_bin) atomicAdd(&hist[key & 0x7Fu], 1u);
                }
                __syncwarp();
                tau_key = (exp_bin << 7) | pick_mantissa(hist, k_rem, take);
            }
            if (lane == 0 && tau_out) tau_out[row] = static_cast<uint16_t>(tau_key);
            guess_low = tau_key > kGuessMargin ? tau_key - kGuessMargin : 0u;
            if (lane == 0) *reinterpret_cast<volatile uint32_t*>(&s_hint) = guess_low;

            // ---- D: ordered emit ------------------------------------------------------------------------
            // The kept entries are placed, in column order, into k staging slots; then they leave with
            // coalesced stores.
            __syncwarp();                                         // the select histogram is dead: its words become the stage
            {
                uint32_t counts = 0;                              // (gt << 16) | eq of this lane's entries
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t key = ent[i] & 0x7FFFu;
                    counts += key > tau_key ? 0x10000u : (key == tau_key ? 1u : 0u);
                }
                const uint32_t before = warp_inclusive_sum(counts) - counts;
                uint32_t e_at = before & 0xFFFFu;                 // ties before this entry
                uint32_t pos = (before >> 16) + (e_at < take ? e_at : take);   // kept entries before it
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t key = ent[i] & 0x7FFFu;
                    const bool is_eq = key == tau_key;
                    const bool keep = key > tau_key || (is_eq && e_at < take);
                    if (keep) stage[pos] = ent[i];
                    pos += keep ? 1u : 0u;
                    e_at += is_eq ? 1u : 0u;
                }
            }
            __syncwarp();
            {
                // the first 256 slots with constant offsets from one pointer each, any further ones in a loop
                int16_t* cp = cols_out + out_base + lane;
                uint16_t* vp = vals_out + out_base + lane;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (lane + 32u * j < k) {
                        const uint32_t e = stage[lane + 32 * j];
                        cp[32 * j] = static_cast<int16_t>(e >> 16);
                        vp[32 * j] = static_cast<uint16_t>(e & 0xFFFFu);
                    }
                }
                for (uint32_t p = lane + 256u; p < k; p += 32) {
                    const uint32_t e = stage[p];
                    cp[p - lane] = static_cast<int16_t>(e >> 16);
                    vp[p - lane] = static_cast<uint16_t>(e & 0xFFFFu);
                }
                if (rows_out)
                    for (uint32_t p = lane; p < k; p += 32) rows_out[out_base + p] = static_cast<int32_t>(row);
            }
            __syncwarp();
        };
        // (Wide rows: the copies for fewer slots are only used when the launch says that nearly every row fits the
        // smallest one -- rows that alternate between two copies of this much code run 15 to 20 % slower.)
        if (E8 <= 12 || few_slots) {
            if (per_lane <= FwdTrips<PL>::kFew)
                finish_row(std::integral_constant<uint32_t, FwdTrips<PL>::kFew>{});
            else if (per_lane <= FwdTrips<PL>::kSome)
                finish_row(std::integral_constant<uint32_t, FwdTrips<PL>::kSome>{});
            else
                finish_row(std::integral_constant<uint32_t, PL>{});
        } else {
            finish_row(std::integral_constant<uint32_t, PL>{});
        }
    }
    // This warp has no row left: the next kernel on the stream may be scheduled as the CTAs of this one retire
    // (its set-up then overlaps the tail of this kernel; it still waits for this kernel's end before it works).
    chain_release_next();
}

template <int E8, int PL>
dct_status_t launch_fwd_bf16_warp_variant(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                          int16_t* cols_out,
                                          void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result,
                                          cudaStream_t stream) {
    using Lay = WarpRowLayout<E8>;
    auto kernel = mp_topk_fwd_bf16_warp_kernel<E8, PL>;
    constexpr int kMaxWarps = fwd_bf16_max_warps<E8, PL>();
    constexpr size_t kSmemBudget = 220 * 1024;            // of the 227 KiB a CTA may use
    static thread_local int configured_device = -1;
    int dev = 0;
    DCT_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        DCT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(kSmemBudget)));   // sized per launch below
        configured_device = dev;
    }
    const size_t per_warp = Lay::warp_bytes(k);
    size_t warps = kSmemBudget / per_warp;                 // one CTA per SM with as many row slots as fit
    if (warps > static_cast<size_t>(kMaxWarps)) warps = kMaxWarps;
    if (warps < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    warps = warps_for_rows(warps, rows, sms);
    const uint64_t ctas_needed = (static_cast<uint64_t>(rows) + warps - 1) / warps;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < static_cast<uint64_t>(sms) ? ctas_needed : sms);
    // a guessed bound leaves about 1.25 k candidates: do (nearly) all rows fit the smallest slot count?
    const bool few_slots = (static_cast<uint64_t>(k) * 13u / 10u + 31u) / 32u <= FwdTrips<PL>::kFew;
    DCT_CUDA_TRY(launch_chained_smem(kernel, grid, static_cast<unsigned>(warps * 32), warps * per_warp, stream,
                                     static_cast<const uint16_t*>(x_act), rows, d, ld, k, cols_out,
                                     static_cast<uint16_t*>(vals_out), rows_out, static_cast<uint16_t*>(tau_out), result,
                                     few_slots));
    return DCT_OK;
}

// 5, 10 or 20 candidates per lane: see fwd_candidates_per_lane.
template <int E8>
dct_status_t launch_fwd_bf16_warp(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                                  void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result,
                                  cudaStream_t stream) {
    const int per_lane = fwd_candidates_per_lane(d, k);
    if constexpr (E8 <= 4) {
        if (per_lane == 5)
            return launch_fwd_bf16_warp_variant<E8, 5>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out,
                                                       result, stream);
    }
    if (per_lane == 10)
        return launch_fwd_bf16_warp_variant<E8, 10>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result,
                                                    stream);
    return launch_fwd_bf16_warp_variant<E8, 20>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result,
                                                stream);
}

int fwd_threads_for(uint32_t d) {
    if (d <= 4096) return 128;
    if (d <= 8192) return 256;
    if (d <= 16384) return 512;
    return 1024;
}

template <typename T>
dct_status_t launch_fwd(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                        void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result,
                        cudaStream_t stream) {
    const size_t smem = ((static_cast<size_t>(d) * sizeof(T)) + 15) & ~static_cast<size_t>(15);
    auto kernel = mp_topk_pack_fwd_kernel<T>;
    // (static shared memory counts against the 48 KiB a kernel gets without asking: ask well below that)
    if (smem > 32 * 1024) DCT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                           static_cast<int>(smem)));
    const int threads = fwd_threads_for(d);
    int per_sm = 0;
    DCT_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem));
    if (per_sm < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t max_grid = static_cast<uint64_t>(sms) * per_sm;
    const uint32_t grid = static_cast<uint32_t>(rows < max_grid ? rows : max_grid);
    const bool rows_aligned16 = aligned_to(x_act, 16) && ((static_cast<size_t>(ld) * sizeof(T)) % 16 == 0);
    kernel<<<grid, threads, smem, stream>>>(static_cast<const T*>(x_act), rows, d, ld, k, cols_out,
                                            static_cast<T*>(vals_out), rows_out, static_cast<T*>(tau_out), result,
                                            rows_aligned16);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

template <typename T>
dct_status_t launch_bwd(const void* x_grad, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, const int16_t* cols,
                        void* gvals_out, dct_result_t* result, cudaStream_t stream) {
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    // A thread per entry: fewer kept columns than lanes, and the widest rows, where it is as fast or faster at every k
    // (3072 rows of 32768 bf16 columns, k = 8192: 0.129 -> 0.073 ms; fp32: 0.127 -> 0.043 ms); on rows of up to 4096 bf16
    // columns the warp per row is 10 to 15 % faster at the denser k and equal otherwise.
    if (k <= 24 || d >= 8192 || (sizeof(T) == 4 && d >= 4096)) {
        const uint64_t total = static_cast<uint64_t>(rows) * k;
        const uint64_t need = (total + 1023) / 1024;
        const uint64_t cap = static_cast<uint64_t>(sms) * 16;
        mp_pack_bwd_flat_kernel<T><<<static_cast<unsigned>(need < cap ? need : cap), 256, 0, stream>>>(
            static_cast<const T*>(x_grad), rows, d, ld, k, cols, static_cast<T*>(gvals_out), result, next_launch_ticket());
        DCT_CUDA_TRY(cudaGetLastError());
        return DCT_OK;
    }
    const uint64_t ctas_needed = (static_cast<uint64_t>(rows) + 7) / 8;
    // one row per warp up to 256 rows per SM: CTAs then start as others finish, which evens out the last round
    // (a grid of 8 resident CTAs per SM with a stride loop gives a warp 1 or 2 rows: 4 % slower at 16384 rows)
    const uint64_t max_grid = static_cast<uint64_t>(sms) * 32;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < max_grid ? ctas_needed : max_grid);
    mp_pack_bwd_kernel<T><<<grid, 256, 0, stream>>>(static_cast<const T*>(x_grad), rows, d, ld, k, cols,
                                                    static_cast<T*>(gvals_out), result, next_launch_ticket());
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

dct_status_t check_mp_args(const void* x, dct_dtype_t dtype, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                           const void* cols, const void* vals, const dct_result_t* result) {
    if (!x || !cols || !vals || rows == 0 || d == 0 || k == 0 || k > d || ld < d) return DCT_ERR_INVALID_ARG;
    if (d > 32768u) return DCT_ERR_INVALID_ARG;
    if (dtype != DCT_F32 && dtype != DCT_BF16) return DCT_ERR_UNSUPPORTED;
    const size_t es = dtype == DCT_F32 ? 4 : 2;
    if (!aligned_to(x, es) || !aligned_to(vals, es) || !aligned_to(cols, 2) || (result && !aligned_to(result, 8)))
        return DCT_ERR_INVALID_ARG;
    return DCT_OK;
}

}  // namespace
}  // namespace dct

using namespace dct;

extern "C" dct_status_t dct_mp_topk_pack_fwd(const void* x_act, dct_dtype_t dtype, uint32_t rows, uint32_t d,
                                             uint32_t ld, uint32_t k, int16_t* cols_out, void* vals_out,
                                             int32_t* rows_out, void* tau_out, dct_result_t* result,
                                             dct_stream_t stream_) {
    const dct_status_t st = check_mp_args(x_act, dtype, rows, d, ld, k, cols_out, vals_out, result);
    if (st != DCT_OK) return st;
    const size_t es = dtype == DCT_F32 ? 4 : 2;
    if ((rows_out && !aligned_to(rows_out, 4)) || (tau_out && !aligned_to(tau_out, es))) return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (dtype == DCT_F32) {
        bool handled = false;
        // narrow rows (256 columns, small k): the row stays in registers, four rows per warp
        const dct_status_t narrow = launch_fwd_f32_narrow(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out,
                                                          result, stream, &handled);
        if (narrow != DCT_OK || handled) return narrow;
        // the warp-per-row fp32 kernel takes the same shapes as the bf16 one below
        const dct_status_t fast = launch_fwd_f32_warp(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out,
                                                      result, stream, &handled);
        if (fast != DCT_OK || handled) return fast;
        // rows of more than 2048 columns that the warp-per-row kernels leave out: one CTA per row
        const dct_status_t wide = launch_fwd_f32_wide(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out,
                                                      result, stream, &handled);
        if (wide != DCT_OK || handled) return wide;
        return launch_fwd<float>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    }
    {   // narrow rows (256 or 512 columns, small k): the row stays in registers, several rows per warp
        bool handled = false;
        const dct_status_t narrow = launch_fwd_bf16_narrow(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out,
                                                           result, stream, &handled);
        if (narrow != DCT_OK || handled) return narrow;
    }
    // The sparse warp-per-row kernel holds up to 320 or 640 candidates in registers and needs a tight leaf bound.
    if (aligned_to(x_act, 16) && (static_cast<size_t>(ld) * 2) % 16 == 0 && d % 8 == 0 && d <= 8192 &&
        fwd_candidates_per_lane(d, k) != 0) {
        // warp-per-row path: the smallest instantiated buffer of 256 * E8 columns that holds the row
#define DCT_BF16_WIDTH(E8) \
    if (d <= 256u * E8)    \
        return launch_fwd_bf16_warp<E8>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream)
        DCT_BF16_WIDTH(1);
        DCT_BF16_WIDTH(2);
        DCT_BF16_WIDTH(3);
        DCT_BF16_WIDTH(4);
        DCT_BF16_WIDTH(5);
        DCT_BF16_WIDTH(6);
        DCT_BF16_WIDTH(7);
        DCT_BF16_WIDTH(8);
        DCT_BF16_WIDTH(10);
        DCT_BF16_WIDTH(12);
        DCT_BF16_WIDTH(14);
        DCT_BF16_WIDTH(16);
        DCT_BF16_WIDTH(24);
        DCT_BF16_WIDTH(32);
#undef DCT_BF16_WIDTH
    }
    // denser k (beyond the candidate registers of the kernels above, up to 3/8 of the row): every lane looks after
    // one contiguous span of the row (mp_pack_span.cu)
    {
        bool handled = false;
        const dct_status_t span = launch_fwd_bf16_span(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out,
                                                       result, stream, &handled);
        if (span != DCT_OK || handled) return span;
    }
    return launch_fwd<uint16_t>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
}

extern "C" dct_status_t dct_mp_pack_bwd(const void* x_grad, dct_dtype_t dtype, uint32_t rows, uint32_t d, uint32_t ld,
                                        uint32_t k, const int16_t* cols, void* gvals_out, dct_result_t* result,
                                        dct_stream_t stream_) {
    const dct_status_t st = check_mp_args(x_grad, dtype, rows, d, ld, k, cols, gvals_out, result);
    if (st != DCT_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (dtype == DCT_F32) return launch_bwd<float>(x_grad, rows, d, ld, k, cols, gvals_out, result, stream);
    return launch_bwd<uint16_t>(x_grad, rows, d, ld, k, cols, gvals_out, result, stream);
}
