// dct_mp_topk_pack_fwd / dct_mp_pack_bwd: Algorithm 2 (DCT-MP).
//
// Forward: one CTA per sample (row).  The row is read from HBM exactly once
// into shared memory; the row threshold tau_i (k-th largest magnitude) is found
// on chip by a most-significant-digit-first radix select over key(x) with 8-bit
// digits (4 passes for fp32's 31 key bits, 2 for bf16's 15); then the kept
// columns -- every key above tau_i plus the lowest-column ties -- are written
// in ascending column order together with their values.  The int16 column list
// is the mask M.
//
// Backward: a gather of X_grad through that column list, one warp per row.
#include "common.cuh"

namespace dct {
namespace {

template <typename T> struct ElemTraits;
template <> struct ElemTraits<float> {
    static constexpr int kPasses = 4;
    __device__ static __forceinline__ uint32_t key(float x) { return key_f32(x); }
    __device__ static __forceinline__ float from_key(uint32_t k) { return __uint_as_float(k); }
    __host__ __device__ static constexpr int shift(int p) { return p == 0 ? 23 : (p == 1 ? 15 : (p == 2 ? 7 : 0)); }
    __host__ __device__ static constexpr int bits(int p) { return p == 3 ? 7 : 8; }
};
template <> struct ElemTraits<uint16_t> {   // bf16 carried as its bit pattern
    static constexpr int kPasses = 2;
    __device__ static __forceinline__ uint32_t key(uint16_t x) { return key_bf16(x); }
    __device__ static __forceinline__ uint16_t from_key(uint32_t k) { return static_cast<uint16_t>(k); }
    __host__ __device__ static constexpr int shift(int p) { return p == 0 ? 7 : 0; }
    __host__ __device__ static constexpr int bits(int p) { return p == 0 ? 8 : 7; }
};

constexpr int kMaxWarps = 32;

template <typename T>
__global__ void mp_topk_pack_fwd_kernel(const T* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                        int16_t* __restrict__ cols_out, T* __restrict__ vals_out,
                                        int32_t* __restrict__ rows_out, T* __restrict__ tau_out,
                                        dct_result_t* __restrict__ result, bool rows_aligned16) {
    using Tr = ElemTraits<T>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* row_s = reinterpret_cast<T*>(smem_raw);
    __shared__ uint32_t s_hist[256];
    __shared__ uint32_t s_prefix, s_krem;
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
        if (tid == 0) {
            s_prefix = 0;
            s_krem = k;
        }

        // ---- radix select of the k-th largest key ------------------------------------------
#pragma unroll
        for (int p = 0; p < Tr::kPasses; ++p) {
            const int shift = Tr::shift(p), bits = Tr::bits(p);
            const uint32_t nbins = 1u << bits;
            for (uint32_t b = tid; b < 256; b += nt) s_hist[b] = 0;
            __syncthreads();
            const uint32_t prefix = s_prefix;
            for (uint32_t j = tid; j < d; j += nt) {
                const uint32_t key = Tr::key(row_s[j]);
                if (p == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&s_hist[(key >> shift) & (nbins - 1u)], 1u);
            }
            __syncthreads();
            if (warp == 0) {
                // lane owns 8 bins, top-down: bin(lane, q) = 255 - (8 lane + q); bins >= nbins are empty
                const uint32_t k_rem = s_krem;
                uint32_t c[8], own = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    c[q] = s_hist[255 - (8 * lane + q)];
                    own += c[q];
                }
                uint32_t incl = own;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= static_cast<uint32_t>(o)) incl += t;
                }
                uint32_t above = incl - own;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (above < k_rem && k_rem <= above + c[q]) {
                        s_prefix = (prefix << bits) | (255u - (8u * lane + q));
                        s_krem = k_rem - above;
                    }
                    above += c[q];
                }
            }
            __syncthreads();
        }
        const uint32_t tau_key = s_prefix;
        const uint32_t take = s_krem;          // ties (key == tau_key) to keep, lowest columns first
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

template <typename T>
__global__ void __launch_bounds__(256)
mp_pack_bwd_kernel(const T* __restrict__ gx, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                   const int16_t* __restrict__ cols, T* __restrict__ gvals, dct_result_t* __restrict__ result) {
    const uint32_t lane = lane_id();
    const uint32_t warps_per_cta = blockDim.x >> 5;
    bool bad = false;
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
                v[u] = (s < k && ok) ? __ldg(gr + c[u]) : T(0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t s = s0 + u * 32 + lane;
                if (s < k) out[s] = v[u];
            }
        }
    }
    if (bad && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_BAD_MASK));
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
    if (smem > 48 * 1024) DCT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
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
    if (result) DCT_CUDA_TRY(cudaMemsetAsync(result, 0, sizeof(dct_result_t), stream));
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t ctas_needed = (static_cast<uint64_t>(rows) + 7) / 8;
    const uint64_t max_grid = static_cast<uint64_t>(sms) * 8;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < max_grid ? ctas_needed : max_grid);
    mp_pack_bwd_kernel<T><<<grid, 256, 0, stream>>>(static_cast<const T*>(x_grad), rows, d, ld, k, cols,
                                                    static_cast<T*>(gvals_out), result);
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
    if (dtype == DCT_F32)
        return launch_fwd<float>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
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
