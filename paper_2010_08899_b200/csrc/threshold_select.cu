// dct_threshold_select: Algorithm 1 (DCT-DP), threshold steps.
//
// tau = k-th largest |grad + residual|, found exactly by a most-significant-
// digit-first radix select on key(w) (31 magnitude bits) instead of the
// copy-and-sort the paper describes: three passes over the data with digits of
// 11, 10 and 10 bits.  Each pass builds a histogram of the current digit over
// the elements whose higher bits equal the prefix chosen so far (per-CTA
// histogram in shared memory, merged into global memory); the last CTA to
// finish a pass scans the histogram from the top, picks the digit that holds
// rank k and extends the prefix.  Nothing is copied, nothing is sorted, and the
// input is never modified.
#include "common.cuh"

namespace dct {
namespace {

constexpr int kSelThreads = 512;
constexpr int kSelVecs = 4;
constexpr uint32_t kSelChunk = kSelThreads * kSelVecs * 4;   // 8192 elements per CTA iteration
constexpr int kBins = 2048;
constexpr int kPasses = 3;

__host__ __device__ constexpr int pass_shift(int p) { return p == 0 ? 20 : (p == 1 ? 10 : 0); }
__host__ __device__ constexpr int pass_bits(int p) { return p == 0 ? 11 : 10; }

struct SelectState {
    uint32_t prefix;      // digits chosen so far (right-aligned)
    uint32_t k_rem;       // rank still to be located inside the prefix bucket
    uint64_t n_gt;        // elements known to be above the bucket
    uint32_t done[kPasses];
};
constexpr size_t kSelStateBytes = 256;

__global__ void select_init_kernel(SelectState* st, uint32_t* hist, uint32_t k) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < kPasses * kBins) hist[i] = 0;
    if (i == 0) {
        st->prefix = 0;
        st->k_rem = k;
        st->n_gt = 0;
        for (int p = 0; p < kPasses; ++p) st->done[p] = 0;
    }
}

template <int kPass, bool kHasResidual, bool kVectorised>
__global__ void __launch_bounds__(kSelThreads)
select_pass_kernel(const float* __restrict__ grad, const float* __restrict__ residual, uint32_t n,
                   SelectState* st, uint32_t* __restrict__ hist_all, float* __restrict__ tau_out,
                   dct_result_t* __restrict__ result) {
    constexpr int shift = pass_shift(kPass);
    constexpr int bits = pass_bits(kPass);
    constexpr uint32_t digit_mask = (1u << bits) - 1u;
    __shared__ uint32_t sh[kBins];
    __shared__ uint32_t s_scan[kSelThreads / 32];
    __shared__ uint32_t s_last;

    for (int b = threadIdx.x; b < kBins; b += kSelThreads) sh[b] = 0;
    const uint32_t prefix = kPass == 0 ? 0u : st->prefix;   // written by the previous launch
    __syncthreads();

    auto consume = [&](float g, float e) {
        const float w = kHasResidual ? __fadd_rn(g, e) : g;
        const uint32_t key = key_f32(w);
        if (kPass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&sh[(key >> shift) & digit_mask], 1u);
    };

    const uint32_t num_chunks = (n + kSelChunk - 1) / kSelChunk;
    for (uint32_t chunk = blockIdx.x; chunk < num_chunks; chunk += gridDim.x) {
        const uint32_t base = chunk * kSelChunk;
        if (kVectorised && base + kSelChunk <= n) {
            float4 g4[kSelVecs], e4[kSelVecs];
#pragma unroll
            for (int j = 0; j < kSelVecs; ++j) {
                const uint32_t off = base + (j * kSelThreads + threadIdx.x) * 4;
                g4[j] = ld_readonly_f4(grad + off);
                if (kHasResidual) e4[j] = ld_readonly_f4(residual + off);
                else e4[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < kSelVecs; ++j) {
                consume(g4[j].x, e4[j].x);
                consume(g4[j].y, e4[j].y);
                consume(g4[j].z, e4[j].z);
                consume(g4[j].w, e4[j].w);
            }
        } else {
            for (uint32_t i = base + threadIdx.x; i < n && i < base + kSelChunk; i += kSelThreads)
                consume(grad[i], kHasResidual ? residual[i] : 0.0f);
        }
    }
    __syncthreads();

    uint32_t* hist = hist_all + kPass * kBins;
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) {
        const uint32_t c = sh[b];
        if (c) atomicAdd(&hist[b], c);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(&st->done[kPass], 1u) == gridDim.x - 1) ? 1u : 0u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // ---- last CTA: locate the digit that holds rank k_rem, counting from the top ----------
    // thread t owns bins top-down: bin(t, q) = kBins-1 - (4t + q), q = 0..3
    const uint32_t k_rem = st->k_rem;
    uint32_t c[4], own = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        c[q] = __ldcg(&hist[kBins - 1 - (4 * threadIdx.x + q)]);
        own += c[q];
    }
    // exclusive prefix (over threads, i.e. over higher bins) of `own`
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
    // `above` = elements in bins higher than this thread's first bin
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (above < k_rem && k_rem <= above + c[q]) {
            const uint32_t digit = kBins - 1 - (4 * threadIdx.x + q);
            const uint32_t new_prefix = (prefix << bits) | digit;
            st->prefix = new_prefix;
            st->k_rem = k_rem - above;
            const uint64_t n_gt = st->n_gt + above;
            st->n_gt = n_gt;
            if (kPass == kPasses - 1) {
                *tau_out = __uint_as_float(new_prefix);
                result->status = DCT_OK;
                result->reserved = 0;
                result->count = 0;
                result->needed = 0;
                result->n_gt = n_gt;
                result->n_eq = c[q];
            }
        }
        above += c[q];
    }
}

template <int kPass>
cudaError_t launch_pass(int grid, cudaStream_t stream, bool has_res, bool vec, const float* grad,
                        const float* residual, uint32_t n, SelectState* st, uint32_t* hist, float* tau_out,
                        dct_result_t* result) {
#define DCT_SEL_LAUNCH(R, V) \
    select_pass_kernel<kPass, R, V><<<grid, kSelThreads, 0, stream>>>(grad, residual, n, st, hist, tau_out, result)
    if (has_res) {
        if (vec) DCT_SEL_LAUNCH(true, true); else DCT_SEL_LAUNCH(true, false);
    } else {
        if (vec) DCT_SEL_LAUNCH(false, true); else DCT_SEL_LAUNCH(false, false);
    }
#undef DCT_SEL_LAUNCH
    return cudaGetLastError();
}

}  // namespace
}  // namespace dct

using namespace dct;

extern "C" size_t dct_threshold_select_workspace_bytes(uint64_t n) {
    if (n == 0 || n > 0x7FFFFFFFull) return 0;
    return kSelStateBytes + sizeof(uint32_t) * kPasses * kBins;
}

extern "C" dct_status_t dct_threshold_select(const float* grad, const float* residual, uint64_t n, uint64_t k,
                                             float* tau_out, dct_result_t* result, void* workspace,
                                             size_t workspace_bytes, dct_stream_t stream_) {
    if (!grad || !tau_out || !result || n == 0 || n > 0x7FFFFFFFull || k == 0 || k > n) return DCT_ERR_INVALID_ARG;
    if (!aligned_to(grad, 4) || (residual && !aligned_to(residual, 4)) || !aligned_to(tau_out, 4) ||
        !aligned_to(result, 8))
        return DCT_ERR_INVALID_ARG;
    if (!workspace || !aligned_to(workspace, 256) || workspace_bytes < dct_threshold_select_workspace_bytes(n))
        return DCT_ERR_WORKSPACE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    auto* st = static_cast<SelectState*>(workspace);
    auto* hist = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + kSelStateBytes);
    const uint32_t n32 = static_cast<uint32_t>(n);
    const uint32_t num_chunks = (n32 + kSelChunk - 1) / kSelChunk;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const int grid = static_cast<int>(num_chunks < static_cast<uint32_t>(sms * 4) ? num_chunks : sms * 4);
    const bool vec = aligned_to(grad, 16) && (!residual || aligned_to(residual, 16));

    select_init_kernel<<<(kPasses * kBins + 1023) / 1024, 1024, 0, stream>>>(st, hist, static_cast<uint32_t>(k));
    DCT_CUDA_TRY(cudaGetLastError());
    DCT_CUDA_TRY(launch_pass<0>(grid, stream, residual != nullptr, vec, grad, residual, n32, st, hist, tau_out, result));
    DCT_CUDA_TRY(launch_pass<1>(grid, stream, residual != nullptr, vec, grad, residual, n32, st, hist, tau_out, result));
    DCT_CUDA_TRY(launch_pass<2>(grid, stream, residual != nullptr, vec, grad, residual, n32, st, hist, tau_out, result));
    return DCT_OK;
}
