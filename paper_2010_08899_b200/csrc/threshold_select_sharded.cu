// dct_threshold_select_shard_*: the threshold steps of Algorithm 1 for ONE gradient vector that is range-partitioned
// over several GPUs (every rank holds a contiguous shard of g and of its error e).
//
// The radix select of threshold_select.cu needs, per pass, nothing but the digit histogram of the elements that
// match the prefix chosen so far -- and histograms add.  So every rank builds the histogram of its own shard
// (dct_threshold_select_shard_pass), the 2048 counts are summed over the ranks by the caller (one all-reduce of 16 KiB
// per pass, any transport: the library itself never talks to another GPU), and every rank scans the summed
// histogram (dct_threshold_select_shard_advance) and arrives at the same digit.  After the three passes (11 / 10 / 10
// bits) every rank holds the same tau, n_gt and n_eq: those of the whole vector.  Compression then needs no exchange
// at all: each rank compresses its shard with that tau (and, for an exact k, a tie budget handed out in rank order
// by the caller from the ranks' own tie counts).
#include "common.cuh"

namespace dct {
namespace {

constexpr int kShardThreads = 512;
constexpr int kShardVecs = 4;
constexpr uint32_t kShardChunk = kShardThreads * kShardVecs * 4;   // elements per CTA iteration
constexpr int kShardBins = 2048;
constexpr int kShardPasses = 3;

__host__ __device__ constexpr int shard_shift(int p) { return p == 0 ? 20 : (p == 1 ? 10 : 0); }
__host__ __device__ constexpr int shard_bits(int p) { return p == 0 ? 11 : 10; }

struct ShardState {           // the same on every rank after every advance
    uint64_t k_rem;           // rank still to be located inside the prefix bucket
    uint64_t n_gt;            // elements (of all shards) known to be above the bucket
    uint32_t prefix;          // digits chosen so far (right-aligned)
    uint32_t passes_done;
};

__global__ void shard_begin_kernel(ShardState* st, uint64_t k) {
    st->k_rem = k;
    st->n_gt = 0;
    st->prefix = 0;
    st->passes_done = 0;
}

__global__ void shard_clear_kernel(unsigned long long* hist) {
    for (int b = threadIdx.x; b < kShardBins; b += blockDim.x) hist[b] = 0;
}

// digit histogram of this rank's shard, restricted to the elements whose higher bits equal the prefix
template <int kPass>
__global__ void __launch_bounds__(kShardThreads)
shard_hist_kernel(const float* __restrict__ grad, const float* __restrict__ residual, uint32_t n,
                  const ShardState* __restrict__ st, unsigned long long* __restrict__ hist, bool vectorised) {
    constexpr int shift = shard_shift(kPass), bits = shard_bits(kPass);
    constexpr uint32_t digit_mask = (1u << bits) - 1u;
    __shared__ uint32_t sh[kShardBins];
    for (int b = threadIdx.x; b < kShardBins; b += kShardThreads) sh[b] = 0;
    const uint32_t prefix = kPass == 0 ? 0u : st->prefix;
    __syncthreads();
    auto consume = [&](uint32_t key) {
        if (kPass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&sh[(key >> shift) & digit_mask], 1u);
    };
    const bool add = residual != nullptr;
    const uint32_t num_chunks = (n + kShardChunk - 1) / kShardChunk;
    for (uint32_t chunk = blockIdx.x; chunk < num_chunks; chunk += gridDim.x) {
        const uint32_t base = chunk * kShardChunk;
        if (vectorised && base + kShardChunk <= n) {
            float4 g4[kShardVecs], e4[kShardVecs];
#pragma unroll
            for (int j = 0; j < kShardVecs; ++j) {
                const uint32_t off = base + (j * kShardThreads + threadIdx.x) * 4;
                g4[j] = ld_readonly_f4(grad + off);
                e4[j] = add ? ld_readonly_f4(residual + off) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < kShardVecs; ++j) {
                consume(key_f32(add ? __fadd_rn(g4[j].x, e4[j].x) : g4[j].x));
                consume(key_f32(add ? __fadd_rn(g4[j].y, e4[j].y) : g4[j].y));
                consume(key_f32(add ? __fadd_rn(g4[j].z, e4[j].z) : g4[j].z));
                consume(key_f32(add ? __fadd_rn(g4[j].w, e4[j].w) : g4[j].w));
            }
        } else {
            const uint32_t lim = n - base < kShardChunk ? n : base + kShardChunk;
            for (uint32_t i = base + threadIdx.x; i < lim; i += kShardThreads)
                consume(key_f32(add ? __fadd_rn(grad[i], residual[i]) : grad[i]));
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kShardBins; b += kShardThreads) {
        const uint32_t c = sh[b];
        if (c) atomicAdd(&hist[b], static_cast<unsigned long long>(c));
    }
}

// one CTA: the digit of the summed histogram that holds rank k_rem, counted from the top
template <int kPass>
__global__ void __launch_bounds__(kShardThreads)
shard_advance_kernel(const unsigned long long* __restrict__ hist, ShardState* st, float* tau_out, dct_result_t* result) {
    constexpr int bits = shard_bits(kPass);
    __shared__ unsigned long long s_scan[kShardThreads / 32];
    // thread t owns bins top-down: bin(t, q) = 2047 - (4 t + q)
    const uint64_t k_rem = st->k_rem;
    const uint32_t prefix = kPass == 0 ? 0u : st->prefix;
    unsigned long long c[4], own = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        c[q] = hist[kShardBins - 1 - (4 * threadIdx.x + q)];
        own += c[q];
    }
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned long long incl = own;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= static_cast<uint32_t>(o)) incl += t;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    unsigned long long above = incl - own;
    for (uint32_t v = 0; v < warp; ++v) above += s_scan[v];
    __syncthreads();                       // every thread has read the state before one of them rewrites it
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (above < k_rem && k_rem <= above + c[q]) {
            const uint32_t digit = kShardBins - 1 - (4 * threadIdx.x + q);
            const uint32_t new_prefix = (prefix << bits) | digit;
            st->prefix = new_prefix;
            st->k_rem = k_rem - above;
            st->n_gt = st->n_gt + above;
            st->passes_done = kPass + 1;
            if (kPass == kShardPasses - 1) {
                *tau_out = __uint_as_float(new_prefix);
                result->status = DCT_OK;
                result->reserved = 0;
                result->count = 0;
                result->needed = 0;
                result->n_gt = st->n_gt;
                result->n_eq = c[q];
            }
        }
        above += c[q];
    }
}

}  // namespace
}  // namespace dct

using namespace dct;

extern "C" size_t dct_threshold_select_shard_workspace_bytes(void) { return 256; }

extern "C" dct_status_t dct_threshold_select_shard_begin(uint64_t k_global, void* workspace, size_t workspace_bytes,
                                                         dct_stream_t stream_) {
    if (k_global == 0) return DCT_ERR_INVALID_ARG;
    if (!workspace || !aligned_to(workspace, 256) || workspace_bytes < dct_threshold_select_shard_workspace_bytes())
        return DCT_ERR_WORKSPACE;
    shard_begin_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream_)>>>(static_cast<ShardState*>(workspace), k_global);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

extern "C" dct_status_t dct_threshold_select_shard_pass(const float* grad, const float* residual, uint64_t n_local,
                                                        uint32_t pass, const void* workspace, uint64_t* hist_out,
                                                        dct_stream_t stream_) {
    if (!hist_out || !workspace || pass >= static_cast<uint32_t>(kShardPasses) || n_local > 0x7FFFFFFFull)
        return DCT_ERR_INVALID_ARG;
    if (n_local > 0 && !grad) return DCT_ERR_INVALID_ARG;
    if (!aligned_to(grad, 4) || (residual && !aligned_to(residual, 4)) || !aligned_to(hist_out, 8) ||
        !aligned_to(workspace, 256))
        return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    auto* hist = reinterpret_cast<unsigned long long*>(hist_out);
    shard_clear_kernel<<<1, 512, 0, stream>>>(hist);
    DCT_CUDA_TRY(cudaGetLastError());
    if (n_local == 0) return DCT_OK;            // a rank without elements contributes an empty histogram
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t chunks = (n_local + kShardChunk - 1) / kShardChunk;
    const int grid = static_cast<int>(chunks < static_cast<uint64_t>(sms) * 4 ? chunks : sms * 4);
    const bool vec = aligned_to(grad, 16) && (!residual || aligned_to(residual, 16));
    const auto* st = static_cast<const ShardState*>(workspace);
    const uint32_t n32 = static_cast<uint32_t>(n_local);
    if (pass == 0)
        shard_hist_kernel<0><<<grid, kShardThreads, 0, stream>>>(grad, residual, n32, st, hist, vec);
    else if (pass == 1)
        shard_hist_kernel<1><<<grid, kShardThreads, 0, stream>>>(grad, residual, n32, st, hist, vec);
    else
        shard_hist_kernel<2><<<grid, kShardThreads, 0, stream>>>(grad, residual, n32, st, hist, vec);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

extern "C" dct_status_t dct_threshold_select_shard_advance(const uint64_t* hist_global, uint32_t pass, void* workspace,
                                                           float* tau_out, dct_result_t* result, dct_stream_t stream_) {
    if (!hist_global || !workspace || pass >= static_cast<uint32_t>(kShardPasses)) return DCT_ERR_INVALID_ARG;
    if (pass == static_cast<uint32_t>(kShardPasses) - 1 && (!tau_out || !result)) return DCT_ERR_INVALID_ARG;
    if (!aligned_to(hist_global, 8) || !aligned_to(workspace, 256) || (tau_out && !aligned_to(tau_out, 4)) ||
        (result && !aligned_to(result, 8)))
        return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const auto* hist = reinterpret_cast<const unsigned long long*>(hist_global);
    auto* st = static_cast<ShardState*>(workspace);
    if (pass == 0)
        shard_advance_kernel<0><<<1, kShardThreads, 0, stream>>>(hist, st, tau_out, result);
    else if (pass == 1)
        shard_advance_kernel<1><<<1, kShardThreads, 0, stream>>>(hist, st, tau_out, result);
    else
        shard_advance_kernel<2><<<1, kShardThreads, 0, stream>>>(hist, st, tau_out, result);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}
