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
                  const ShardState* __restrict__ st, unsigned long long* __restrict__ hist, bool vectorised,
                  const uint32_t* __restrict__ skip_if = nullptr) {
    constexpr int shift = shard_shift(kPass), bits = shard_bits(kPass);
    constexpr uint32_t digit_mask = (1u << bits) - 1u;
    if (skip_if && *skip_if) return;                   // (the sampled variant: the candidates are used instead)
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


// ---- the sampled variant: one streaming pass over the shard instead of three ---------------------------------------
// As in the single-GPU select (threshold_select.cu): a sample of the vector (groups of 8 neighbours, the same stride
// on every rank, so every element is sampled at the same rate) is radix-selected for a rank chosen six standard
// deviations on the safe side -- its histograms add over the ranks like any other -- which gives a key `lo` with,
// almost surely, between k and a few k elements of the whole vector at or above it; every rank then streams its shard
// once and keeps its keys >= lo; the candidate counts are summed over the ranks; and the three exact passes run over
// the candidates only.  If the candidates are fewer than k, or do not fit some rank's buffer, the three passes run
// over the shards instead: every rank takes that decision from the same summed counts.
constexpr uint32_t kShardSampleTarget = 1u << 20;       // sampled elements of the whole vector, about
constexpr uint32_t kShardGroup = 8;
constexpr uint64_t kShardMinSampledN = 1ull << 25;
constexpr uint32_t kShardMaxCandidates = 1u << 22;
constexpr int kShardStages = 6;                         // 2 sample passes, the filter, 3 exact passes

struct SampledState {
    ShardState main;             // offset 0: the exact select (k_global)
    ShardState sample;           // the select over the sample
    uint32_t stride;             // elements between two sample groups
    uint32_t lo_key;             // written after the second sample pass
    uint32_t cand_count;         // this rank's keys >= lo (may exceed the capacity)
    uint32_t cand_capacity;
    uint32_t use_candidates;     // decided from the summed counts, alike on every rank
    uint32_t pad[3];
};
constexpr size_t kSampledHeaderBytes = 256;
static_assert(sizeof(SampledState) <= kSampledHeaderBytes, "header too small");

__global__ void sampled_begin_kernel(SampledState* st, uint64_t k, uint64_t sample_k, uint32_t stride, uint32_t capacity) {
    st->main.k_rem = k;
    st->main.n_gt = 0;
    st->main.prefix = 0;
    st->main.passes_done = 0;
    st->sample.k_rem = sample_k;
    st->sample.n_gt = 0;
    st->sample.prefix = 0;
    st->sample.passes_done = 0;
    st->stride = stride;
    st->lo_key = 0;
    st->cand_count = 0;
    st->cand_capacity = capacity;
    st->use_candidates = 0;
}

// digit histogram of this rank's part of the sample: element (i / 8) * stride + i % 8 for every whole group
template <int kPass>
__global__ void __launch_bounds__(kShardThreads)
sampled_hist_kernel(const float* __restrict__ grad, const float* __restrict__ residual, uint32_t n,
                    const SampledState* __restrict__ sst, unsigned long long* __restrict__ hist) {
    const ShardState* st = &sst->sample;
    const uint32_t stride = sst->stride;
    constexpr int shift = shard_shift(kPass), bits = shard_bits(kPass);
    constexpr uint32_t digit_mask = (1u << bits) - 1u;
    __shared__ uint32_t sh[kShardBins];
    for (int b = threadIdx.x; b < kShardBins; b += kShardThreads) sh[b] = 0;
    const uint32_t prefix = kPass == 0 ? 0u : st->prefix;
    __syncthreads();
    const uint32_t groups = n >= kShardGroup ? (n - kShardGroup) / stride + 1u : 0u;
    const uint32_t total = groups * kShardGroup;
    for (uint32_t i = blockIdx.x * kShardThreads + threadIdx.x; i < total; i += gridDim.x * kShardThreads) {
        const size_t j = static_cast<size_t>(i / kShardGroup) * stride + (i % kShardGroup);
        const uint32_t key = key_f32(residual ? __fadd_rn(grad[j], residual[j]) : grad[j]);
        if (kPass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&sh[(key >> shift) & digit_mask], 1u);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kShardBins; b += kShardThreads) {
        const uint32_t c = sh[b];
        if (c) atomicAdd(&hist[b], static_cast<unsigned long long>(c));
    }
}

__global__ void sampled_lo_kernel(SampledState* st) {     // after the second sample pass: 21 key bits are known
    st->lo_key = st->sample.prefix << shard_shift(1);
}

// the one streaming pass: every key >= lo of the shard goes to this rank's candidate buffer
__global__ void __launch_bounds__(kShardThreads)
sampled_filter_kernel(const float* __restrict__ grad, const float* __restrict__ residual, uint32_t n, SampledState* st,
                      uint32_t* __restrict__ cand_keys, bool vectorised) {
    const uint32_t lo = st->lo_key, capacity = st->cand_capacity;
    const bool add = residual != nullptr;
    // Each warp collects its survivors in a small shared-memory buffer and moves them to the candidate buffer 64 or
    // more at a time, so the global counter sees one atomic per flush, not one per survivor.
    constexpr uint32_t kWarpBuf = 96, kFlushAt = 64;
    __shared__ uint32_t s_buf[kShardThreads / 32][kWarpBuf];
    uint32_t* wbuf = s_buf[threadIdx.x >> 5];
    uint32_t held = 0;                                  // warp-uniform
    auto flush = [&]() {
        __syncwarp();
        uint32_t base = 0;
        if (lane_id() == 0) base = atomicAdd(&st->cand_count, held);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        for (uint32_t i = lane_id(); i < held; i += 32)
            if (base + i < capacity) cand_keys[base + i] = wbuf[i];
        __syncwarp();
        held = 0;
    };
    auto keep = [&](bool pred, uint32_t key) {          // called by whole warps
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, pred);
        if (bal == 0) return;
        if (pred) wbuf[held + __popc(bal & lanemask_lt())] = key;
        held += __popc(bal);
        if (held >= kFlushAt) flush();
    };
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
                const uint32_t k0 = key_f32(add ? __fadd_rn(g4[j].x, e4[j].x) : g4[j].x);
                const uint32_t k1 = key_f32(add ? __fadd_rn(g4[j].y, e4[j].y) : g4[j].y);
                const uint32_t k2 = key_f32(add ? __fadd_rn(g4[j].z, e4[j].z) : g4[j].z);
                const uint32_t k3 = key_f32(add ? __fadd_rn(g4[j].w, e4[j].w) : g4[j].w);
                if (__any_sync(0xFFFFFFFFu, max(max(k0, k1), max(k2, k3)) >= lo)) {
                    keep(k0 >= lo, k0);
                    keep(k1 >= lo, k1);
                    keep(k2 >= lo, k2);
                    keep(k3 >= lo, k3);
                }
            }
        } else {
            // whole warps stay together so that the ballots above see every lane
            for (uint32_t i0 = base + (threadIdx.x & ~31u); i0 < n && i0 < base + kShardChunk; i0 += kShardThreads) {
                const uint32_t i = i0 + lane_id();
                const bool in = i < n && i < base + kShardChunk;
                const uint32_t key = in ? key_f32(add ? __fadd_rn(grad[i], residual[i]) : grad[i]) : 0u;
                keep(in && key >= lo, key);
            }
        }
    }
    if (held) flush();
}

// what the filter found, as the first two of the 2048 counts the ranks sum: candidates, and 1 if they did not fit
__global__ void sampled_counts_kernel(const SampledState* st, unsigned long long* hist) {
    hist[0] = st->cand_count;
    hist[1] = st->cand_count > st->cand_capacity ? 1ull : 0ull;
}
// the decision every rank takes alike from the summed counts
__global__ void sampled_decide_kernel(SampledState* st, const unsigned long long* hist_global) {
    const unsigned long long k = st->main.k_rem;        // (no exact pass has run yet: still k_global)
    st->use_candidates = (hist_global[1] == 0 && hist_global[0] >= k) ? 1u : 0u;
}

// digit histogram of this rank's candidates (if they are used)
template <int kPass>
__global__ void __launch_bounds__(kShardThreads)
sampled_cand_hist_kernel(const uint32_t* __restrict__ keys, const SampledState* __restrict__ st,
                         unsigned long long* __restrict__ hist) {
    constexpr int shift = shard_shift(kPass), bits = shard_bits(kPass);
    constexpr uint32_t digit_mask = (1u << bits) - 1u;
    if (!st->use_candidates) return;
    __shared__ uint32_t sh[kShardBins];
    for (int b = threadIdx.x; b < kShardBins; b += kShardThreads) sh[b] = 0;
    const uint32_t prefix = kPass == 0 ? 0u : st->main.prefix;
    const uint32_t n = st->cand_count;
    __syncthreads();
    for (uint32_t i = blockIdx.x * kShardThreads + threadIdx.x; i < n; i += gridDim.x * kShardThreads) {
        const uint32_t key = keys[i];
        if (kPass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&sh[(key >> shift) & digit_mask], 1u);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kShardBins; b += kShardThreads) {
        const uint32_t c = sh[b];
        if (c) atomicAdd(&hist[b], static_cast<unsigned long long>(c));
    }
}

// Rank to select in the sample (rate = sampled fraction of the vector) so that the number of vector elements at or
// above the sampled value is, six standard deviations out, still at least k; 0 if the candidates could overflow one
// rank's buffer even if all of them lay on that rank.
uint64_t shard_sample_rank(uint64_t n, uint64_t k, double rate) {
    const double m = static_cast<double>(k) * rate;
    const double r = m + 6.0 * __builtin_sqrt(m + 1.0) + 20.0;
    const double expected_max = (r + 6.0 * __builtin_sqrt(r)) / rate;
    if (r >= static_cast<double>(n) * rate / 4.0 || expected_max > kShardMaxCandidates) return 0;
    return static_cast<uint64_t>(r);
}
uint32_t shard_stride(uint64_t n_global) {
    return static_cast<uint32_t>(n_global / (kShardSampleTarget / kShardGroup)) & ~(kShardGroup - 1u);
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

// ---- sampled variant: six stages of (local pass, sum of 2048 counts over the ranks, advance) -----------------------
extern "C" size_t dct_threshold_select_shard_sampled_workspace_bytes(uint64_t n_local) {
    if (n_local > 0x7FFFFFFFull) return 0;
    const uint64_t cap = n_local < kShardMaxCandidates ? n_local : kShardMaxCandidates;
    return (kSampledHeaderBytes + sizeof(uint32_t) * static_cast<size_t>(cap) + 255) & ~static_cast<size_t>(255);
}

extern "C" dct_status_t dct_threshold_select_shard_sampled_begin(uint64_t k_global, uint64_t n_global, uint64_t n_local,
                                                                 void* workspace, size_t workspace_bytes,
                                                                 dct_stream_t stream_) {
    if (k_global == 0 || k_global > n_global || n_local > n_global || n_local > 0x7FFFFFFFull) return DCT_ERR_INVALID_ARG;
    if (!workspace || !aligned_to(workspace, 256) ||
        workspace_bytes < dct_threshold_select_shard_sampled_workspace_bytes(n_local))
        return DCT_ERR_WORKSPACE;
    if (n_global < kShardMinSampledN) return DCT_ERR_UNSUPPORTED;       // the three-pass version is cheaper
    const uint32_t stride = shard_stride(n_global);
    if (stride < kShardGroup) return DCT_ERR_UNSUPPORTED;
    const uint64_t sample_k = shard_sample_rank(n_global, k_global, static_cast<double>(kShardGroup) / stride);
    if (sample_k == 0) return DCT_ERR_UNSUPPORTED;                      // too dense for the candidate buffers
    const uint32_t cap = static_cast<uint32_t>(n_local < kShardMaxCandidates ? n_local : kShardMaxCandidates);
    sampled_begin_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream_)>>>(static_cast<SampledState*>(workspace),
                                                                          k_global, sample_k, stride, cap);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

extern "C" dct_status_t dct_threshold_select_shard_sampled_pass(const float* grad, const float* residual,
                                                                uint64_t n_local, uint32_t stage, void* workspace,
                                                                uint64_t* hist_out, dct_stream_t stream_) {
    if (!hist_out || !workspace || stage >= static_cast<uint32_t>(kShardStages) || n_local > 0x7FFFFFFFull)
        return DCT_ERR_INVALID_ARG;
    if (n_local > 0 && !grad) return DCT_ERR_INVALID_ARG;
    if (!aligned_to(grad, 4) || (residual && !aligned_to(residual, 4)) || !aligned_to(hist_out, 8) ||
        !aligned_to(workspace, 256))
        return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    auto* hist = reinterpret_cast<unsigned long long*>(hist_out);
    auto* st = static_cast<SampledState*>(workspace);
    auto* cand_keys = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + kSampledHeaderBytes);
    shard_clear_kernel<<<1, 512, 0, stream>>>(hist);
    DCT_CUDA_TRY(cudaGetLastError());
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint32_t n32 = static_cast<uint32_t>(n_local);
    const uint64_t chunks = (n_local + kShardChunk - 1) / kShardChunk;
    const int grid = static_cast<int>(chunks < static_cast<uint64_t>(sms) * 4 ? (chunks ? chunks : 1) : sms * 4);
    const bool vec = aligned_to(grad, 16) && (!residual || aligned_to(residual, 16));
    if (stage < 2) {                                    // the sample: stride and prefix come from the state
        if (n_local == 0) return DCT_OK;
        // (the stride is in the state; the grid only has to cover the sample)
        const int sgrid = sms * 2;
        if (stage == 0)
            sampled_hist_kernel<0><<<sgrid, kShardThreads, 0, stream>>>(grad, residual, n32, st, hist);
        else
            sampled_hist_kernel<1><<<sgrid, kShardThreads, 0, stream>>>(grad, residual, n32, st, hist);
        DCT_CUDA_TRY(cudaGetLastError());
        return DCT_OK;
    }
    if (stage == 2) {                                   // the filter, then its counts as the ranks' message
        if (n_local > 0) {
            sampled_filter_kernel<<<grid, kShardThreads, 0, stream>>>(grad, residual, n32, st, cand_keys, vec);
            DCT_CUDA_TRY(cudaGetLastError());
        }
        sampled_counts_kernel<<<1, 1, 0, stream>>>(st, hist);
        DCT_CUDA_TRY(cudaGetLastError());
        return DCT_OK;
    }
    // stages 3..5: the exact passes over the candidates or, if the summed counts said so, over the shard
    const uint32_t pass = stage - 3;
    if (pass == 0)
        sampled_cand_hist_kernel<0><<<sms, kShardThreads, 0, stream>>>(cand_keys, st, hist);
    else if (pass == 1)
        sampled_cand_hist_kernel<1><<<sms, kShardThreads, 0, stream>>>(cand_keys, st, hist);
    else
        sampled_cand_hist_kernel<2><<<sms, kShardThreads, 0, stream>>>(cand_keys, st, hist);
    DCT_CUDA_TRY(cudaGetLastError());
    if (n_local == 0) return DCT_OK;
    if (pass == 0)
        shard_hist_kernel<0><<<grid, kShardThreads, 0, stream>>>(grad, residual, n32, &st->main, hist, vec, &st->use_candidates);
    else if (pass == 1)
        shard_hist_kernel<1><<<grid, kShardThreads, 0, stream>>>(grad, residual, n32, &st->main, hist, vec, &st->use_candidates);
    else
        shard_hist_kernel<2><<<grid, kShardThreads, 0, stream>>>(grad, residual, n32, &st->main, hist, vec, &st->use_candidates);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

extern "C" dct_status_t dct_threshold_select_shard_sampled_advance(const uint64_t* hist_global, uint32_t stage,
                                                                   void* workspace, float* tau_out, dct_result_t* result,
                                                                   dct_stream_t stream_) {
    if (!hist_global || !workspace || stage >= static_cast<uint32_t>(kShardStages)) return DCT_ERR_INVALID_ARG;
    if (stage == static_cast<uint32_t>(kShardStages) - 1 && (!tau_out || !result)) return DCT_ERR_INVALID_ARG;
    if (!aligned_to(hist_global, 8) || !aligned_to(workspace, 256) || (tau_out && !aligned_to(tau_out, 4)) ||
        (result && !aligned_to(result, 8)))
        return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const auto* hist = reinterpret_cast<const unsigned long long*>(hist_global);
    auto* st = static_cast<SampledState*>(workspace);
    if (stage == 0) {
        shard_advance_kernel<0><<<1, kShardThreads, 0, stream>>>(hist, &st->sample, nullptr, nullptr);
    } else if (stage == 1) {
        shard_advance_kernel<1><<<1, kShardThreads, 0, stream>>>(hist, &st->sample, nullptr, nullptr);
        DCT_CUDA_TRY(cudaGetLastError());
        sampled_lo_kernel<<<1, 1, 0, stream>>>(st);
    } else if (stage == 2) {
        sampled_decide_kernel<<<1, 1, 0, stream>>>(st, hist);
    } else if (stage == 3) {
        shard_advance_kernel<0><<<1, kShardThreads, 0, stream>>>(hist, &st->main, tau_out, result);
    } else if (stage == 4) {
        shard_advance_kernel<1><<<1, kShardThreads, 0, stream>>>(hist, &st->main, tau_out, result);
    } else {
        shard_advance_kernel<2><<<1, kShardThreads, 0, stream>>>(hist, &st->main, tau_out, result);
    }
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}
