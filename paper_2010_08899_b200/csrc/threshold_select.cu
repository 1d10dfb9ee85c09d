// dct_threshold_select: Algorithm 1 (DCT-DP), threshold steps.
//
// tau = k-th largest |grad + residual|, found exactly by a most-significant-digit-first radix
// select on key(w) (31 magnitude bits, digits of 11/10/10 bits) instead of the copy-and-sort the
// paper describes.  One radix pass streams its source once, builds the histogram of the current
// digit over the elements whose higher bits equal the prefix chosen so far (per-CTA histogram in
// shared memory, merged into global memory); the last CTA to finish the pass scans the histogram
// from the top, picks the digit that holds rank k and extends the prefix.  Nothing is copied,
// nothing is sorted, and the input is never modified.
//
// Three radix passes over the whole vector cost 12 B per element against a floor of 4 B.  When k is
// small against n (the method's regime) the vector is therefore read only ONCE:
//   1. a sample of 2^20 elements -- 2^17 evenly spaced groups of 8 consecutive elements, i.e. whole
//      32-byte sectors, so the sample costs 4 MiB of HBM traffic and then lives in L2 -- is
//      radix-selected for a rank chosen so that, with overwhelming probability, between k and a few k
//      elements of the whole vector lie at or above the sampled value `lo`;
//   2. one streaming pass over the vector appends every key >= key(lo) to a candidate buffer in the
//      workspace and counts them;
//   3. if the count c satisfies k <= c <= capacity, tau is the k-th largest candidate (radix select
//      over the small buffer) and n_gt, n_eq follow from the candidates, since every element >= tau
//      is one of them.  Otherwise -- the sample misjudged the vector -- the three full passes run.
// When k is too large for all elements >= lo to fit the candidate buffer (k of a few per cent of n and
// more), the sample also gives an upper bound `hi`, chosen the same way on the other side of tau: the
// streaming pass counts the keys above hi and keeps the keys in [lo, hi] -- a band around tau that holds
// a fraction of a per cent of the vector whatever k is -- and tau is the (k - count above hi)-th largest
// of those.
// Every decision is taken on the device; all kernels are enqueued up front and the ones that are
// not needed return at once.  The result is exact in every case.
#include "common.cuh"
#include "dp_chain.cuh"

namespace dct {
namespace {

constexpr int kSelThreads = 512;
constexpr int kSelVecs = 4;
constexpr uint32_t kSelChunk = kSelThreads * kSelVecs * 4;   // 8192 elements per CTA iteration
constexpr int kBins = 2048;
constexpr int kPasses = 3;
constexpr uint32_t kSampleSize = 1u << 20;                   // elements in the sample
constexpr uint32_t kSampleGroup = 8;                         // consecutive elements taken at each sample position
constexpr uint32_t kMaxCandidates = 1u << 23;                // candidate buffer: at most 32 MiB
constexpr uint32_t kMinSampledN = 1u << 25;                  // below this the three plain passes are cheaper
constexpr uint64_t kBandFromK = 1u << 21;                    // from this k on the filter keeps a band around tau, if it can

__host__ __device__ constexpr int pass_shift(int p) { return p == 0 ? 20 : (p == 1 ? 10 : 0); }
__host__ __device__ constexpr int pass_bits(int p) { return p == 0 ? 11 : 10; }

// One radix select in flight.
struct SelectState {
    uint32_t prefix;      // digits chosen so far (right-aligned)
    uint32_t k_rem;       // rank still to be located inside the prefix bucket
    uint64_t n_gt;        // elements known to be above the bucket
    uint32_t done[kPasses];
    uint32_t enabled;     // 0: every kernel of this select returns at once
    uint32_t n;           // elements of the source (written on the device for the candidate buffer)
    uint32_t key_out;     // the selected key (the sample select hands `lo` to the filter this way)
    uint32_t last_pass;   // the pass that ends this select: 2, or 1 for a select that only needs a lower bound of the
                          // rank-th key (its lower 10 bits are then zero)
    uint32_t hist[kPasses * kBins];
};

// Workspace layout: the select states (whole vector, sample for the lower bound, candidates, sample for the
// upper bound), the counters of the filter pass, the candidate keys.
struct SelectWorkspace {
    SelectState full, sample, cand, sample_hi;
    uint32_t cand_count;      // keys in [lo, hi] met by the filter pass (may exceed the capacity)
    uint32_t cand_capacity;
    uint32_t above_count;     // keys above hi met by the filter pass (0 without an upper bound)
    uint32_t filter_done;     // CTAs of the filter pass that have finished
    uint32_t k_total;         // the rank the call asks for
    uint32_t pad[59];
};

constexpr int kInitThreads = 1024;
__device__ __forceinline__ void reset_state(SelectState* st, uint32_t k, uint32_t n, uint32_t enabled, uint32_t i,
                                            uint32_t stride, uint32_t last_pass = kPasses - 1) {
    for (uint32_t b = i; b < kPasses * kBins; b += stride) st->hist[b] = 0;
    if (i == 0) {
        st->prefix = 0;
        st->k_rem = k;
        st->n_gt = 0;
        for (int p = 0; p < kPasses; ++p) st->done[p] = 0;
        st->enabled = enabled;
        st->n = n;
        st->key_out = 0;
        st->last_pass = last_pass;
    }
}

__global__ void select_init_kernel(SelectWorkspace* ws, uint32_t n, uint32_t k, uint32_t sample_n, uint32_t sample_k,
                                   uint32_t cand_capacity, dct_result_t* result, uint32_t sample_k_hi = 0) {
    chain_release_next();
    const uint32_t i = threadIdx.x;
    const bool sampled = sample_n != 0;
    reset_state(&ws->full, k, n, sampled ? 0u : 1u, i, kInitThreads);
    // the sample only has to give a lower bound of its rank-th key: two passes (21 of the 31 key bits) do
    reset_state(&ws->sample, sample_k, sample_n, sampled ? 1u : 0u, i, kInitThreads, 1u);
    reset_state(&ws->cand, k, 0u, 0u, i, kInitThreads);
    // the upper bound, where the call uses one: the select rounds down, the filter adds the bits it left out
    reset_state(&ws->sample_hi, sample_k_hi, sample_n, sampled && sample_k_hi ? 1u : 0u, i, kInitThreads, 1u);
    if (i == 0) {
        ws->cand_count = 0;
        ws->cand_capacity = cand_capacity;
        ws->above_count = 0;
        ws->filter_done = 0;
        ws->k_total = k;
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }
}

// Where a pass reads its keys from.
struct VectorSource {        // key(fl32(grad[i] + residual[i])), skip <= i < n
    const float* grad;
    const float* residual;   // may be null
    uint32_t skip = 0;       // leading elements that are not the vector's (a vector that starts 4, 8 or 12 bytes past a
                             // 16-byte boundary is read from that boundary, so that the 16-byte loads apply)
};
template <typename Source> __device__ __forceinline__ uint32_t skip_of(const Source&) { return 0u; }
__device__ __forceinline__ uint32_t skip_of(const VectorSource& s) { return s.skip; }
struct StridedSource {       // the same at (i / 8) * stride + i % 8: groups of 8 neighbours, `stride` elements apart
    const float* grad;
    const float* residual;
    uint32_t stride;
};
struct KeySource {           // keys stored in the workspace
    const uint32_t* keys;
};
struct ValueSource {         // key(values[i]): a list of packed values
    const float* values;
};

__device__ __forceinline__ uint32_t key_at(const VectorSource& s, uint32_t i) {
    return key_f32(s.residual ? __fadd_rn(s.grad[i], s.residual[i]) : s.grad[i]);
}
__device__ __forceinline__ uint32_t key_at(const StridedSource& s, uint32_t i) {
    const size_t j = static_cast<size_t>(i / kSampleGroup) * s.stride + (i % kSampleGroup);
    return key_f32(s.residual ? __fadd_rn(s.grad[j], s.residual[j]) : s.grad[j]);
}
__device__ __forceinline__ uint32_t key_at(const KeySource& s, uint32_t i) { return s.keys[i]; }
__device__ __forceinline__ uint32_t key_at(const ValueSource& s, uint32_t i) { return key_f32(s.values[i]); }

// Scan of one pass's histogram by the last CTA: the digit that holds rank k_rem, counted from the top.
template <int kPass>
__device__ __forceinline__ void finish_pass(SelectState* st, uint32_t prefix, uint32_t* s_scan, float* tau_out,
                                            dct_result_t* result) {
    constexpr int bits = pass_bits(kPass);
    const uint32_t* hist = st->hist + kPass * kBins;
    // thread t owns bins top-down: bin(t, q) = kBins-1 - (4t + q), q = 0..3
    const uint32_t k_rem = st->k_rem;
    uint32_t c[4], own = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        c[q] = __ldcg(&hist[kBins - 1 - (4 * threadIdx.x + q)]);
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
            const uint32_t digit = kBins - 1 - (4 * threadIdx.x + q);
            const uint32_t new_prefix = (prefix << bits) | digit;
            st->prefix = new_prefix;
            st->k_rem = k_rem - above;
            const uint64_t n_gt = st->n_gt + above;
            st->n_gt = n_gt;
            if (kPass == static_cast<int>(st->last_pass)) {
                const uint32_t key = new_prefix << pass_shift(kPass);      // (the bits no pass has looked at are zero)
                st->key_out = key;
                if (tau_out) {           // this select produces the call's answer
                    *tau_out = __uint_as_float(key);
                    result->n_gt = n_gt;
                    result->n_eq = c[q];
                }
            }
        }
        above += c[q];
    }
}

// One radix pass of one select by the whole grid.  sh (kBins words, cleared by the caller), s_scan and s_last are the
// CTA's shared memory; the caller has waited for the previous kernel of the chain.
template <int kPass, typename Source, bool kVectorised>
__device__ __forceinline__ void select_pass_body(const Source& src, SelectState* st, float* __restrict__ tau_out,
                                                 dct_result_t* __restrict__ result, uint32_t n, uint32_t* sh,
                                                 uint32_t* s_scan, uint32_t& s_last) {
    constexpr int shift = pass_shift(kPass);
    constexpr int bits = pass_bits(kPass);
    constexpr uint32_t digit_mask = (1u << bits) - 1u;
    const uint32_t prefix = kPass == 0 ? 0u : st->prefix;   // written by the previous launch
    __syncthreads();

    auto consume = [&](uint32_t key) {
        if (kPass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&sh[(key >> shift) & digit_mask], 1u);
    };

    const uint32_t num_chunks = (n + kSelChunk - 1) / kSelChunk;
    for (uint32_t chunk = blockIdx.x; chunk < num_chunks; chunk += gridDim.x) {
        const uint32_t base = chunk * kSelChunk;
        bool done = false;
        if constexpr (kVectorised) {      // VectorSource with 16-byte aligned pointers
            if (base + kSelChunk <= n && base >= skip_of(src)) {
                float4 g4[kSelVecs], e4[kSelVecs];
#pragma unroll
                for (int j = 0; j < kSelVecs; ++j) {
                    const uint32_t off = base + (j * kSelThreads + threadIdx.x) * 4;
                    g4[j] = ld_readonly_f4(src.grad + off);
                    e4[j] = src.residual ? ld_readonly_f4(src.residual + off) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                const bool add = src.residual != nullptr;
#pragma unroll
                for (int j = 0; j < kSelVecs; ++j) {
                    consume(key_f32(add ? __fadd_rn(g4[j].x, e4[j].x) : g4[j].x));
                    consume(key_f32(add ? __fadd_rn(g4[j].y, e4[j].y) : g4[j].y));
                    consume(key_f32(add ? __fadd_rn(g4[j].z, e4[j].z) : g4[j].z));
                    consume(key_f32(add ? __fadd_rn(g4[j].w, e4[j].w) : g4[j].w));
                }
                done = true;
            }
        }
        if (!done) {
            // scalar loads, eight per thread in flight before their histogram updates
            const uint32_t lim = n - base < kSelChunk ? n : base + kSelChunk;
            constexpr int kBatch = 8;
            for (uint32_t i0 = base + threadIdx.x; i0 < lim; i0 += kSelThreads * kBatch) {
                uint32_t key[kBatch];
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const uint32_t i = i0 + u * kSelThreads;
                    key[u] = i < lim ? key_at(src, i) : 0u;
                }
#pragma unroll
                for (int u = 0; u < kBatch; ++u)
                    if (i0 + u * kSelThreads < lim && i0 + u * kSelThreads >= skip_of(src)) consume(key[u]);
            }
        }
    }
    // this CTA's share of the pass is read: once every CTA is here the next kernel of the chain may be scheduled
    // (not earlier: the kernels after it would follow one by one and sit on the SMs while this one still works)
    chain_release_next();
    __syncthreads();

    uint32_t* hist = st->hist + kPass * kBins;
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
    finish_pass<kPass>(st, prefix, s_scan, tau_out, result);
}

template <int kPass, typename Source, bool kVectorised>
__global__ void __launch_bounds__(kSelThreads)
select_pass_kernel(Source src, SelectState* st, float* __restrict__ tau_out, dct_result_t* __restrict__ result) {
    __shared__ uint32_t sh[kBins];
    __shared__ uint32_t s_scan[kSelThreads / 32];
    __shared__ uint32_t s_last;
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) sh[b] = 0;
    chain_wait_previous();
    if (!st->enabled) return;
    select_pass_body<kPass, Source, kVectorised>(src, st, tau_out, result, st->n, sh, s_scan, s_last);
}

// The same pass for one of two selects: the one over the few candidates (the normal case) or, should the sample have
// misjudged the vector, the plain one over the whole vector -- one launch instead of two, of which one would return
// at once.  Which one: with k_decide == 0 the enabled flags of the two states say (a kernel before this one set
// them); otherwise every CTA of every pass decides for itself from the candidate count that the filter left, the
// same way each time: the candidates if rank k_decide lies among them (fewer than k_decide keys above them, at least
// k_decide together with those) and all fitted into their buffer.
template <int kPass, typename CandSource, bool kVectorised>
__global__ void __launch_bounds__(kSelThreads)
select_pass_either_kernel(CandSource cand_src, VectorSource full_src, SelectWorkspace* ws, uint32_t k_decide,
                          float* __restrict__ tau_out, dct_result_t* __restrict__ result) {
    __shared__ uint32_t sh[kBins];
    __shared__ uint32_t s_scan[kSelThreads / 32];
    __shared__ uint32_t s_last;
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) sh[b] = 0;
    chain_wait_previous();
    bool use_cand, use_full;
    uint32_t cand_n;
    if (k_decide) {
        cand_n = ws->cand_count;
        const uint32_t above = ws->above_count;       // (the filter has set the candidates' rank to k_decide - above)
        use_cand = above < k_decide && k_decide - above <= cand_n && cand_n <= ws->cand_capacity;
        use_full = !use_cand;
    } else {
        cand_n = ws->cand.n;
        use_cand = ws->cand.enabled != 0;
        use_full = ws->full.enabled != 0;
    }
    if (use_cand)
        select_pass_body<kPass, CandSource, false>(cand_src, &ws->cand, tau_out, result, cand_n, sh, s_scan, s_last);
    else if (use_full)
        select_pass_body<kPass, VectorSource, kVectorised>(full_src, &ws->full, tau_out, result, ws->full.n, sh, s_scan,
                                                           s_last);
}

// The single streaming pass of the sampled path: every key in [lo, hi] goes to the candidate buffer and the keys
// above hi are counted (without an upper bound hi is the largest key: nothing is above it).  The last CTA to finish
// hands the candidate select its rank: k less the keys above hi.
template <bool kVectorised, bool kBand>
__global__ void __launch_bounds__(kSelThreads)
select_filter_kernel(VectorSource src, uint32_t n, SelectWorkspace* ws, uint32_t* __restrict__ cand_keys) {
    chain_wait_previous();
    if (!ws->sample.enabled) return;
    const uint32_t lo = ws->sample.key_out;
    const uint32_t hi = kBand ? (ws->sample_hi.key_out | ((1u << pass_shift(1)) - 1u)) : 0xFFFFFFFFu;
    const uint32_t capacity = ws->cand_capacity;
    uint32_t above = 0;                             // keys above hi seen by this thread
    // Each warp collects its survivors in a small shared-memory buffer and moves them to the candidate
    // buffer 64 or more at a time, so the global counter sees one atomic per flush, not one per survivor.
    constexpr uint32_t kWarpBuf = 96, kFlushAt = 64;
    __shared__ uint32_t s_buf[kSelThreads / 32][kWarpBuf];
    uint32_t* wbuf = s_buf[threadIdx.x >> 5];
    uint32_t held = 0;                              // warp-uniform
    auto flush = [&]() {
        __syncwarp();
        uint32_t base = 0;
        if (lane_id() == 0) base = atomicAdd(&ws->cand_count, held);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        for (uint32_t i = lane_id(); i < held; i += 32)
            if (base + i < capacity) cand_keys[base + i] = wbuf[i];
        __syncwarp();
        held = 0;
    };
    auto keep = [&](bool pred, uint32_t key) {      // called by whole warps
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, pred);
        if (bal == 0) return;
        if (pred) wbuf[held + __popc(bal & lanemask_lt())] = key;
        held += __popc(bal);
        if (held >= kFlushAt) flush();
    };
    const uint32_t num_chunks = (n + kSelChunk - 1) / kSelChunk;
    for (uint32_t chunk = blockIdx.x; chunk < num_chunks; chunk += gridDim.x) {
        const uint32_t base = chunk * kSelChunk;
        if (kVectorised && base + kSelChunk <= n && base >= src.skip) {
            float4 g4[kSelVecs], e4[kSelVecs];
#pragma unroll
            for (int j = 0; j < kSelVecs; ++j) {
                const uint32_t off = base + (j * kSelThreads + threadIdx.x) * 4;
                g4[j] = ld_readonly_f4(src.grad + off);
                e4[j] = src.residual ? ld_readonly_f4(src.residual + off) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const bool add = src.residual != nullptr;
#pragma unroll
            for (int j = 0; j < kSelVecs; ++j) {
                const uint32_t k0 = key_f32(add ? __fadd_rn(g4[j].x, e4[j].x) : g4[j].x);
                const uint32_t k1 = key_f32(add ? __fadd_rn(g4[j].y, e4[j].y) : g4[j].y);
                const uint32_t k2 = key_f32(add ? __fadd_rn(g4[j].z, e4[j].z) : g4[j].z);
                const uint32_t k3 = key_f32(add ? __fadd_rn(g4[j].w, e4[j].w) : g4[j].w);
                if (kBand) above += (k0 > hi ? 1u : 0u) + (k1 > hi ? 1u : 0u) + (k2 > hi ? 1u : 0u) + (k3 > hi ? 1u : 0u);
                const bool in0 = k0 >= lo && (!kBand || k0 <= hi), in1 = k1 >= lo && (!kBand || k1 <= hi);
                const bool in2 = k2 >= lo && (!kBand || k2 <= hi), in3 = k3 >= lo && (!kBand || k3 <= hi);
                const uint32_t top = max(max(k0, k1), max(k2, k3));
                if (__any_sync(0xFFFFFFFFu, kBand ? (in0 || in1 || in2 || in3) : top >= lo)) {
                    keep(in0, k0);
                    keep(in1, k1);
                    keep(in2, k2);
                    keep(in3, k3);
                }
            }
        } else {
            // whole warps stay together so that the ballots above see every lane
            for (uint32_t i0 = base + (threadIdx.x & ~31u); i0 < n && i0 < base + kSelChunk; i0 += kSelThreads) {
                const uint32_t i = i0 + lane_id();
                const bool in = i < n && i < base + kSelChunk && i >= src.skip;
                const uint32_t key = in ? key_at(src, i) : 0u;
                above += in && key > hi ? 1u : 0u;
                keep(in && key >= lo && key <= hi, key);
            }
        }
    }
    chain_release_next();
    if (held) flush();
    above = __reduce_add_sync(0xFFFFFFFFu, above);
    if (lane_id() == 0 && above) atomicAdd(&ws->above_count, above);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0 && atomicAdd(&ws->filter_done, 1u) == gridDim.x - 1) {
        __threadfence();
        const uint32_t all_above = ld_relaxed_u32(&ws->above_count), k = ws->k_total;
        ws->cand.k_rem = all_above < k ? k - all_above : k;     // (not below k: the candidates are not used then)
        ws->cand.n_gt = all_above;
    }
}

template <typename Source, bool kVectorised>
cudaError_t launch_three_passes(int grid, cudaStream_t stream, Source src, SelectState* st, float* tau_out,
                                dct_result_t* result, int passes = kPasses) {
    cudaError_t e = launch_chained(select_pass_kernel<0, Source, kVectorised>, grid, kSelThreads, stream, src, st, tau_out, result);
    if (e == cudaSuccess && passes > 1)
        e = launch_chained(select_pass_kernel<1, Source, kVectorised>, grid, kSelThreads, stream, src, st, tau_out, result);
    if (e == cudaSuccess && passes > 2)
        e = launch_chained(select_pass_kernel<2, Source, kVectorised>, grid, kSelThreads, stream, src, st, tau_out, result);
    return e;
}

// The two passes of the sample select (its state says that pass 1 is its last).
constexpr int kSamplePasses = 2;

// Three launches that run the candidate select or the select over the whole vector (k_decide: see the kernel).  The
// grid is the vector's: the few candidates are spread over it.
template <typename CandSource>
cudaError_t launch_three_either(int grid, cudaStream_t stream, CandSource csrc, VectorSource vsrc, bool vectorised,
                                SelectWorkspace* ws, uint32_t k_decide, float* tau_out, dct_result_t* result) {
    cudaError_t e;
    if (vectorised) {
        e = launch_chained(select_pass_either_kernel<0, CandSource, true>, grid, kSelThreads, stream, csrc, vsrc, ws, k_decide, tau_out, result);
        if (e == cudaSuccess)
            e = launch_chained(select_pass_either_kernel<1, CandSource, true>, grid, kSelThreads, stream, csrc, vsrc, ws, k_decide, tau_out, result);
        if (e == cudaSuccess)
            e = launch_chained(select_pass_either_kernel<2, CandSource, true>, grid, kSelThreads, stream, csrc, vsrc, ws, k_decide, tau_out, result);
    } else {
        e = launch_chained(select_pass_either_kernel<0, CandSource, false>, grid, kSelThreads, stream, csrc, vsrc, ws, k_decide, tau_out, result);
        if (e == cudaSuccess)
            e = launch_chained(select_pass_either_kernel<1, CandSource, false>, grid, kSelThreads, stream, csrc, vsrc, ws, k_decide, tau_out, result);
        if (e == cudaSuccess)
            e = launch_chained(select_pass_either_kernel<2, CandSource, false>, grid, kSelThreads, stream, csrc, vsrc, ws, k_decide, tau_out, result);
    }
    return e;
}

// Rank to select in the sample so that the number of vector elements at or above the sampled value is,
// six standard deviations out, still at least k: returns 0 if that would overflow the candidate buffer.
uint32_t sample_rank(uint64_t n, uint64_t k, uint32_t sample_n, uint32_t capacity) {
    const double m = static_cast<double>(k) * sample_n / static_cast<double>(n);   // expected sample rank of tau
    const double r = m + 6.0 * __builtin_sqrt(m + 1.0) + 20.0;
    const double expected_max = (r + 6.0 * __builtin_sqrt(r)) * static_cast<double>(n) / sample_n;
    if (r >= sample_n / 4.0 || expected_max > capacity) return 0;
    return static_cast<uint32_t>(r);
}

// The same for k too large for that: two ranks, one on either side of tau's expected rank in the sample, so that
// rank k lies, six standard deviations out, between the two sampled values, and the vector elements between them
// fit the candidate buffer.  Returns false if there is no such pair.
bool sample_band(uint64_t n, uint64_t k, uint32_t sample_n, uint32_t capacity, uint32_t* rank_lo, uint32_t* rank_hi) {
    const double m = static_cast<double>(k) * sample_n / static_cast<double>(n);
    const double margin = 6.0 * __builtin_sqrt(m + 1.0) + 20.0;
    const double lo = m + margin, hi = m - margin;
    if (hi < 1.0 || lo >= sample_n / 2.0) return false;
    const double between = lo - hi;
    const double per_sample = static_cast<double>(n) / sample_n;
    // the elements between the two sampled values, six standard deviations out, and those the two-pass sample
    // selects add by rounding their values to 21 bits
    const double expected_max = (between + 6.0 * __builtin_sqrt(between)) * per_sample + static_cast<double>(n) / 2048.0;
    if (expected_max > capacity) return false;
    *rank_lo = static_cast<uint32_t>(lo);
    *rank_hi = static_cast<uint32_t>(hi);
    return true;
}

uint32_t candidate_capacity(uint64_t n) {
    return static_cast<uint32_t>(n < kMaxCandidates ? n : kMaxCandidates);
}

// L = 1: after the compress pass that extracted the candidates.  The list is usable if it holds at least k
// elements and nothing was cut off; otherwise the plain select runs on w.
__global__ void l1_decide_kernel(SelectWorkspace* ws, L1Block* block, uint32_t k, uint32_t cand_capacity) {
    chain_release_next();
    chain_wait_previous();
    const uint64_t found = block->cand_result.needed;
    const bool ok = block->cand_result.status == DCT_OK && found >= k && found <= cand_capacity;
    block->use_candidates = ok ? 1u : 0u;
    block->fallback = ok ? 0u : 1u;
    block->cand_count = static_cast<uint32_t>(block->cand_result.count);
    ws->cand.n = static_cast<uint32_t>(found);
    ws->cand.enabled = ok ? 1u : 0u;
    ws->full.enabled = ok ? 0u : 1u;
}
// the candidates go back into the residual, which then holds w = g + e everywhere
__global__ void l1_restore_kernel(const int32_t* __restrict__ cand_idx, const float* __restrict__ cand_val,
                                  float* __restrict__ residual, const L1Block* block) {
    chain_release_next();
    chain_wait_previous();
    if (!block->fallback) return;
    const uint32_t c = block->cand_count;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < c; i += gridDim.x * blockDim.x)
        residual[cand_idx[i]] = cand_val[i];
}
__global__ void l1_budget_kernel(L1Block* block, const dct_result_t* sel, uint64_t k) {
    chain_release_next();
    chain_wait_previous();
    block->n_gt = sel->n_gt;
    block->n_eq = sel->n_eq;
    block->tie_budget = k > sel->n_gt ? k - sel->n_gt : 0;
}

}  // namespace

bool l1_sampled_path_applies(uint64_t n, uint64_t k, uint64_t cand_capacity) {
    if (n < kMinSampledN || n > 0x7FFFFFFFull || cand_capacity == 0) return false;
    const uint64_t cap = cand_capacity < 0xFFFFFFFFull ? cand_capacity : 0xFFFFFFFFull;
    return sample_rank(n, k, kSampleSize, static_cast<uint32_t>(cap)) != 0;
}

dct_status_t l1_sample_bound(const float* grad, const float* residual, uint64_t n, uint64_t k, uint64_t cand_capacity,
                             L1Block* block, void* select_ws, cudaStream_t stream) {
    auto* ws = static_cast<SelectWorkspace*>(select_ws);
    const uint32_t n32 = static_cast<uint32_t>(n), k32 = static_cast<uint32_t>(k);
    const uint32_t cap = static_cast<uint32_t>(cand_capacity < 0xFFFFFFFFull ? cand_capacity : 0xFFFFFFFFull);
    const uint32_t sample_k = sample_rank(n, k, kSampleSize, cap);
    if (sample_k == 0) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint32_t stride = (n32 / (kSampleSize / kSampleGroup)) & ~(kSampleGroup - 1u);
    select_init_kernel<<<1, kInitThreads, 0, stream>>>(ws, n32, k32, kSampleSize, sample_k, cap, &block->scratch);
    DCT_CUDA_TRY(cudaGetLastError());
    const StridedSource ssrc{grad, residual, stride};
    const uint64_t chunks = (kSampleSize + kSelChunk - 1) / kSelChunk;
    const int grid = static_cast<int>(chunks < static_cast<uint64_t>(sms) * 4 ? chunks : sms * 4);
    DCT_CUDA_TRY((launch_three_passes<StridedSource, false>(grid, stream, ssrc, &ws->sample, &block->lo, &block->scratch,
                                                            kSamplePasses)));
    return DCT_OK;
}

dct_status_t l1_exact_threshold(const int32_t* cand_idx, const float* cand_val, uint64_t cand_capacity, float* residual,
                                uint64_t n, uint64_t k, float* tau_out, L1Block* block, void* select_ws,
                                cudaStream_t stream) {
    auto* ws = static_cast<SelectWorkspace*>(select_ws);
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint32_t cap = static_cast<uint32_t>(cand_capacity < 0xFFFFFFFFull ? cand_capacity : 0xFFFFFFFFull);
    DCT_CUDA_TRY(launch_chained(l1_decide_kernel, 1, 1, stream, ws, block, static_cast<uint32_t>(k), cap));
    DCT_CUDA_TRY(launch_chained(l1_restore_kernel, sms * 2, 256, stream, cand_idx, cand_val, residual,
                                static_cast<const L1Block*>(block)));
    // the exact select: over the candidates (normally), or over w
    const ValueSource csrc{cand_val};
    const VectorSource wsrc{residual, nullptr};
    const uint64_t chunks = (n + kSelChunk - 1) / kSelChunk;
    const int grid = static_cast<int>(chunks < static_cast<uint64_t>(sms) * 4 ? (chunks ? chunks : 1) : sms * 4);
    DCT_CUDA_TRY(launch_three_either(grid, stream, csrc, wsrc, aligned_to(residual, 16), ws, 0u, tau_out,
                                     &block->scratch));
    DCT_CUDA_TRY(launch_chained(l1_budget_kernel, 1, 1, stream, block, static_cast<const dct_result_t*>(&block->scratch), k));
    return DCT_OK;
}

}  // namespace dct

using namespace dct;

extern "C" size_t dct_threshold_select_workspace_bytes(uint64_t n) {
    if (n == 0 || n > 0x7FFFFFFFull) return 0;
    size_t bytes = sizeof(SelectWorkspace);
    if (n >= kMinSampledN) bytes += sizeof(uint32_t) * static_cast<size_t>(candidate_capacity(n));
    return (bytes + 255) & ~static_cast<size_t>(255);
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
    auto* ws = static_cast<SelectWorkspace*>(workspace);
    auto* cand_keys = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + sizeof(SelectWorkspace));
    // A vector 4, 8 or 12 bytes past a 16-byte boundary (and a residual, if any, at the same offset) is read from that
    // boundary: the 1 to 3 elements before it share its first 16 bytes, are loaded and not counted.
    uint32_t lead = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(grad) & 15u) / 4u);
    if ((residual && lead != (reinterpret_cast<uintptr_t>(residual) & 15u) / 4u) || n + lead > 0x7FFFFFFFull) lead = 0;
    grad -= lead;
    if (residual) residual -= lead;
    const uint64_t n_own = n;                       // (the workspace was sized for this many elements)
    n += lead;
    const uint32_t n32 = static_cast<uint32_t>(n), k32 = static_cast<uint32_t>(k);
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    auto grid_for = [&](uint64_t elems) {
        const uint64_t chunks = (elems + kSelChunk - 1) / kSelChunk;
        return static_cast<int>(chunks < static_cast<uint64_t>(sms) * 4 ? (chunks ? chunks : 1) : sms * 4);
    };
    const bool vec = aligned_to(grad, 16) && (!residual || aligned_to(residual, 16));
    const VectorSource vsrc{grad, residual, lead};

    // sampled single-pass path?
    uint32_t sample_n = 0, sample_k = 0, sample_k_hi = 0, stride = 0, capacity = 0;
    if (n_own >= kMinSampledN) {
        capacity = candidate_capacity(n_own);
        stride = (n32 / (kSampleSize / kSampleGroup)) & ~(kSampleGroup - 1u);   // groups start on 32-byte boundaries
        sample_n = kSampleSize;
        // millions of elements above tau: the band around tau is the shorter candidate list, where there is one
        const bool band = k >= kBandFromK && sample_band(n, k, sample_n, capacity, &sample_k, &sample_k_hi);
        if (!band) {
            sample_k = sample_rank(n, k, sample_n, capacity);
            if (sample_k == 0 && !sample_band(n, k, sample_n, capacity, &sample_k, &sample_k_hi)) sample_n = 0;
        }
    }

    select_init_kernel<<<1, kInitThreads, 0, stream>>>(ws, n32, k32, sample_n, sample_k, capacity, result, sample_k_hi);
    DCT_CUDA_TRY(cudaGetLastError());
    if (sample_n) {
        const StridedSource ssrc{grad, residual, stride};
        DCT_CUDA_TRY((launch_three_passes<StridedSource, false>(grid_for(sample_n), stream, ssrc, &ws->sample, nullptr,
                                                                result, kSamplePasses)));
        if (sample_k_hi)
            DCT_CUDA_TRY((launch_three_passes<StridedSource, false>(grid_for(sample_n), stream, ssrc, &ws->sample_hi,
                                                                    nullptr, result, kSamplePasses)));
        auto* filter = vec ? (sample_k_hi ? select_filter_kernel<true, true> : select_filter_kernel<true, false>)
                           : (sample_k_hi ? select_filter_kernel<false, true> : select_filter_kernel<false, false>);
        DCT_CUDA_TRY(launch_chained(filter, grid_for(n), kSelThreads, stream, vsrc, n32, ws, cand_keys));
        // the exact select over the candidates (their count is only known on the device) or, should the sample
        // have misjudged the vector, over the vector itself: the same three launches serve either
        const KeySource ksrc{cand_keys};
        DCT_CUDA_TRY(launch_three_either(grid_for(n), stream, ksrc, vsrc, vec, ws, k32, tau_out, result));
        return DCT_OK;
    }
    // small or dense problems: the plain three passes
    if (vec)
        DCT_CUDA_TRY((launch_three_passes<VectorSource, true>(grid_for(n), stream, vsrc, &ws->full, tau_out, result)));
    else
        DCT_CUDA_TRY((launch_three_passes<VectorSource, false>(grid_for(n), stream, vsrc, &ws->full, tau_out, result)));
    return DCT_OK;
}
