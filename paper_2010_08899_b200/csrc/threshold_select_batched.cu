// dct_threshold_select_batched: Algorithm 1 (DCT-DP), threshold steps, for all the layers of a model at
// once (Sec. 2.1: each layer has a threshold of its own, renewed every L iterations).
//
// The same most-significant-digit-first radix select as dct_threshold_select (digits of 11/10/10 bits
// over the 31 magnitude bits), carried out for every layer in the same three passes.  The elements of all
// layers are cut into chunks of 8192; every CTA takes a contiguous run of chunks, so it changes layer
// rarely, keeps the digit histogram of the layer it is in in shared memory and merges it into that
// layer's histogram in global memory when it moves on.  After each pass one CTA per layer scans the
// layer's histogram from the top, picks the digit that holds rank k and extends the layer's prefix.
#include <cstddef>
#include <vector>

#include "common.cuh"

namespace dct {
namespace {

constexpr int kThreads = 512;
constexpr int kVecs = 4;
constexpr uint32_t kChunk = kThreads * kVecs * 4;            // 8192 elements
constexpr int kBins = 2048;
constexpr int kPasses = 3;

__host__ __device__ constexpr int pass_shift(int p) { return p == 0 ? 20 : (p == 1 ? 10 : 0); }
__host__ __device__ constexpr int pass_bits(int p) { return p == 0 ? 11 : 10; }

struct LayerState {                 // device copy of a layer's description + its select in flight
    const float* grad;
    const float* residual;
    float* tau_out;
    dct_result_t* result;
    uint64_t first_chunk;           // index of the layer's first chunk among all chunks
    uint64_t n_gt;                  // elements known to be above the prefix bucket
    uint32_t n, k;
    uint32_t prefix, k_rem;
    uint32_t skip;                  // leading elements that are not the layer's (see LayerHead::skip)
    uint32_t pad;
    uint32_t hist[kPasses][kBins];
};

// What the host says about a layer: the head of its LayerState.  The heads of all layers travel as one contiguous copy
// into a staging area behind the states (a strided copy of 48 bytes per 24 KiB cost 0.6 ms for 4096 layers); the
// reset kernel puts each into place.
struct LayerHead {
    const float* grad;
    const float* residual;
    float* tau_out;
    dct_result_t* result;
    uint64_t first_chunk;
    uint64_t n_gt;
    uint32_t n, k;
    uint32_t skip;                  // a layer 4, 8 or 12 bytes past a 16-byte boundary (and its residual with it) is read
    uint32_t pad;                   // from that boundary: grad, residual and n count from there, the first `skip`
};                                  // elements are loaded and not counted

// chunk -> layer: the last layer whose first chunk is <= chunk
__device__ __forceinline__ uint32_t layer_of_chunk(const LayerState* layers, uint32_t num_layers, uint64_t chunk) {
    uint32_t lo = 0, hi = num_layers - 1;
    while (lo < hi) {
        const uint32_t mid = (lo + hi + 1) >> 1;
        if (layers[mid].first_chunk <= chunk) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__global__ void batched_init_kernel(LayerState* layers, const LayerHead* heads, uint32_t num_layers) {
    chain_release_next();
    // put the description in place; clear the select state, the histograms and the result
    for (uint32_t l = blockIdx.x; l < num_layers; l += gridDim.x) {
        LayerState* st = layers + l;
        uint32_t* h = &st->hist[0][0];
        for (uint32_t b = threadIdx.x; b < kPasses * kBins; b += blockDim.x) h[b] = 0;
        if (threadIdx.x == 0) {
            const LayerHead hd = heads[l];
            st->grad = hd.grad;
            st->residual = hd.residual;
            st->tau_out = hd.tau_out;
            st->result = hd.result;
            st->first_chunk = hd.first_chunk;
            st->n = hd.n;
            st->k = hd.k;
            st->skip = hd.skip;
            st->n_gt = 0;
            st->prefix = 0;
            st->k_rem = hd.k;
            dct_result_t* r = st->result;
            r->status = DCT_OK;
            r->reserved = 0;
            r->count = 0;
            r->needed = 0;
            r->n_gt = 0;
            r->n_eq = 0;
        }
    }
}

template <int kPass>
__global__ void __launch_bounds__(kThreads)
batched_pass_kernel(LayerState* layers, uint32_t num_layers, uint64_t total_chunks) {
    constexpr int shift = pass_shift(kPass);
    constexpr int bits = pass_bits(kPass);
    constexpr uint32_t digit_mask = (1u << bits) - 1u;
    __shared__ uint32_t sh[kBins];

    // this CTA's contiguous run of chunks
    const uint64_t per_cta = (total_chunks + gridDim.x - 1) / gridDim.x;
    const uint64_t c_begin = static_cast<uint64_t>(blockIdx.x) * per_cta;
    const uint64_t c_end = c_begin + per_cta < total_chunks ? c_begin + per_cta : total_chunks;
    if (c_begin >= c_end) return;

    for (int b = threadIdx.x; b < kBins; b += kThreads) sh[b] = 0;
    chain_wait_previous();
    uint32_t layer = layer_of_chunk(layers, num_layers, c_begin);
    __syncthreads();

    auto flush = [&](uint32_t l) {          // merge the shared histogram into layer l's and clear it
        __syncthreads();
        uint32_t* hist = layers[l].hist[kPass];
        for (int b = threadIdx.x; b < kBins; b += kThreads) {
            const uint32_t c = sh[b];
            if (c) {
                atomicAdd(&hist[b], c);
                sh[b] = 0;
            }
        }
        __syncthreads();
    };

    for (uint64_t chunk = c_begin; chunk < c_end; ++chunk) {
        while (layer + 1 < num_layers && layers[layer + 1].first_chunk <= chunk) {     // the run has entered the next layer
            flush(layer);
            ++layer;
        }
        const LayerState& st = layers[layer];
        const float* __restrict__ grad = st.grad;
        const float* __restrict__ residual = st.residual;
        const uint32_t n = st.n;
        const uint32_t prefix = kPass == 0 ? 0u : st.prefix;      // written by the scan kernel of the previous pass
        const uint32_t base = static_cast<uint32_t>(chunk - st.first_chunk) * kChunk;
        auto consume = [&](uint32_t key) {
            if (kPass == 0 || (key >> (shift + bits)) == prefix) atomicAdd(&sh[(key >> shift) & digit_mask], 1u);
        };
        const bool vec = (reinterpret_cast<uintptr_t>(grad) & 15u) == 0 &&
                         (residual == nullptr || (reinterpret_cast<uintptr_t>(residual) & 15u) == 0);
        const uint32_t skip = st.skip;
        if (vec && base + kChunk <= n && base >= skip) {
            float4 g4[kVecs], e4[kVecs];
#pragma unroll
            for (int j = 0; j < kVecs; ++j) {
                const uint32_t off = base + (j * kThreads + threadIdx.x) * 4;
                g4[j] = ld_readonly_f4(grad + off);
                e4[j] = residual ? ld_readonly_f4(residual + off) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const bool add = residual != nullptr;
#pragma unroll
            for (int j = 0; j < kVecs; ++j) {
                consume(key_f32(add ? __fadd_rn(g4[j].x, e4[j].x) : g4[j].x));
                consume(key_f32(add ? __fadd_rn(g4[j].y, e4[j].y) : g4[j].y));
                consume(key_f32(add ? __fadd_rn(g4[j].z, e4[j].z) : g4[j].z));
                consume(key_f32(add ? __fadd_rn(g4[j].w, e4[j].w) : g4[j].w));
            }
        } else {
            for (uint32_t i = base + threadIdx.x; i < n && i < base + kChunk; i += kThreads)
                if (i >= skip) consume(key_f32(residual ? __fadd_rn(grad[i], residual[i]) : grad[i]));
        }
    }
    chain_release_next();
    flush(layer);
}

// One CTA per layer: the digit that holds rank k_rem, counted from the top of the layer's histogram.
template <int kPass>
__global__ void __launch_bounds__(kThreads)
batched_scan_kernel(LayerState* layers, uint32_t num_layers) {
    constexpr int bits = pass_bits(kPass);
    __shared__ uint32_t s_scan[kThreads / 32];
    chain_release_next();
    chain_wait_previous();
    for (uint32_t l = blockIdx.x; l < num_layers; l += gridDim.x) {
        LayerState* st = layers + l;
        const uint32_t* hist = st->hist[kPass];
        const uint32_t prefix = kPass == 0 ? 0u : st->prefix;
        const uint32_t k_rem = st->k_rem;
        // thread t owns bins top-down: bin(t, q) = kBins-1 - (4t + q), q = 0..3
        uint32_t c[4], own = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            c[q] = hist[kBins - 1 - (4 * threadIdx.x + q)];
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
        __syncthreads();                       // also: every thread has read prefix and k_rem
        uint32_t above = incl - own;
        for (uint32_t v = 0; v < warp; ++v) above += s_scan[v];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (above < k_rem && k_rem <= above + c[q]) {
                const uint32_t digit = kBins - 1 - (4 * threadIdx.x + q);
                const uint32_t new_prefix = (prefix << bits) | digit;
                const uint64_t n_gt = st->n_gt + above;
                st->prefix = new_prefix;
                st->k_rem = k_rem - above;
                st->n_gt = n_gt;
                if (kPass == kPasses - 1) {
                    *st->tau_out = __uint_as_float(new_prefix);
                    st->result->n_gt = n_gt;
                    st->result->n_eq = c[q];
                }
            }
            above += c[q];
        }
        __syncthreads();                       // s_scan is reused for the next layer
    }
}

}  // namespace
}  // namespace dct

using namespace dct;

extern "C" size_t dct_threshold_select_batched_workspace_bytes(uint32_t num_layers) {
    if (num_layers == 0) return 0;
    return (static_cast<size_t>(num_layers) * (sizeof(LayerState) + sizeof(LayerHead)) + 255) & ~static_cast<size_t>(255);
}

extern "C" dct_status_t dct_threshold_select_batched(const dct_select_layer_t* layers, uint32_t num_layers,
                                                     void* workspace, size_t workspace_bytes, dct_stream_t stream_) {
    if (!layers || num_layers == 0) return DCT_ERR_INVALID_ARG;
    if (stream_is_capturing(static_cast<cudaStream_t>(stream_))) return DCT_ERR_UNSUPPORTED;   // uploads a temporary table
    uint64_t total_chunks = 0, total_elems = 0;
    for (uint32_t l = 0; l < num_layers; ++l) {
        const dct_select_layer_t& a = layers[l];
        if (!a.grad || !a.tau_out || !a.result || a.n == 0 || a.n > 0x7FFFFFFFull || a.k == 0 || a.k > a.n)
            return DCT_ERR_INVALID_ARG;
        if (!aligned_to(a.grad, 4) || (a.residual && !aligned_to(a.residual, 4)) || !aligned_to(a.tau_out, 4) ||
            !aligned_to(a.result, 8))
            return DCT_ERR_INVALID_ARG;
        total_elems += a.n;
    }
    if (total_elems >= (1ull << 44)) return DCT_ERR_INVALID_ARG;
    if (!workspace || !aligned_to(workspace, 256) ||
        workspace_bytes < dct_threshold_select_batched_workspace_bytes(num_layers))
        return DCT_ERR_WORKSPACE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    auto* dev_layers = static_cast<LayerState*>(workspace);
    auto* dev_heads = reinterpret_cast<LayerHead*>(dev_layers + num_layers);
    // only the descriptions travel; the histograms are cleared on the device
    std::vector<LayerHead> heads(num_layers);
    for (uint32_t l = 0; l < num_layers; ++l) {
        const dct_select_layer_t& a = layers[l];
        uint32_t lead = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(a.grad) & 15u) / 4u);
        if ((a.residual && lead != (reinterpret_cast<uintptr_t>(a.residual) & 15u) / 4u) || a.n + lead > 0x7FFFFFFFull)
            lead = 0;
        const uint64_t n_view = a.n + lead;
        heads[l] = LayerHead{a.grad - lead, a.residual ? a.residual - lead : nullptr, a.tau_out, a.result, total_chunks, 0,
                             static_cast<uint32_t>(n_view), static_cast<uint32_t>(a.k), lead, 0};
        total_chunks += (n_view + kChunk - 1) / kChunk;
    }
    // pageable source: the runtime has staged the bytes by the time the call returns, so `heads` may go away
    DCT_CUDA_TRY(cudaMemcpyAsync(dev_heads, heads.data(), sizeof(LayerHead) * num_layers, cudaMemcpyHostToDevice, stream));
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint32_t init_grid = num_layers < 1024u ? num_layers : 1024u;
    batched_init_kernel<<<init_grid, kThreads, 0, stream>>>(dev_layers, dev_heads, num_layers);
    DCT_CUDA_TRY(cudaGetLastError());
    const uint64_t want = static_cast<uint64_t>(sms) * 4;
    const uint32_t grid = static_cast<uint32_t>(total_chunks < want ? total_chunks : want);
    const uint32_t scan_grid = num_layers < static_cast<uint32_t>(sms) * 4u ? num_layers : static_cast<uint32_t>(sms) * 4u;
    // each kernel from here on is a programmatic dependent of the one before it (common.cuh)
    DCT_CUDA_TRY(launch_chained(batched_pass_kernel<0>, grid, kThreads, stream, dev_layers, num_layers, total_chunks));
    DCT_CUDA_TRY(launch_chained(batched_scan_kernel<0>, scan_grid, kThreads, stream, dev_layers, num_layers));
    DCT_CUDA_TRY(launch_chained(batched_pass_kernel<1>, grid, kThreads, stream, dev_layers, num_layers, total_chunks));
    DCT_CUDA_TRY(launch_chained(batched_scan_kernel<1>, scan_grid, kThreads, stream, dev_layers, num_layers));
    DCT_CUDA_TRY(launch_chained(batched_pass_kernel<2>, grid, kThreads, stream, dev_layers, num_layers, total_chunks));
    DCT_CUDA_TRY(launch_chained(batched_scan_kernel<2>, scan_grid, kThreads, stream, dev_layers, num_layers));
    return DCT_OK;
}
