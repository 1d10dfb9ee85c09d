// dct_dp_select_compress: Algorithm 1 with threshold life-span L = 1 -- the threshold is recomputed from
// the very vector that is compressed (the branch "L divides the iteration number" taken every time), which
// is the plain top-K-with-error-feedback scheme the paper starts from and finds too expensive on CPUs.
//
// Small vectors (below 2^25 elements) and dense k: exact select on fl32(grad + residual) -> tie budget k - n_gt ->
// compress with that budget, two operators back to back (20 bytes per element).
//
// Large vectors, k small against n (the method's regime): the vector is streamed ONCE, at the 12 bytes per
// element of a fixed-threshold iteration.
//   1. a lower bound `lo` of the threshold from a sector-wise sample of w = fl32(grad + residual) (the sample of
//      dct_threshold_select: k .. a few k elements lie at or above it, almost surely);
//   2. the streaming compress kernel with `lo` as its threshold: it forms w, leaves w in the residual, and packs
//      every element at or above `lo` -- the candidates -- in index order into the workspace (their residual
//      slots are zeroed, as for sent elements);
//   3. the exact radix select over the candidate values: tau, n_gt, n_eq are those of the whole vector, since
//      every element >= tau is a candidate;
//   4. a pass over the candidates only: the survivors (key > tau, then the lowest-index ties up to k) go, still in
//      index order, to the caller's buffers; the other candidates go back into their residual slots.
// If the sample has misjudged the vector (fewer than k candidates, or more than the list holds), the candidates are
// written back -- the residual then holds w everywhere -- and the plain select and compress run on w.  Every
// decision is taken on the device; the kernels of the path not taken return at once.
// Either way exactly k elements are sent (lowest index first among the ties) and the results are identical.
#include "common.cuh"
#include "dp_chain.cuh"

namespace dct {
namespace {

struct ChainBlock {            // lives at the start of the workspace (two-operator path)
    dct_result_t select_result;
    uint64_t tie_budget;
};
constexpr size_t kChainBytes = 256;

__global__ void chain_budget_kernel(ChainBlock* chain, uint64_t k) {
    const uint64_t n_gt = chain->select_result.n_gt;
    chain->tie_budget = k > n_gt ? k - n_gt : 0;
}
__global__ void chain_finish_kernel(const ChainBlock* chain, dct_result_t* result) {
    result->n_gt = chain->select_result.n_gt;
    result->n_eq = chain->select_result.n_eq;
}

// ---- one-pass path: the pass over the candidates -----------------------------------------------------------
constexpr uint64_t kL1MaxCandidates = 1ull << 22;     // 32 MiB of (index, value) pairs at most
constexpr uint32_t kL1MinN = 1u << 25;
constexpr int kFinGrid = 256, kFinThreads = 1024;
static_assert(sizeof(L1Block) <= 256, "the L = 1 state must fit its 256-byte slot");

__device__ __forceinline__ void fin_range(uint32_t c, uint32_t& begin, uint32_t& end) {
    const uint32_t per = (c + kFinGrid - 1) / kFinGrid;
    begin = blockIdx.x * per < c ? blockIdx.x * per : c;
    end = begin + per < c ? begin + per : c;
}
// (gt, eq) counts of every CTA's range of the candidate list
__global__ void __launch_bounds__(kFinThreads)
l1_count_kernel(const float* __restrict__ cand_val, const float* __restrict__ tau, const L1Block* block,
                uint2* __restrict__ counts) {
    chain_release_next();
    chain_wait_previous();
    if (!block->use_candidates) return;
    const uint32_t tau_key = key_f32(*tau);
    uint32_t begin, end;
    fin_range(block->cand_count, begin, end);
    uint32_t gt = 0, eq = 0;
    for (uint32_t i = begin + threadIdx.x; i < end; i += kFinThreads) {
        const uint32_t key = key_f32(cand_val[i]);
        gt += key > tau_key ? 1u : 0u;
        eq += key == tau_key ? 1u : 0u;
    }
    __shared__ uint32_t s_gt[kFinThreads / 32], s_eq[kFinThreads / 32];
    gt = __reduce_add_sync(0xFFFFFFFFu, gt);
    eq = __reduce_add_sync(0xFFFFFFFFu, eq);
    if (lane_id() == 0) {
        s_gt[threadIdx.x >> 5] = gt;
        s_eq[threadIdx.x >> 5] = eq;
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        gt = __reduce_add_sync(0xFFFFFFFFu, s_gt[threadIdx.x]);
        eq = __reduce_add_sync(0xFFFFFFFFu, s_eq[threadIdx.x]);
        if (threadIdx.x == 0) counts[blockIdx.x] = make_uint2(gt, eq);
    }
}
// Survivors to the caller's buffers in index order, the other candidates back into the residual.
__global__ void __launch_bounds__(kFinThreads)
l1_write_kernel(const int32_t* __restrict__ cand_idx, const float* __restrict__ cand_val, const float* __restrict__ tau,
                const L1Block* block, const uint2* __restrict__ counts, float* __restrict__ residual,
                int32_t* __restrict__ idx_out, float* __restrict__ val_out, uint64_t capacity,
                dct_result_t* __restrict__ result) {
    chain_release_next();
    chain_wait_previous();
    if (!block->use_candidates) return;
    __shared__ uint32_t s_gt[32], s_eq[32];
    __shared__ uint32_t s_base[2];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    const uint32_t tau_key = key_f32(*tau);
    const uint64_t budget = block->tie_budget;
    // counts of the ranges before this CTA's
    {
        uint32_t gt = 0, eq = 0;
        for (uint32_t b = threadIdx.x; b < blockIdx.x; b += kFinThreads) {
            const uint2 c = counts[b];
            gt += c.x;
            eq += c.y;
        }
        gt = __reduce_add_sync(0xFFFFFFFFu, gt);
        eq = __reduce_add_sync(0xFFFFFFFFu, eq);
        if (lane == 0) {
            s_gt[warp] = gt;
            s_eq[warp] = eq;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t a = 0, b = 0;
            for (int v = 0; v < kFinThreads / 32; ++v) {
                a += s_gt[v];
                b += s_eq[v];
            }
            s_base[0] = a;
            s_base[1] = b;
            if (blockIdx.x == gridDim.x - 1) {      // the last CTA knows the totals: the call's result
                const uint2 mine = counts[blockIdx.x];
                const uint64_t all_gt = static_cast<uint64_t>(a) + mine.x, all_eq = static_cast<uint64_t>(b) + mine.y;
                const uint64_t kept = all_gt + (all_eq < budget ? all_eq : budget);
                result->needed = kept;
                result->count = kept < capacity ? kept : capacity;
                result->n_gt = block->n_gt;
                result->n_eq = block->n_eq;
                result->status = kept > capacity ? DCT_ERR_CAPACITY : DCT_OK;
                result->reserved = 0;
            }
        }
        __syncthreads();
    }
    uint32_t gt_run = s_base[0], eq_run = s_base[1];
    uint32_t begin, end;
    fin_range(block->cand_count, begin, end);
    for (uint32_t i0 = begin; i0 < end; i0 += kFinThreads) {
        const uint32_t i = i0 + threadIdx.x;
        const bool in = i < end;
        const float v = in ? cand_val[i] : 0.0f;
        const int32_t at = in ? cand_idx[i] : 0;
        const uint32_t key = key_f32(v);
        const bool is_gt = in && key > tau_key, is_eq = in && key == tau_key;
        const uint32_t bg = __ballot_sync(0xFFFFFFFFu, is_gt), be = __ballot_sync(0xFFFFFFFFu, is_eq);
        __syncthreads();                      // the previous round's partial sums have been read
        if (lane == 0) {
            s_gt[warp] = __popc(bg);
            s_eq[warp] = __popc(be);
        }
        __syncthreads();
        uint32_t g_before = gt_run, e_before = eq_run, g_all = 0, e_all = 0;
        for (uint32_t w = 0; w < kFinThreads / 32; ++w) {
            const uint32_t a = s_gt[w], b = s_eq[w];
            if (w < warp) {
                g_before += a;
                e_before += b;
            }
            g_all += a;
            e_all += b;
        }
        g_before += __popc(bg & lanemask_lt());
        e_before += __popc(be & lanemask_lt());
        if (in) {
            const bool keep = is_gt || (is_eq && e_before < budget);
            const uint64_t pos = static_cast<uint64_t>(g_before) + (e_before < budget ? e_before : budget);
            if (keep && pos < capacity) {
                idx_out[pos] = at;
                val_out[pos] = v;
            } else {
                residual[at] = v;             // not sent: back into the error (its slot was zeroed with the candidates)
            }
        }
        gt_run += g_all;
        eq_run += e_all;
    }
}
// n_gt / n_eq of the exact threshold into the caller's result block (the plain way's compress has reset it)
__global__ void l1_finish_kernel(const L1Block* block, dct_result_t* result) {
    chain_wait_previous();
    if (!block->fallback) return;
    result->n_gt = block->n_gt;
    result->n_eq = block->n_eq;
}

size_t round256(size_t b) { return (b + 255) & ~static_cast<size_t>(255); }
constexpr size_t round_up_const(size_t b) { return (b + 255) & ~static_cast<size_t>(255); }

}  // namespace
}  // namespace dct

using namespace dct;

namespace {
uint64_t l1_candidate_capacity(uint64_t n) { return n < kL1MaxCandidates ? n : kL1MaxCandidates; }
constexpr size_t kFinCountBytes = round_up_const(sizeof(uint2) * kFinGrid);
}  // namespace

extern "C" size_t dct_dp_select_compress_workspace_bytes(uint64_t n) {
    const size_t a = dct_threshold_select_workspace_bytes(n), b = dct_dp_compress_workspace_bytes(n);
    if (a == 0 || b == 0) return 0;
    size_t bytes = kChainBytes + round256(a) + round256(b);
    if (n >= kL1MinN) bytes += kFinCountBytes + 2 * round256(sizeof(float) * static_cast<size_t>(l1_candidate_capacity(n)));
    return bytes;
}

extern "C" dct_status_t dct_dp_select_compress(const float* grad, float* residual, uint64_t n, uint64_t k,
                                               float* tau_out, int32_t* idx_out, float* val_out, uint64_t capacity,
                                               dct_result_t* result, void* workspace, size_t workspace_bytes,
                                               dct_stream_t stream_) {
    if (!grad || !residual || !tau_out || !result || n == 0 || n > 0x7FFFFFFFull || k == 0 || k > n)
        return DCT_ERR_INVALID_ARG;
    if (capacity > 0 && (!idx_out || !val_out)) return DCT_ERR_INVALID_ARG;
    if (!workspace || !aligned_to(workspace, 256) || workspace_bytes < dct_dp_select_compress_workspace_bytes(n))
        return DCT_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    char* ws = static_cast<char*>(workspace);
    const size_t sel_bytes = round256(dct_threshold_select_workspace_bytes(n));
    const size_t cmp_bytes = round256(dct_dp_compress_workspace_bytes(n));
    void* sel_ws = ws + kChainBytes;
    void* cmp_ws = ws + kChainBytes + sel_bytes;

    const uint64_t cand_cap = l1_candidate_capacity(n);
    if (n >= kL1MinN && l1_sampled_path_applies(n, k, cand_cap)) {
        // one streaming pass: sample bound -> candidates (compress kernel) -> exact select over them -> survivors
        auto* block = reinterpret_cast<L1Block*>(ws);
        char* at = ws + kChainBytes + sel_bytes + cmp_bytes;
        auto* counts = reinterpret_cast<uint2*>(at);
        at += kFinCountBytes;
        auto* cand_idx = reinterpret_cast<int32_t*>(at);
        at += round256(sizeof(float) * static_cast<size_t>(cand_cap));
        auto* cand_val = reinterpret_cast<float*>(at);
        dct_status_t st = l1_sample_bound(grad, residual, n, k, cand_cap, block, sel_ws, stream);
        if (st != DCT_OK) return st;
        st = dct_dp_compress(grad, residual, n, &block->lo, nullptr, cand_idx, cand_val, cand_cap, &block->cand_result,
                             cmp_ws, cmp_bytes, stream_);
        if (st != DCT_OK) return st;
        st = l1_exact_threshold(cand_idx, cand_val, cand_cap, residual, n, k, tau_out, block, sel_ws, stream);
        if (st != DCT_OK) return st;
        DCT_CUDA_TRY(launch_chained(l1_count_kernel, kFinGrid, kFinThreads, stream, static_cast<const float*>(cand_val),
                                    static_cast<const float*>(tau_out), static_cast<const L1Block*>(block), counts));
        DCT_CUDA_TRY(launch_chained(l1_write_kernel, kFinGrid, kFinThreads, stream, static_cast<const int32_t*>(cand_idx),
                                    static_cast<const float*>(cand_val), static_cast<const float*>(tau_out),
                                    static_cast<const L1Block*>(block), static_cast<const uint2*>(counts), residual, idx_out,
                                    val_out, capacity, result));
        // the plain way on w, should the sample have misjudged the vector (returns at once otherwise)
        st = compress_presummed_if(&block->fallback, residual, n, tau_out, &block->tie_budget, idx_out, val_out, capacity,
                                   result, cmp_ws, cmp_bytes, stream);
        if (st != DCT_OK) return st;
        l1_finish_kernel<<<1, 1, 0, stream>>>(block, result);
        DCT_CUDA_TRY(cudaGetLastError());
        return DCT_OK;
    }

    auto* chain = reinterpret_cast<ChainBlock*>(ws);
    dct_status_t st = dct_threshold_select(grad, residual, n, k, tau_out, &chain->select_result, sel_ws, sel_bytes,
                                           stream_);
    if (st != DCT_OK) return st;
    chain_budget_kernel<<<1, 1, 0, stream>>>(chain, k);
    DCT_CUDA_TRY(cudaGetLastError());
    st = dct_dp_compress(grad, residual, n, tau_out, &chain->tie_budget, idx_out, val_out, capacity, result, cmp_ws,
                         cmp_bytes, stream_);
    if (st != DCT_OK) return st;
    chain_finish_kernel<<<1, 1, 0, stream>>>(chain, result);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}
