// dct_dp_select_compress: Algorithm 1 with threshold life-span L = 1 -- the threshold is recomputed from
// the very vector that is compressed (the branch "L divides the iteration number" taken every time), which
// is the plain top-K-with-error-feedback scheme the paper starts from and finds too expensive on CPUs.
//
// On the stream: exact select on fl32(grad + residual) -> tie budget k - n_gt -> compress with that
// budget, so that exactly k elements are sent (lowest index first among the ties) however many elements
// equal the threshold.  No host round trip in between.
#include "common.cuh"

namespace dct {
namespace {

struct ChainBlock {            // lives at the start of the workspace
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

size_t round256(size_t b) { return (b + 255) & ~static_cast<size_t>(255); }

}  // namespace
}  // namespace dct

using namespace dct;

extern "C" size_t dct_dp_select_compress_workspace_bytes(uint64_t n) {
    const size_t a = dct_threshold_select_workspace_bytes(n), b = dct_dp_compress_workspace_bytes(n);
    if (a == 0 || b == 0) return 0;
    return kChainBytes + round256(a) + round256(b);
}

extern "C" dct_status_t dct_dp_select_compress(const float* grad, float* residual, uint64_t n, uint64_t k,
                                               float* tau_out, int32_t* idx_out, float* val_out, uint64_t capacity,
                                               dct_result_t* result, void* workspace, size_t workspace_bytes,
                                               dct_stream_t stream_) {
    if (!grad || !residual || !tau_out || !result || n == 0 || n > 0x7FFFFFFFull || k == 0 || k > n)
        return DCT_ERR_INVALID_ARG;
    if (!workspace || !aligned_to(workspace, 256) || workspace_bytes < dct_dp_select_compress_workspace_bytes(n))
        return DCT_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    char* ws = static_cast<char*>(workspace);
    auto* chain = reinterpret_cast<ChainBlock*>(ws);
    const size_t sel_bytes = round256(dct_threshold_select_workspace_bytes(n));
    void* sel_ws = ws + kChainBytes;
    void* cmp_ws = ws + kChainBytes + sel_bytes;

    dct_status_t st = dct_threshold_select(grad, residual, n, k, tau_out, &chain->select_result, sel_ws, sel_bytes,
                                           stream_);
    if (st != DCT_OK) return st;
    chain_budget_kernel<<<1, 1, 0, stream>>>(chain, k);
    DCT_CUDA_TRY(cudaGetLastError());
    st = dct_dp_compress(grad, residual, n, tau_out, &chain->tie_budget, idx_out, val_out, capacity, result, cmp_ws,
                         workspace_bytes - kChainBytes - sel_bytes, stream_);
    if (st != DCT_OK) return st;
    chain_finish_kernel<<<1, 1, 0, stream>>>(chain, result);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}
