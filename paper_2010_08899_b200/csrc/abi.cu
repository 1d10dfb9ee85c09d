// Host-side pieces of the C ABI that are not tied to one kernel: status names,
// error text, device queries, the testing knobs and the host-buffer wrappers.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace dct {

namespace {
thread_local char g_last_error[256] = "";
}

void note_cuda_error(cudaError_t e) {
    std::snprintf(g_last_error, sizeof g_last_error, "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    (void)cudaGetLastError();   // clear the sticky-free error state
}

namespace {
// about one second of waiting at the back-off the look-back uses; tile ids start at 0
std::atomic<uint32_t> g_spin_limit{1u << 21};
std::atomic<uint32_t> g_first_ticket{0u};
}  // namespace

DebugConfig debug_config() {
    return DebugConfig{g_spin_limit.load(std::memory_order_relaxed), g_first_ticket.load(std::memory_order_relaxed)};
}

int sm_count() {
    static std::mutex mu;
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
        cached[dev] = v;
    }
    return cached[dev];
}

uint32_t next_launch_ticket() {
    static std::atomic<uint32_t> counter{0x5EED0000u};
    uint32_t t = counter.fetch_add(1u, std::memory_order_relaxed) + 1u;
    return t != 0u ? t : counter.fetch_add(1u, std::memory_order_relaxed) + 1u;
}

}  // namespace dct

using namespace dct;

extern "C" const char* dct_status_string(dct_status_t s) {
    switch (s) {
        case DCT_OK: return "DCT_OK";
        case DCT_ERR_INVALID_ARG: return "DCT_ERR_INVALID_ARG";
        case DCT_ERR_WORKSPACE: return "DCT_ERR_WORKSPACE";
        case DCT_ERR_UNSUPPORTED: return "DCT_ERR_UNSUPPORTED";
        case DCT_ERR_CUDA: return "DCT_ERR_CUDA";
        case DCT_ERR_CAPACITY: return "DCT_ERR_CAPACITY";
        case DCT_ERR_TIMEOUT: return "DCT_ERR_TIMEOUT";
        case DCT_ERR_BAD_MASK: return "DCT_ERR_BAD_MASK";
    }
    return "DCT_ERR_UNKNOWN";
}

extern "C" const char* dct_last_cuda_error(void) { return g_last_error; }

extern "C" void dct_debug_configure(uint32_t spin_limit, uint32_t first_ticket) {
#ifndef DCT_NO_TEST_HOOKS
    g_spin_limit.store(spin_limit, std::memory_order_relaxed);
    g_first_ticket.store(first_ticket, std::memory_order_relaxed);
#else
    (void)spin_limit;
    (void)first_ticket;
#endif
}

extern "C" dct_status_t dct_dp_compress_host(const float* grad_host, float* grad_dev, float* residual_dev, uint64_t n,
                                             const float* tau_dev, const uint64_t* tie_budget_dev, int32_t* idx_dev,
                                             float* val_dev, uint64_t capacity, int32_t* idx_host, float* val_host,
                                             dct_result_t* result_dev, dct_result_t* result_host, void* workspace,
                                             size_t workspace_bytes, dct_stream_t stream_) {
    if (!grad_host || !grad_dev || !result_host || (capacity > 0 && (!idx_host || !val_host)))
        return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    DCT_CUDA_TRY(cudaMemcpyAsync(grad_dev, grad_host, n * sizeof(float), cudaMemcpyHostToDevice, stream));
    const dct_status_t st = dct_dp_compress(grad_dev, residual_dev, n, tau_dev, tie_budget_dev, idx_dev, val_dev,
                                            capacity, result_dev, workspace, workspace_bytes, stream_);
    if (st != DCT_OK) {
        (void)cudaStreamSynchronize(stream);      // the upload above is in flight: the caller's buffers are free on return
        return st;
    }
    DCT_CUDA_TRY(cudaMemcpyAsync(result_host, result_dev, sizeof(dct_result_t), cudaMemcpyDeviceToHost, stream));
    DCT_CUDA_TRY(cudaStreamSynchronize(stream));
    const uint64_t count = result_host->count;
    if (count > 0) {
        DCT_CUDA_TRY(cudaMemcpyAsync(idx_host, idx_dev, count * sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
        DCT_CUDA_TRY(cudaMemcpyAsync(val_host, val_dev, count * sizeof(float), cudaMemcpyDeviceToHost, stream));
        DCT_CUDA_TRY(cudaStreamSynchronize(stream));
    }
    return static_cast<dct_status_t>(result_host->status);
}

extern "C" dct_status_t dct_threshold_select_host(const float* grad_host, float* grad_dev, const float* residual_dev,
                                                  uint64_t n, uint64_t k, float* tau_dev, float* tau_host,
                                                  dct_result_t* result_dev, dct_result_t* result_host,
                                                  void* workspace, size_t workspace_bytes, dct_stream_t stream_) {
    if (!grad_host || !grad_dev || !result_host) return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    DCT_CUDA_TRY(cudaMemcpyAsync(grad_dev, grad_host, n * sizeof(float), cudaMemcpyHostToDevice, stream));
    const dct_status_t st = dct_threshold_select(grad_dev, residual_dev, n, k, tau_dev, result_dev, workspace,
                                                 workspace_bytes, stream_);
    if (st != DCT_OK) {
        (void)cudaStreamSynchronize(stream);
        return st;
    }
    if (tau_host) DCT_CUDA_TRY(cudaMemcpyAsync(tau_host, tau_dev, sizeof(float), cudaMemcpyDeviceToHost, stream));
    DCT_CUDA_TRY(cudaMemcpyAsync(result_host, result_dev, sizeof(dct_result_t), cudaMemcpyDeviceToHost, stream));
    DCT_CUDA_TRY(cudaStreamSynchronize(stream));
    return static_cast<dct_status_t>(result_host->status);
}

extern "C" dct_status_t dct_mp_pack_host(const void* x_act_host, const void* x_grad_host, void* x_act_dev,
                                         void* x_grad_dev, dct_dtype_t dtype, uint32_t rows, uint32_t d, uint32_t ld,
                                         uint32_t k, int16_t* cols_dev, void* vals_dev, void* gvals_dev,
                                         int16_t* cols_host, void* vals_host, void* gvals_host,
                                         dct_result_t* result_dev, dct_result_t* result_host, dct_stream_t stream_) {
    if (!x_act_host || !x_grad_host || !x_act_dev || !x_grad_dev || !cols_host || !vals_host || !gvals_host ||
        !result_dev || !result_host)
        return DCT_ERR_INVALID_ARG;
    if (dtype != DCT_F32 && dtype != DCT_BF16) return DCT_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t es = dtype == DCT_F32 ? 4 : 2;
    const size_t mat_bytes = static_cast<size_t>(rows) * ld * es;
    const size_t slots = static_cast<size_t>(rows) * k;
    DCT_CUDA_TRY(cudaMemcpyAsync(x_act_dev, x_act_host, mat_bytes, cudaMemcpyHostToDevice, stream));
    dct_status_t st = dct_mp_topk_pack_fwd(x_act_dev, dtype, rows, d, ld, k, cols_dev, vals_dev, nullptr, nullptr,
                                           result_dev, stream_);
    if (st != DCT_OK) {
        (void)cudaStreamSynchronize(stream);
        return st;
    }
    // the forward status leaves the device before the backward call reuses the result block
    DCT_CUDA_TRY(cudaMemcpyAsync(result_host, result_dev, sizeof(dct_result_t), cudaMemcpyDeviceToHost, stream));
    DCT_CUDA_TRY(cudaMemcpyAsync(cols_host, cols_dev, slots * sizeof(int16_t), cudaMemcpyDeviceToHost, stream));
    DCT_CUDA_TRY(cudaMemcpyAsync(vals_host, vals_dev, slots * es, cudaMemcpyDeviceToHost, stream));
    DCT_CUDA_TRY(cudaMemcpyAsync(x_grad_dev, x_grad_host, mat_bytes, cudaMemcpyHostToDevice, stream));
    st = dct_mp_pack_bwd(x_grad_dev, dtype, rows, d, ld, k, cols_dev, gvals_dev, result_dev, stream_);
    if (st != DCT_OK) {
        (void)cudaStreamSynchronize(stream);
        return st;
    }
    DCT_CUDA_TRY(cudaMemcpyAsync(gvals_host, gvals_dev, slots * es, cudaMemcpyDeviceToHost, stream));
    dct_result_t backward;
    DCT_CUDA_TRY(cudaMemcpyAsync(&backward, result_dev, sizeof(dct_result_t), cudaMemcpyDeviceToHost, stream));
    DCT_CUDA_TRY(cudaStreamSynchronize(stream));
    if (backward.status > result_host->status) result_host->status = backward.status;   // the worse of the two
    return static_cast<dct_status_t>(result_host->status);
}
