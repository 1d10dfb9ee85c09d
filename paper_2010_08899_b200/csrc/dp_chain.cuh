// Internal pieces that dct_dp_select_compress (threshold life-span L = 1 of Algorithm 1) borrows from the
// select and compress translation units.  Nothing here is exported from the library.
#pragma once
#include "common.cuh"

namespace dct {

// Device-side state of one L = 1 call, at the start of its workspace.
struct L1Block {
    dct_result_t cand_result;   // result block of the compress pass that extracts the candidates
    dct_result_t scratch;       // result block the sample select writes into (its counts are not used)
    uint64_t tie_budget;        // k - n_gt once the exact threshold is known
    uint64_t n_gt, n_eq;        // of the exact threshold
    float lo;                   // the sampled lower bound of the threshold
    uint32_t use_candidates;    // 1: the candidate list holds every element >= tau (the normal case)
    uint32_t fallback;          // 1: the sample misjudged the vector; the plain way runs on w = g + e
    uint32_t cand_count;        // candidates in the list
};

// threshold_select.cu ------------------------------------------------------------------------------------
// Would the sampled bound be used for (n, k) with room for `cand_capacity` candidates?
bool l1_sampled_path_applies(uint64_t n, uint64_t k, uint64_t cand_capacity);
// Resets the select workspace and enqueues the radix select over the sector-wise sample of fl32(grad + residual);
// block->lo receives a value with, almost surely, between k and cand_capacity elements at or above it.
dct_status_t l1_sample_bound(const float* grad, const float* residual, uint64_t n, uint64_t k, uint64_t cand_capacity,
                             L1Block* block, void* select_ws, cudaStream_t stream);
// After the compress pass with block->lo (candidates in cand_idx / cand_val, count in block->cand_result, residual
// = w with the candidates zeroed): decides whether the list is usable; if not, writes the candidates back into the
// residual (which then holds w everywhere); then the exact select over the candidates, or over w; tau_out,
// block->n_gt / n_eq / tie_budget are written either way.
dct_status_t l1_exact_threshold(const int32_t* cand_idx, const float* cand_val, uint64_t cand_capacity, float* residual,
                                uint64_t n, uint64_t k, float* tau_out, L1Block* block, void* select_ws,
                                cudaStream_t stream);

// dp_compress.cu -------------------------------------------------------------------------------------------
// dct_dp_compress on a vector w that is already summed (w lies in `residual`, there is no gradient to add), run
// only if *enabled != 0 on the device (every kernel returns at once otherwise, and `result` is left alone).
dct_status_t compress_presummed_if(const uint32_t* enabled, float* residual, uint64_t n, const float* tau,
                                   const uint64_t* tie_budget, int32_t* idx_out, float* val_out, uint64_t capacity,
                                   dct_result_t* result, void* workspace, size_t workspace_bytes, cudaStream_t stream);

}  // namespace dct
