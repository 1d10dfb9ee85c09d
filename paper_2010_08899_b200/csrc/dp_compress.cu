// dct_dp_compress: Algorithm 1 (DCT-DP) for a fixed threshold, in one streaming pass.
//
//   w = grad + residual           (error feedback)
//   M = I(|w| >= tau)             (mask; optional tie budget on |w| == tau)
//   (idx, val) of survivors       (compressed gradient, ascending index)
//   residual = w - w .* M         (error)
//
// One CTA handles one tile of kTileElems consecutive elements.  Tiles are
// handed out by an atomic ticket, so a tile's predecessors have always started
// before it; the global output offset of a tile comes from a decoupled
// look-back over one 64-bit descriptor per tile (2 status bits + two 31-bit
// running counts: elements above tau and elements equal to tau).
//
// HBM traffic: read grad, read residual, write residual = 12 B per element,
// plus 8 B per survivor.  The residual is stored before the look-back finishes
// (assuming every flagged element is sent); the rare elements that turn out not
// to be sent (capacity exceeded, tie budget used up, wait timed out) are
// rewritten afterwards by the same thread.
#include "common.cuh"

namespace dct {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kVecs = 4;                                // 128-bit loads per thread and operand
constexpr uint32_t kWarpElems = 32u * kVecs * 4u;       // 512
constexpr uint32_t kTileElems = kWarps * kWarpElems;    // 4096

constexpr uint64_t kStatusAggregate = 1ull << 62;       // descriptor holds the tile's own counts
constexpr uint64_t kStatusInclusive = 2ull << 62;       // descriptor holds counts of tiles 0..this
constexpr uint64_t kStatusMask = 3ull << 62;
constexpr uint64_t kCountMask = 0x7FFFFFFFull;

__device__ __forceinline__ uint64_t pack_counts(uint64_t status, uint32_t gt, uint32_t eq) {
    return status | (static_cast<uint64_t>(gt) << 31) | eq;
}
__device__ __forceinline__ uint32_t desc_gt(uint64_t d) { return static_cast<uint32_t>((d >> 31) & kCountMask); }
__device__ __forceinline__ uint32_t desc_eq(uint64_t d) { return static_cast<uint32_t>(d & kCountMask); }

// ctrl[0] = next tile ticket, ctrl[1] = abort flag (a wait gave up somewhere)
struct CompressCtrl {
    uint32_t ticket;
    uint32_t abort;
};
constexpr size_t kCtrlBytes = 256;

__global__ void dp_compress_init_kernel(CompressCtrl* ctrl, uint64_t* tile_state, uint32_t num_tiles,
                                        dct_result_t* result, uint32_t first_ticket) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < num_tiles) tile_state[i] = 0;
    if (i == 0) {
        ctrl->ticket = first_ticket;
        ctrl->abort = 0;
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }
}

// Look-back by one warp: returns the counts of all tiles before `tile`.
// Every wait is bounded; on expiry *timed_out is set and the result is unusable.
__device__ __forceinline__ void lookback(const uint64_t* tile_state, const CompressCtrl* ctrl,
                                         uint32_t tile, uint32_t spin_limit,
                                         uint32_t& excl_gt, uint32_t& excl_eq, bool& timed_out) {
    const uint32_t lane = lane_id();
    uint32_t sum_gt = 0, sum_eq = 0;
    bool fail = false;
    int64_t window_end = static_cast<int64_t>(tile);   // tiles [window_end-32, window_end) are examined
    while (true) {
        const int64_t t = window_end - 1 - lane;
        uint64_t d = kStatusInclusive;                   // tiles before the first one: empty prefix
        if (t >= 0) {
            uint32_t spins = 0;
            while (true) {
                d = ld_relaxed_u64(tile_state + t);
                if (d & kStatusMask) break;
                if (spins >= spin_limit || ((spins & 31u) == 31u && ld_relaxed_u32(&ctrl->abort))) {
                    fail = true;
                    break;
                }
                ++spins;
                if (spins > 16) __nanosleep(spins > 256 ? 400 : 50);
            }
        }
        if (__any_sync(0xFFFFFFFFu, fail)) {
            timed_out = true;
            return;
        }
        const uint32_t inclusive = __ballot_sync(0xFFFFFFFFu, (d & kStatusMask) == kStatusInclusive);
        // lanes 0..first (nearest tiles up to and including the first inclusive one) contribute
        const uint32_t first = inclusive ? (__ffs(inclusive) - 1) : 31u;
        const bool use = lane <= first;
        sum_gt += __reduce_add_sync(0xFFFFFFFFu, use ? desc_gt(d) : 0u);
        sum_eq += __reduce_add_sync(0xFFFFFFFFu, use ? desc_eq(d) : 0u);
        if (inclusive) break;
        window_end -= 32;
    }
    excl_gt = sum_gt;
    excl_eq = sum_eq;
    timed_out = false;
}

template <bool kVectorised>
__global__ void __launch_bounds__(kThreads)
dp_compress_kernel(const float* __restrict__ grad, float* __restrict__ residual, uint32_t n,
                   const float* __restrict__ tau_p, const uint64_t* __restrict__ budget_p,
                   int32_t* __restrict__ idx_out, float* __restrict__ val_out, uint64_t capacity,
                   dct_result_t* __restrict__ result, CompressCtrl* ctrl,
                   uint64_t* __restrict__ tile_state, uint32_t num_tiles, uint32_t spin_limit) {
    __shared__ uint32_t s_tile;
    __shared__ uint32_t s_warp_tot[kWarps];   // (gt << 16) | eq of each warp, each <= 512
    __shared__ uint32_t s_excl[2];
    __shared__ uint32_t s_abort;

    if (threadIdx.x == 0) {
        s_tile = atomicAdd(&ctrl->ticket, 1u);
        s_abort = 0;
    }
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= num_tiles) return;            // only reachable with a testing ticket offset

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t tile_base = tile * kTileElems;
    const uint32_t warp_base = tile_base + warp * kWarpElems;
    const uint32_t tau_key = key_f32(__ldg(tau_p));
    const uint64_t budget = budget_p ? *budget_p : ~0ull;

    // ---- load, error feedback, flags --------------------------------------------------
    float w[kVecs * 4];
    const bool full_tile = kVectorised && (tile_base + kTileElems <= n);
    if (full_tile) {
        float4 g4[kVecs], e4[kVecs];
#pragma unroll
        for (int j = 0; j < kVecs; ++j) g4[j] = ld_readonly_f4(grad + warp_base + j * 128 + lane * 4);
#pragma unroll
        for (int j = 0; j < kVecs; ++j) e4[j] = ld_stream_f4(residual + warp_base + j * 128 + lane * 4);
#pragma unroll
        for (int j = 0; j < kVecs; ++j) {
            w[4 * j + 0] = __fadd_rn(g4[j].x, e4[j].x);
            w[4 * j + 1] = __fadd_rn(g4[j].y, e4[j].y);
            w[4 * j + 2] = __fadd_rn(g4[j].z, e4[j].z);
            w[4 * j + 3] = __fadd_rn(g4[j].w, e4[j].w);
        }
    } else {
#pragma unroll
        for (int j = 0; j < kVecs; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t i = warp_base + j * 128 + lane * 4 + c;
                w[4 * j + c] = (i < n) ? __fadd_rn(grad[i], residual[i]) : 0.0f;
            }
    }

    uint32_t gt_mask = 0, eq_mask = 0;        // bit 4*j + c
#pragma unroll
    for (int b = 0; b < kVecs * 4; ++b) {
        const uint32_t i = warp_base + (b >> 2) * 128 + lane * 4 + (b & 3);
        const bool valid = full_tile || (i < n);
        const uint32_t kw = key_f32(w[b]);
        gt_mask |= (valid && kw > tau_key) ? (1u << b) : 0u;
        eq_mask |= (valid && kw == tau_key) ? (1u << b) : 0u;
    }

    // ---- tile aggregate, published as early as possible ---------------------------------
    const uint32_t warp_tot =
        __reduce_add_sync(0xFFFFFFFFu, (static_cast<uint32_t>(__popc(gt_mask)) << 16) | __popc(eq_mask));
    if (lane == 0) s_warp_tot[warp] = warp_tot;
    __syncthreads();
    uint32_t cta_tot = 0, before_warp = 0;
#pragma unroll
    for (int v = 0; v < kWarps; ++v) {
        const uint32_t t = s_warp_tot[v];
        cta_tot += t;
        before_warp += (v < static_cast<int>(warp)) ? t : 0u;
    }
    const uint32_t cta_gt = cta_tot >> 16, cta_eq = cta_tot & 0xFFFFu;
    if (threadIdx.x == 0)
        st_relaxed_u64(tile_state + tile,
                       pack_counts(tile == 0 ? kStatusInclusive : kStatusAggregate, cta_gt, cta_eq));

    // ---- residual: +0 where flagged, w elsewhere ----------------------------------------
    const uint32_t flagged = gt_mask | eq_mask;
    if (full_tile) {
#pragma unroll
        for (int j = 0; j < kVecs; ++j) {
            float4 e;
            e.x = (flagged >> (4 * j + 0)) & 1u ? 0.0f : w[4 * j + 0];
            e.y = (flagged >> (4 * j + 1)) & 1u ? 0.0f : w[4 * j + 1];
            e.z = (flagged >> (4 * j + 2)) & 1u ? 0.0f : w[4 * j + 2];
            e.w = (flagged >> (4 * j + 3)) & 1u ? 0.0f : w[4 * j + 3];
            st_stream_f4(residual + warp_base + j * 128 + lane * 4, e);
        }
    } else {
#pragma unroll
        for (int b = 0; b < kVecs * 4; ++b) {
            const uint32_t i = warp_base + (b >> 2) * 128 + lane * 4 + (b & 3);
            if (i < n) residual[i] = (flagged >> b) & 1u ? 0.0f : w[b];
        }
    }

    // ---- look-back for the exclusive prefix (warp 0) --------------------------------------
    if (warp == 0) {
        uint32_t excl_gt = 0, excl_eq = 0;
        bool timed_out = false;
        if (tile > 0) lookback(tile_state, ctrl, tile, spin_limit, excl_gt, excl_eq, timed_out);
        if (lane == 0) {
            if (timed_out) {
                atomicExch(&ctrl->abort, 1u);
                atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
                s_abort = 1;
            } else {
                if (tile > 0)
                    st_relaxed_u64(tile_state + tile,
                                   pack_counts(kStatusInclusive, excl_gt + cta_gt, excl_eq + cta_eq));
                s_excl[0] = excl_gt;
                s_excl[1] = excl_eq;
                if (tile == num_tiles - 1) {
                    const uint64_t total_gt = static_cast<uint64_t>(excl_gt) + cta_gt;
                    const uint64_t total_eq = static_cast<uint64_t>(excl_eq) + cta_eq;
                    const uint64_t needed = total_gt + (total_eq < budget ? total_eq : budget);
                    result->needed = needed;
                    result->count = needed < capacity ? needed : capacity;
                    if (needed > capacity) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_CAPACITY));
                }
            }
        }
    }
    if (cta_tot == 0) return;                  // nothing flagged in this tile: no output, no fix-up
    __syncthreads();
    if (warp_tot == 0) return;
    const bool aborted = s_abort != 0;
    const uint64_t excl_gt = s_excl[0], excl_eq = s_excl[1];

    // ---- positions of this warp's flagged elements -------------------------------------------
    // Element order inside a warp's 512-element span is (j, lane, c).  Per-j counts (<= 4 per
    // lane, <= 128 per warp) are packed one per byte so that one warp scan serves all four j.
    uint32_t pg = 0, pe = 0;
#pragma unroll
    for (int j = 0; j < kVecs; ++j) {
        pg |= static_cast<uint32_t>(__popc((gt_mask >> (4 * j)) & 0xFu)) << (8 * j);
        pe |= static_cast<uint32_t>(__popc((eq_mask >> (4 * j)) & 0xFu)) << (8 * j);
    }
    uint32_t ig = pg, ie = pe;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t tg = __shfl_up_sync(0xFFFFFFFFu, ig, o);
        const uint32_t te = __shfl_up_sync(0xFFFFFFFFu, ie, o);
        if (lane >= static_cast<uint32_t>(o)) {
            ig += tg;
            ie += te;
        }
    }
    const uint32_t tot_g = __shfl_sync(0xFFFFFFFFu, ig, 31), tot_e = __shfl_sync(0xFFFFFFFFu, ie, 31);
    const uint32_t ex_g = ig - pg, ex_e = ie - pe;
    uint32_t base_g = before_warp >> 16, base_e = before_warp & 0xFFFFu;
    if (flagged) {
#pragma unroll
        for (int j = 0; j < kVecs; ++j) {
            uint32_t g0 = base_g + ((ex_g >> (8 * j)) & 0xFFu);
            uint32_t e0 = base_e + ((ex_e >> (8 * j)) & 0xFFu);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int b = 4 * j + c;
                const bool is_gt = (gt_mask >> b) & 1u, is_eq = (eq_mask >> b) & 1u;
                if (is_gt || is_eq) {
                    const uint64_t gt_before = excl_gt + g0;
                    const uint64_t eq_before = excl_eq + e0;
                    const bool pass = is_gt || eq_before < budget;
                    const uint64_t pos = gt_before + (eq_before < budget ? eq_before : budget);
                    const uint32_t i = warp_base + j * 128 + lane * 4 + c;
                    if (pass && pos < capacity && !aborted) {
                        idx_out[pos] = static_cast<int32_t>(i);
                        val_out[pos] = w[b];
                    } else {
                        residual[i] = w[b];    // not sent after all: it stays in the error
                    }
                    g0 += is_gt;
                    e0 += is_eq;
                }
            }
            base_g += (tot_g >> (8 * j)) & 0xFFu;
            base_e += (tot_e >> (8 * j)) & 0xFFu;
        }
    }
}

}  // namespace

uint32_t dp_compress_num_tiles(uint64_t n) { return static_cast<uint32_t>((n + kTileElems - 1) / kTileElems); }

}  // namespace dct

using namespace dct;

extern "C" size_t dct_dp_compress_workspace_bytes(uint64_t n) {
    if (n == 0 || n > 0x7FFFFFFFull) return 0;
    const size_t bytes = kCtrlBytes + sizeof(uint64_t) * static_cast<size_t>(dp_compress_num_tiles(n));
    return (bytes + 255) & ~static_cast<size_t>(255);
}

extern "C" dct_status_t dct_dp_compress(const float* grad, float* residual, uint64_t n,
                                        const float* tau, const uint64_t* tie_budget,
                                        int32_t* idx_out, float* val_out, uint64_t capacity,
                                        dct_result_t* result, void* workspace, size_t workspace_bytes,
                                        dct_stream_t stream_) {
    if (!grad || !residual || !tau || !result || n == 0 || n > 0x7FFFFFFFull) return DCT_ERR_INVALID_ARG;
    if (capacity > 0 && (!idx_out || !val_out)) return DCT_ERR_INVALID_ARG;
    if (!aligned_to(grad, 4) || !aligned_to(residual, 4) || !aligned_to(tau, 4) ||
        !aligned_to(result, 8) || (tie_budget && !aligned_to(tie_budget, 8)) ||
        !aligned_to(idx_out, 4) || !aligned_to(val_out, 4))
        return DCT_ERR_INVALID_ARG;
    {   // grad must not overlap residual (residual is rewritten while grad is read)
        const uintptr_t g0 = reinterpret_cast<uintptr_t>(grad), e0 = reinterpret_cast<uintptr_t>(residual);
        const uintptr_t bytes = static_cast<uintptr_t>(n) * 4;
        if (g0 < e0 + bytes && e0 < g0 + bytes) return DCT_ERR_INVALID_ARG;
    }
    if (!workspace || !aligned_to(workspace, 256) || workspace_bytes < dct_dp_compress_workspace_bytes(n))
        return DCT_ERR_WORKSPACE;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    auto* ctrl = static_cast<CompressCtrl*>(workspace);
    auto* tile_state = reinterpret_cast<uint64_t*>(static_cast<char*>(workspace) + kCtrlBytes);
    const uint32_t num_tiles = dp_compress_num_tiles(n);
    const DebugConfig& dbg = debug_config();

    dp_compress_init_kernel<<<(num_tiles + 1023) / 1024, 1024, 0, stream>>>(ctrl, tile_state, num_tiles, result,
                                                                            dbg.first_ticket);
    DCT_CUDA_TRY(cudaGetLastError());
    const bool vec = aligned_to(grad, 16) && aligned_to(residual, 16);
    if (vec)
        dp_compress_kernel<true><<<num_tiles, kThreads, 0, stream>>>(
            grad, residual, static_cast<uint32_t>(n), tau, tie_budget, idx_out, val_out, capacity, result, ctrl,
            tile_state, num_tiles, dbg.spin_limit);
    else
        dp_compress_kernel<false><<<num_tiles, kThreads, 0, stream>>>(
            grad, residual, static_cast<uint32_t>(n), tau, tie_budget, idx_out, val_out, capacity, result, ctrl,
            tile_state, num_tiles, dbg.spin_limit);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}
