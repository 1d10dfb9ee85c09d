// dct_dp_compress: Algorithm 1 (DCT-DP) for a fixed threshold, in one streaming pass.
//
//   w = grad + residual           (error feedback)
//   M = I(|w| >= tau)             (mask; optional tie budget on |w| == tau)
//   (idx, val) of survivors       (compressed gradient, ascending index)
//   residual = w - w .* M         (error)
//
// The vector is cut into tiles of kTileElems consecutive elements.  Tiles are
// handed out by an atomic ticket, so a tile's predecessors have always been
// taken by a running CTA before it; the global output offset of a tile comes
// from a decoupled look-back over one 64-bit descriptor per tile (2 status bits
// + two 31-bit running counts: elements above tau and elements equal to tau).
//
// HBM traffic: read grad, read residual, write residual = 12 B per element,
// plus 8 B per survivor.  The residual of a tile is stored before its look-back
// finishes, assuming that every flagged element is sent; the rare elements that
// turn out not to be sent (capacity exceeded, tie budget used up, wait timed
// out) are rewritten afterwards.
//
// Two kernels share the per-tile arithmetic:
//   * dp_compress_stream_kernel -- the fast path for 16-byte aligned vectors.
//     Persistent CTAs with four roles.  A load warp takes tickets and streams
//     tiles into a ring of shared-memory stages with bulk asynchronous copies
//     (TMA engine, plain copies).  Eight compute warps threshold a stage, store
//     the new residual with 128-bit stores, publish the tile's counts and push
//     the tile's survivors, in index order, into a shared-memory ring that holds
//     a whole tile's worth of entries.  A look-back warp finds each tile's output
//     offset, starting from the tile the CTA resolved before it, and two drain
//     warps write the tile's ring entries to (idx, val).  Nothing on the compute warps'
//     path waits for another CTA, whatever the density of the survivors; they wait
//     for their own drain warps only when the ring or the slot table is full.
//   * dp_compress_tile_kernel -- one CTA per tile with plain loads and stores:
//     the ragged last tile and vectors that are not 16-byte aligned.
#include <mutex>
#include <vector>

#include "common.cuh"
#include "dp_chain.cuh"

namespace dct {
namespace {

constexpr int kThreads = 256;                           // compute threads per CTA
constexpr int kWarps = kThreads / 32;
constexpr int kVecs = 4;                                // 128-bit vectors per thread and operand
constexpr uint32_t kWarpElems = 32u * kVecs * 4u;       // 512
constexpr uint32_t kTileElems = kWarps * kWarpElems;    // 4096
constexpr uint32_t kTileBytes = kTileElems * 4u;        // 16 KiB per operand

constexpr int kStages = 2;                              // ring depth of the streaming kernel
constexpr uint32_t kInvalidTile = 0xFFFFFFFFu;
constexpr uint32_t kMbarLimit = 1u << 24;               // polls before an mbarrier wait gives up

constexpr uint64_t kStatusAggregate = 1ull << 62;       // descriptor holds the tile's own counts
constexpr uint64_t kStatusInclusive = 2ull << 62;       // descriptor holds counts of tiles 0..this
constexpr uint64_t kStatusMask = 3ull << 62;
constexpr uint64_t kCountMask = 0x7FFFFFFFull;

__device__ __forceinline__ uint64_t pack_counts(uint64_t status, uint32_t gt, uint32_t eq) {
    return status | (static_cast<uint64_t>(gt) << 31) | eq;
}
__device__ __forceinline__ uint32_t desc_gt(uint64_t d) { return static_cast<uint32_t>((d >> 31) & kCountMask); }
__device__ __forceinline__ uint32_t desc_eq(uint64_t d) { return static_cast<uint32_t>(d & kCountMask); }

struct CompressCtrl {
    uint32_t ticket;       // next tile to hand out
    uint32_t abort;        // a bounded wait gave up somewhere: everybody stops waiting
    uint32_t slow_ticket;  // batched calls: next work item of the tile kernel
};
constexpr size_t kCtrlBytes = 256;

__global__ void dp_compress_init_kernel(CompressCtrl* ctrl, uint64_t* tile_state, uint32_t num_tiles,
                                        dct_result_t* result, uint32_t first_ticket,
                                        const uint32_t* __restrict__ enabled = nullptr) {
    // the streaming kernel that follows may be scheduled already (it waits for this grid before it touches the
    // control block): its launch latency and set-up then overlap this kernel
    chain_release_next();
    // launched as a programmatic dependent itself: the kernel before it on the stream (say, the previous call's
    // streaming kernel, which still reads these descriptors) has to be finished before anything is reset
    chain_wait_previous();
    if (enabled && *enabled == 0) return;     // a conditional call that is not needed: nothing is touched
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

// Look-back by one warp: counts of all tiles before `tile`.  Each round examines a window of
// 32 * kLookWide descriptors (all loads of a round are in flight together, so a round costs one
// L2 round trip).  The walk ends at the nearest descriptor that holds an inclusive prefix, or at
// `anchor`: a tile whose inclusive counts the caller already knows (-1 and zeros: the empty prefix
// before tile 0).  A persistent CTA passes the tile it resolved last, about one grid width back,
// so its look-back needs only the other tiles' own counts, which their CTAs publish at once, and
// never waits for another CTA's look-back.  Every wait is bounded.
constexpr int kLookWide = 10;
struct LookAnchor {
    int64_t tile;
    uint32_t gt, eq;
};
__device__ __forceinline__ void lookback(const uint64_t* tile_state, const CompressCtrl* ctrl,
                                         uint32_t tile, uint32_t spin_limit, const LookAnchor& anchor,
                                         uint32_t& excl_gt, uint32_t& excl_eq, bool& timed_out) {
    const uint32_t lane = lane_id();
    uint32_t sum_gt = 0, sum_eq = 0;
    int64_t window_end = static_cast<int64_t>(tile);   // tiles [window_end - 32 kLookWide, window_end)
    timed_out = false;
    while (true) {
        uint64_t d[kLookWide];
#pragma unroll
        for (int q = 0; q < kLookWide; ++q) {            // distance from the tile: q * 32 + lane + 1
            const int64_t t = window_end - 1 - (q * 32 + static_cast<int64_t>(lane));
            d[q] = t > anchor.tile ? ld_relaxed_u64(tile_state + t)
                                   : pack_counts(kStatusInclusive, t == anchor.tile ? anchor.gt : 0u,
                                                 t == anchor.tile ? anchor.eq : 0u);
        }
        bool done = false;
#pragma unroll
        for (int q = 0; q < kLookWide; ++q) {
            if (done) break;
            const int64_t t = window_end - 1 - (q * 32 + static_cast<int64_t>(lane));
            uint32_t spins = 0;
            bool fail = false;
            while ((d[q] & kStatusMask) == 0) {          // not published yet: poll this descriptor
                if (spins >= spin_limit || ((spins & 31u) == 31u && ld_relaxed_u32(&ctrl->abort))) {
                    fail = true;
                    break;
                }
                ++spins;
                if (spins > 16) __nanosleep(spins > 256 ? 400 : 50);
                d[q] = ld_relaxed_u64(tile_state + t);
            }
            if (__any_sync(0xFFFFFFFFu, fail)) {
                timed_out = true;
                return;
            }
            const uint32_t inclusive = __ballot_sync(0xFFFFFFFFu, (d[q] & kStatusMask) == kStatusInclusive);
            // lanes 0..first (nearest tiles up to and including the first inclusive one) contribute
            const uint32_t first = inclusive ? (__ffs(inclusive) - 1) : 31u;
            const bool use = lane <= first;
            sum_gt += __reduce_add_sync(0xFFFFFFFFu, use ? desc_gt(d[q]) : 0u);
            sum_eq += __reduce_add_sync(0xFFFFFFFFu, use ? desc_eq(d[q]) : 0u);
            if (inclusive) done = true;
        }
        if (done) break;
        window_end -= 32 * kLookWide;
    }
    excl_gt = sum_gt;
    excl_eq = sum_eq;
}

// A tile's own counts, visible to every later tile as early as possible.
__device__ __forceinline__ void publish_tile_aggregate(uint64_t* tile_state, uint32_t tile, uint32_t cta_gt,
                                                       uint32_t cta_eq) {
    st_relaxed_u64(tile_state + tile, pack_counts(tile == 0 ? kStatusInclusive : kStatusAggregate, cta_gt, cta_eq));
}

// Publishes the tile's descriptors, runs the look-back and, for the last tile of the vector,
// writes the result block.  Called by one full warp.  Returns false if the wait gave up.
__device__ __forceinline__ bool resolve_tile_prefix(uint64_t* tile_state, CompressCtrl* ctrl, dct_result_t* result,
                                                    uint32_t tile, uint32_t last_tile, uint32_t cta_gt,
                                                    uint32_t cta_eq, uint64_t budget, uint64_t capacity,
                                                    uint32_t spin_limit, uint32_t& excl_gt, uint32_t& excl_eq,
                                                    bool publish_aggregate,
                                                    const LookAnchor& anchor = LookAnchor{-1, 0u, 0u}) {
    const uint32_t lane = lane_id();
    if (lane == 0 && publish_aggregate) publish_tile_aggregate(tile_state, tile, cta_gt, cta_eq);
    bool timed_out = false;
    excl_gt = 0;
    excl_eq = 0;
    if (tile > 0) lookback(tile_state, ctrl, tile, spin_limit, anchor, excl_gt, excl_eq, timed_out);
    if (timed_out) {
        if (lane == 0) {
            atomicExch(&ctrl->abort, 1u);
            atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
        }
        return false;
    }
    if (lane == 0) {
        if (tile > 0)
            st_relaxed_u64(tile_state + tile, pack_counts(kStatusInclusive, excl_gt + cta_gt, excl_eq + cta_eq));
        if (tile == last_tile) {
            const uint64_t total_gt = static_cast<uint64_t>(excl_gt) + cta_gt;
            const uint64_t total_eq = static_cast<uint64_t>(excl_eq) + cta_eq;
            const uint64_t needed = total_gt + (total_eq < budget ? total_eq : budget);
            result->needed = needed;
            result->count = needed < capacity ? needed : capacity;
            if (needed > capacity) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_CAPACITY));
        }
    }
    return true;
}

// Error feedback for 16 elements of one thread: element b = 4 j + c sits at
// warp_base + j * 128 + lane * 4 + c.  Returns the flag masks (bit b).
__device__ __forceinline__ void flag_elements(const float (&w)[kVecs * 4], uint32_t tau_key, uint32_t valid_mask,
                                              uint32_t& gt_mask, uint32_t& eq_mask) {
    gt_mask = 0;
    eq_mask = 0;
#pragma unroll
    for (int b = 0; b < kVecs * 4; ++b) {
        const uint32_t kw = key_f32(w[b]);
        gt_mask |= (kw > tau_key) ? (1u << b) : 0u;
        eq_mask |= (kw == tau_key) ? (1u << b) : 0u;
    }
    gt_mask &= valid_mask;
    eq_mask &= valid_mask;
}

// Visits the flagged elements of one warp's 512-element span in index order:
//   visit(b, i, local_gt, local_eq, is_eq)
// with b the register slot, i the element index and local_* the number of flagged elements of
// each kind that precede it inside the tile (before_warp: packed counts of the lower warps).
// Must be called by all 32 lanes of the warp.
template <typename Visit>
__device__ __forceinline__ void for_each_flagged(uint32_t gt_mask, uint32_t eq_mask, uint32_t warp_base,
                                                 uint32_t before_warp, Visit&& visit) {
    const uint32_t lane = lane_id();
    // Element order inside the span is (j, lane, c).  Per-j counts (<= 4 per lane, <= 128 per
    // warp) are packed one per byte so that one warp scan serves all four j.
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
    if ((gt_mask | eq_mask) == 0) return;
#pragma unroll
    for (int j = 0; j < kVecs; ++j) {
        uint32_t g0 = base_g + ((ex_g >> (8 * j)) & 0xFFu);
        uint32_t e0 = base_e + ((ex_e >> (8 * j)) & 0xFFu);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int b = 4 * j + c;
            const bool is_gt = (gt_mask >> b) & 1u, is_eq = (eq_mask >> b) & 1u;
            if (is_gt || is_eq) {
                visit(b, warp_base + j * 128 + lane * 4 + c, g0, e0, is_eq);
                g0 += is_gt;
                e0 += is_eq;
            }
        }
        base_g += (tot_g >> (8 * j)) & 0xFFu;
        base_e += (tot_e >> (8 * j)) & 0xFFu;
    }
}

// The same for a span without elements equal to tau (the usual case: one packed scan, no second kind to carry):
//   visit(b, j * 128 + c, local_gt)      with the element at warp_base + lane * 4 + j * 128 + c
template <typename Visit>
__device__ __forceinline__ void for_each_above(uint32_t gt_mask, uint32_t before, Visit&& visit) {
    const uint32_t lane = lane_id();
    uint32_t pg = 0;
#pragma unroll
    for (int j = 0; j < kVecs; ++j) pg |= static_cast<uint32_t>(__popc((gt_mask >> (4 * j)) & 0xFu)) << (8 * j);
    uint32_t ig = pg;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t tg = __shfl_up_sync(0xFFFFFFFFu, ig, o);
        if (lane >= static_cast<uint32_t>(o)) ig += tg;
    }
    const uint32_t tot_g = __shfl_sync(0xFFFFFFFFu, ig, 31);
    const uint32_t ex_g = ig - pg;
    if (gt_mask == 0) return;
    uint32_t base_g = before;
#pragma unroll
    for (int j = 0; j < kVecs; ++j) {
        uint32_t g0 = base_g + ((ex_g >> (8 * j)) & 0xFFu);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int b = 4 * j + c;
            if ((gt_mask >> b) & 1u) {
                visit(b, static_cast<uint32_t>(j * 128 + c), g0);
                ++g0;
            }
        }
        base_g += (tot_g >> (8 * j)) & 0xFFu;
    }
}

// One flagged element whose global counts of preceding flagged elements are known: it is either
// written to the output or, if it is not sent after all, put back into the residual.
__device__ __forceinline__ void place_survivor(uint32_t i, float w, bool is_eq, uint64_t gt_before,
                                               uint64_t eq_before, uint64_t budget, uint64_t capacity, bool aborted,
                                               int32_t* __restrict__ idx_out, float* __restrict__ val_out,
                                               float* __restrict__ residual) {
    const bool pass = !is_eq || eq_before < budget;
    const uint64_t pos = gt_before + (eq_before < budget ? eq_before : budget);
    if (pass && pos < capacity && !aborted) {
        idx_out[pos] = static_cast<int32_t>(i);
        val_out[pos] = w;
    } else {
        residual[i] = w;
    }
}

// Writes the survivors of one warp's span straight from registers.
__device__ __forceinline__ void emit_warp(const float (&w)[kVecs * 4], uint32_t gt_mask, uint32_t eq_mask,
                                          uint32_t warp_base, uint32_t before_warp, uint64_t excl_gt,
                                          uint64_t excl_eq, uint64_t budget, uint64_t capacity, bool aborted,
                                          int32_t* __restrict__ idx_out, float* __restrict__ val_out,
                                          float* __restrict__ residual) {
    for_each_flagged(gt_mask, eq_mask, warp_base, before_warp,
                     [&](int b, uint32_t i, uint32_t local_gt, uint32_t local_eq, bool is_eq) {
                         place_survivor(i, w[b], is_eq, excl_gt + local_gt, excl_eq + local_eq, budget, capacity,
                                        aborted, idx_out, val_out, residual);
                     });
}

// ------------------------------------------------------------------------------------------
// generic path: one CTA per tile, plain loads/stores, any alignment, ragged tail
// ------------------------------------------------------------------------------------------
constexpr int kTileKernelMinBlocks = 4;                 // CTAs of the tile kernel the register budget must allow per SM
// One tile, by one CTA, with plain loads and stores (every thread of the CTA calls this with the same tile).
template <bool kVectorised>
__device__ __forceinline__ void compress_tile_body(const float* __restrict__ grad, float* __restrict__ residual,
                                                   uint32_t n, const float* __restrict__ tau_p,
                                                   const uint64_t* __restrict__ budget_p,
                                                   int32_t* __restrict__ idx_out, float* __restrict__ val_out,
                                                   uint64_t capacity, dct_result_t* __restrict__ result,
                                                   CompressCtrl* ctrl, uint64_t* __restrict__ tile_state,
                                                   uint32_t num_tiles, uint32_t tile, uint32_t spin_limit,
                                                   uint32_t first_valid = 0) {
    // first_valid != 0: grad and residual point first_valid (1 to 3) elements BEFORE the vector, on the 16-byte boundary
    // below it, and n counts from there.  Those elements are read (they share the vector's first 16 bytes) but belong to
    // somebody else: never flagged, never written; the indices that go out count from the vector's own first element.
    __shared__ uint32_t s_warp_tot[kWarps];   // (gt << 16) | eq of each warp, each <= 512
    __shared__ uint32_t s_excl[2];
    __shared__ uint32_t s_abort;

    const uint32_t lane = lane_id();
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t tile_base = tile * kTileElems;
    const uint32_t warp_base = tile_base + warp * kWarpElems;
    const uint32_t tau_key = key_f32(__ldg(tau_p));
    const uint64_t budget = budget_p ? *budget_p : ~0ull;

    float w[kVecs * 4];
    uint32_t valid_mask = 0xFFFFu;
    const bool full_tile = kVectorised && (tile_base + kTileElems <= n) && tile_base >= first_valid;
    if (full_tile) {
        float4 g4[kVecs], e4[kVecs];
#pragma unroll
        for (int j = 0; j < kVecs; ++j)
            g4[j] = grad ? ld_readonly_f4(grad + warp_base + j * 128 + lane * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < kVecs; ++j) e4[j] = ld_stream_f4(residual + warp_base + j * 128 + lane * 4);
#pragma unroll
        for (int j = 0; j < kVecs; ++j) {
            // (no gradient: w is the stored value itself, bit for bit -- adding +0 would turn -0 into +0)
            w[4 * j + 0] = grad ? __fadd_rn(g4[j].x, e4[j].x) : e4[j].x;
            w[4 * j + 1] = grad ? __fadd_rn(g4[j].y, e4[j].y) : e4[j].y;
            w[4 * j + 2] = grad ? __fadd_rn(g4[j].z, e4[j].z) : e4[j].z;
            w[4 * j + 3] = grad ? __fadd_rn(g4[j].w, e4[j].w) : e4[j].w;
        }
    } else {
        valid_mask = 0;
#pragma unroll
        for (int b = 0; b < kVecs * 4; ++b) {
            const uint32_t i = warp_base + (b >> 2) * 128 + lane * 4 + (b & 3);
            const bool valid = i < n && i >= first_valid;
            w[b] = valid ? (grad ? __fadd_rn(grad[i], residual[i]) : residual[i]) : 0.0f;
            valid_mask |= valid ? (1u << b) : 0u;
        }
    }
    uint32_t gt_mask, eq_mask;
    flag_elements(w, tau_key, valid_mask, gt_mask, eq_mask);

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

    // residual: +0 where flagged, w elsewhere (flagged elements are rewritten later if not sent)
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
            if ((valid_mask >> b) & 1u) residual[i] = (flagged >> b) & 1u ? 0.0f : w[b];
        }
    }

    if (warp == 0) {
        uint32_t excl_gt, excl_eq;
        const bool ok = resolve_tile_prefix(tile_state, ctrl, result, tile, num_tiles - 1, cta_gt, cta_eq, budget,
                                            capacity, spin_limit, excl_gt, excl_eq, true);
        if (lane == 0) {
            s_abort = ok ? 0u : 1u;
            s_excl[0] = excl_gt;
            s_excl[1] = excl_eq;
        }
    }
    if (cta_tot != 0) {                        // (nothing flagged in this tile: no output, no rewrite)
        __syncthreads();
        if (warp_tot != 0)
            emit_warp(w, gt_mask, eq_mask, warp_base - first_valid, before_warp, s_excl[0], s_excl[1], budget, capacity,
                      s_abort != 0, idx_out, val_out, residual + first_valid);
    }
}

template <bool kVectorised>
__global__ void __launch_bounds__(kThreads, kTileKernelMinBlocks)
dp_compress_tile_kernel(const float* __restrict__ grad, float* __restrict__ residual, uint32_t n,
                        const float* __restrict__ tau_p, const uint64_t* __restrict__ budget_p,
                        int32_t* __restrict__ idx_out, float* __restrict__ val_out, uint64_t capacity,
                        dct_result_t* __restrict__ result, CompressCtrl* ctrl,
                        uint64_t* __restrict__ tile_state, uint32_t num_tiles, uint32_t fixed_tile,
                        uint32_t spin_limit, const uint32_t* __restrict__ enabled = nullptr, uint32_t first_valid = 0) {
    __shared__ uint32_t s_tile;
    if (enabled && *enabled == 0) return;     // a conditional call that is not needed
    // A CTA works through tickets until none is left (the grid need not be as large as the number of tiles).  Tiles
    // are only taken by running CTAs and in order, so the oldest unfinished tile never waits for one not yet taken.
    for (;;) {
        if (threadIdx.x == 0) s_tile = fixed_tile != kInvalidTile ? fixed_tile : atomicAdd(&ctrl->ticket, 1u);
        __syncthreads();
        const uint32_t tile = s_tile;
        if (tile >= num_tiles) return;
        compress_tile_body<kVectorised>(grad, residual, n, tau_p, budget_p, idx_out, val_out, capacity, result, ctrl,
                                        tile_state, num_tiles, tile, spin_limit, first_valid);
        if (fixed_tile != kInvalidTile) return;
        __syncthreads();                      // the tile's shared-memory words are free for the next one
    }
}

// ------------------------------------------------------------------------------------------
// fast path: persistent CTAs; load warp + compute warps + look-back warp + drain warps
// ------------------------------------------------------------------------------------------
constexpr int kSlots = 16;                               // tiles a CTA may be ahead of its drain warp
constexpr uint32_t kRingEntries = 6016;                  // survivors waiting in shared memory: any one tile fits
constexpr uint32_t kEqBit = 0x80000000u;                 // ring entry: "equal to tau"
constexpr uint32_t kAheadGrace = 8;                      // polls of a waiting compute warp before it counts tiles ahead
constexpr int kDrainWarps = 2;                           // warps that share the write-out of a tile's entries
constexpr int kLoadWarp = kWarps, kLookWarp = kWarps + 1, kDrainWarp0 = kWarps + 2;
constexpr int kStreamThreads = kThreads + 64 + 32 * kDrainWarps;
static_assert(kRingEntries >= kTileElems && kTileElems <= 4096, "a tile fits the ring; 12-bit fields");

struct __align__(128) StreamSmem {
    float g[kStages][kTileElems];
    float e[kStages][kTileElems];
    // survivors of the tiles that are not written out yet, in tile order and, inside a tile, index order:
    // x = offset inside the tile | (equal-to-tau elements of the tile before it) << 12 | kEqBit, y = value bits
    uint2 ring[kRingEntries];
    uint64_t full[kStages];              // load -> compute: stage holds a tile (bulk loads landed)
    uint64_t empty[kStages];             // compute -> load: stage may be refilled
    uint64_t agg_ready[kSlots];          // compute (thread 0) -> look-back: tile and counts of the slot are written
    uint64_t entries_ready[kSlots];      // compute (8 warps) -> drain: the tile's ring entries are written
    uint64_t prefix_ready[kSlots];       // look-back -> drain: exclusive prefix of the slot's tile is in prefix[]
    uint32_t tile[kStages];
    uint32_t layer[kStages];             // batched calls: which vector the stage's tile belongs to
    uint32_t warp_tot[2][kWarps];
    uint32_t slot_tile[kSlots];
    uint32_t slot_layer[kSlots];
    uint32_t slot_agg[kSlots];           // (gt << 16) | eq of the tile
    uint32_t slot_start[kSlots];         // ring position of the tile's first entry
    uint32_t slot_head[kSlots];          // running count of ring entries up to and including the tile's
    uint32_t prefix[kSlots][2];
    uint32_t aborted[kSlots];
    // batched calls: what the drain warps need to know about the slot's vector, from the look-back warp, which has
    // read the vector's description anyway
    int32_t* slot_idx_out[kSlots];
    float* slot_val_out[kSlots];
    float* slot_residual[kSlots];
    uint64_t slot_budget[kSlots];
    uint64_t slot_capacity[kSlots];
    uint32_t slot_bias[kSlots];
    uint32_t ahead[4];                   // counts of a tile taken ahead of its turn: eq | gt << 13 | warps that added << 26
    volatile uint32_t ring_tail[kDrainWarps];   // drain warp -> compute: running count of ring entries it is done with
    volatile uint32_t drained[kDrainWarps];     // drain warp -> compute: tiles it is done with (their slots may be reused)
    volatile uint32_t stop;              // a bounded wait gave up inside this CTA
};
// two CTAs per SM: the SM has 228 KiB, of which each CTA costs 1 KiB on top of what it asks for
static_assert(sizeof(StreamSmem) <= 113 * 1024, "two CTAs of the streaming kernel per SM");

// Bounded wait until a counter another warp advances has reached `target` (wrapping 32-bit counts).
__device__ __forceinline__ bool counter_wait_bounded(const volatile uint32_t* counter, uint32_t target, uint32_t limit,
                                                     const volatile uint32_t* stop) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (static_cast<int32_t>(*counter - target) >= 0) return true;
        if ((i & 63u) == 63u && *stop) return false;
        if (i >= 4) __nanosleep(100);          // leave the shared-memory pipe to the warps that are being waited for
    }
    return false;
}

// One vector of a call as the kernels see it (a batched call has a table of these in the workspace).
struct LayerDesc {
    const float* grad;
    float* residual;
    const float* tau;
    const uint64_t* tie_budget;
    int32_t* idx_out;
    float* val_out;
    dct_result_t* result;
    uint64_t capacity;
    uint32_t n;
    uint32_t first_desc;   // index of the vector's first tile descriptor
    uint32_t num_full;     // full tiles handled by the streaming kernel (0 for an unaligned vector)
    uint32_t num_tiles;    // all tiles, a ragged last one included
    uint32_t idx_bias;     // grad and residual point this many elements before the vector (see compress_tile_body)
};
struct BatchTable {
    const LayerDesc* layers;
    const uint32_t* full_prefix;   // [num_layers + 1] running count of streaming-kernel tiles
    const uint32_t* slow_prefix;   // [num_layers + 1] running count of tile-kernel tiles
    const uint32_t* head_layers;   // vectors whose first tile goes to the tile kernel ahead of the streaming kernel
    uint32_t num_layers;
};
// What a role needs to know about the vector it is working on, held in registers.
struct TileParams {
    const float* grad;
    float* residual;
    int32_t* idx_out;
    float* val_out;
    dct_result_t* result;
    uint64_t* tile_state;          // descriptors of this vector: look-back never leaves them
    uint64_t capacity, budget;
    uint32_t tau_key, last_tile, idx_bias;
};
__device__ __forceinline__ TileParams load_params(const LayerDesc& d, uint64_t* tile_state_base) {
    TileParams p;
    p.grad = d.grad;
    p.residual = d.residual;
    p.idx_out = d.idx_out;
    p.val_out = d.val_out;
    p.result = d.result;
    p.tile_state = tile_state_base + d.first_desc;
    p.capacity = d.capacity;
    p.budget = d.tie_budget ? *d.tie_budget : ~0ull;
    p.tau_key = key_f32(*d.tau);
    p.last_tile = d.num_tiles - 1;
    p.idx_bias = d.idx_bias;
    return p;
}

// kBatched == false: one vector, described by `single`, work items are its full tiles.
// kBatched == true : work items are the full tiles of all vectors of `batch`, in table order; a role
//                    reloads its TileParams whenever the vector changes under it.
template <bool kBatched>
__global__ void __launch_bounds__(kStreamThreads, 2)
dp_compress_stream_kernel(const LayerDesc single, const BatchTable batch, uint32_t total_work, CompressCtrl* ctrl,
                          uint64_t* __restrict__ tile_state_base, uint32_t spin_limit) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    StreamSmem& sm = *reinterpret_cast<StreamSmem*>(smem_raw);
    const uint32_t tid = threadIdx.x, lane = lane_id(), warp = tid >> 5;

    if (tid < static_cast<uint32_t>(kSlots)) {
        mbar_init(&sm.agg_ready[tid], 1);
        mbar_init(&sm.entries_ready[tid], kWarps);
        mbar_init(&sm.prefix_ready[tid], 1);
        if (tid < static_cast<uint32_t>(kStages)) {
            mbar_init(&sm.full[tid], 1);
            mbar_init(&sm.empty[tid], 1);
        }
        if (tid < static_cast<uint32_t>(kDrainWarps)) {
            sm.ring_tail[tid] = 0;
            sm.drained[tid] = 0;
        }
        if (tid < 4) sm.ahead[tid] = 0;
        if (tid == 0) sm.stop = 0;
        mbar_init_fence();
        fence_proxy_async_all();
    }
    __syncthreads();
    // launched as a programmatic dependent of the kernel that resets the control block: everything above ran
    // while that kernel was still at work, nothing below may (a no-op under an ordinary launch)
    chain_wait_previous();
    // The kernels after this one on the stream may be scheduled from here on: each of them waits for this grid to
    // finish before it touches anything, so all they gain is that their launch latency and set-up are behind them
    // when this grid ends (their CTAs take the places this grid's CTAs leave).
    chain_release_next();

    if (warp == kLoadWarp) {
        // ================= load warp (one lane): tickets and bulk loads ====================
        if (lane != 0) return;
        const float* grad = single.grad;
        const float* residual = single.residual;
        uint32_t cur_layer = 0, work_lo = 0, work_hi = total_work;     // work items of the current vector
        uint32_t first_full = 0;             // batched: the vector's first tile of this kernel (1 if its tile 0 is a head)
        if (kBatched) {
            work_hi = batch.full_prefix[1];
            grad = batch.layers[0].grad;
            residual = batch.layers[0].residual;
            first_full = batch.layers[0].idx_bias ? 1u : 0u;
        }
        uint32_t ticket = atomicAdd(&ctrl->ticket, 1u);
        for (uint32_t it = 0;; ++it) {
            const int s = it % kStages;
            uint32_t tile = ticket < total_work ? ticket : kInvalidTile;
            if (kBatched && tile != kInvalidTile) {
                if (tile >= work_hi) {
                    // Tickets only grow: the first later vector whose tiles reach beyond this one.  With large vectors it
                    // is the next one or two; with thousands of small ones a CTA's next ticket lies hundreds of vectors
                    // on, and stepping through them one dependent load at a time held the whole CTA up.  So: steps of
                    // 1, 2, 4, ... vectors (the first probes share a cache line), then bisection inside the last step.
                    const uint32_t last = batch.num_layers - 1;
                    uint32_t lo = cur_layer + 1, hi = lo, step = 1;
                    while (hi < last && batch.full_prefix[hi + 1] <= tile) {
                        lo = hi + 1;
                        hi = last - hi > step ? hi + step : last;
                        step <<= 1;
                    }
                    while (lo < hi) {
                        const uint32_t mid = (lo + hi) >> 1;
                        if (batch.full_prefix[mid + 1] > tile) hi = mid; else lo = mid + 1;
                    }
                    cur_layer = lo;
                    work_lo = batch.full_prefix[lo];
                    work_hi = batch.full_prefix[lo + 1];
                    grad = batch.layers[cur_layer].grad;
                    residual = batch.layers[cur_layer].residual;
                    first_full = batch.layers[cur_layer].idx_bias ? 1u : 0u;
                }
                tile = tile - work_lo + first_full;                    // tile index inside its vector
            }
            // the next ticket is requested now; its latency overlaps the wait below
            if (tile != kInvalidTile) ticket = atomicAdd(&ctrl->ticket, 1u);
            if (it >= static_cast<uint32_t>(kStages) &&
                !mbar_wait_bounded(&sm.empty[s], ((it / kStages) - 1u) & 1u, kMbarLimit, &sm.stop)) {
                sm.stop = 1;
                return;
            }
            sm.tile[s] = tile;
            sm.layer[s] = cur_layer;
            if (tile == kInvalidTile) {
                mbar_arrive(&sm.full[s]);
                return;
            }
            mbar_arrive_expect_tx(&sm.full[s], 2u * kTileBytes);
            bulk_load(sm.g[s], grad + static_cast<size_t>(tile) * kTileElems, kTileBytes, &sm.full[s]);
            bulk_load(sm.e[s], residual + static_cast<size_t>(tile) * kTileElems, kTileBytes, &sm.full[s]);
        }
    }

    if (warp == kLookWarp) {
        // ================= look-back warp: the exclusive prefix of each tile, in the CTA's tile order ==========
        TileParams P;
        uint32_t cur_layer = 0xFFFFFFFFu;
        if (!kBatched) P = load_params(single, tile_state_base);
        LookAnchor anchor{-1, 0u, 0u};        // the tile this warp resolved last (same vector), with its inclusive counts
        bool chain_ok = true;                 // false once a look-back of this CTA gave up: nothing later is sent
        for (uint32_t it = 0;; ++it) {
            const int r = it % kSlots;
            const uint32_t parity = (it / kSlots) & 1u;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&sm.agg_ready[r], parity, kMbarLimit, &sm.stop))) {
                sm.stop = 1;
                return;
            }
            const uint32_t tile = sm.slot_tile[r];
            if (tile == kInvalidTile) {
                if (lane == 0) mbar_arrive(&sm.prefix_ready[r]);
                return;
            }
            if (kBatched && sm.slot_layer[r] != cur_layer) {
                cur_layer = sm.slot_layer[r];
                P = load_params(batch.layers[cur_layer], tile_state_base);
                anchor = LookAnchor{-1, 0u, 0u};
            }
            const uint32_t tot = sm.slot_agg[r];
            const uint32_t cta_gt = tot >> 16, cta_eq = tot & 0xFFFFu;
            uint32_t excl_gt = 0, excl_eq = 0;
            chain_ok = chain_ok && resolve_tile_prefix(P.tile_state, ctrl, P.result, tile, P.last_tile, cta_gt, cta_eq,
                                                       P.budget, P.capacity, spin_limit, excl_gt, excl_eq, false, anchor);
            anchor = LookAnchor{static_cast<int64_t>(tile), excl_gt + cta_gt, excl_eq + cta_eq};
            if (lane == 0) {
                sm.prefix[r][0] = excl_gt;
                sm.prefix[r][1] = excl_eq;
                sm.aborted[r] = chain_ok ? 0u : 1u;
                if (kBatched) {
                    sm.slot_idx_out[r] = P.idx_out;
                    sm.slot_val_out[r] = P.val_out;
                    sm.slot_residual[r] = P.residual + P.idx_bias;        // (the vector's own first element)
                    sm.slot_budget[r] = P.budget;
                    sm.slot_capacity[r] = P.capacity;
                    sm.slot_bias[r] = P.idx_bias;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.prefix_ready[r]);
        }
    }

    if (warp >= kDrainWarp0) {
        // ================= drain warps: ring entries of each tile -> (idx, val), 32 entries per warp in turn =====
        const uint32_t dw = warp - kDrainWarp0;
        TileParams P;
        if (!kBatched) P = load_params(single, tile_state_base);
        for (uint32_t it = 0;; ++it) {
            const int r = it % kSlots;
            const uint32_t parity = (it / kSlots) & 1u;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&sm.prefix_ready[r], parity, kMbarLimit, &sm.stop))) {
                sm.stop = 1;
                return;
            }
            const uint32_t tile = sm.slot_tile[r];
            if (tile == kInvalidTile) return;
            if (kBatched) {
                P.idx_out = sm.slot_idx_out[r];
                P.val_out = sm.slot_val_out[r];
                P.residual = sm.slot_residual[r];
                P.budget = sm.slot_budget[r];
                P.capacity = sm.slot_capacity[r];
                P.idx_bias = sm.slot_bias[r];
            }
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&sm.entries_ready[r], parity, kMbarLimit, &sm.stop))) {
                sm.stop = 1;
                return;
            }
            const uint32_t tot = sm.slot_agg[r];
            const uint32_t cnt = (tot >> 16) + (tot & 0xFFFFu);
            const uint32_t start = sm.slot_start[r];
            const uint64_t excl_gt = sm.prefix[r][0], excl_eq = sm.prefix[r][1];
            const bool aborted = sm.aborted[r] != 0;
            // (indices count from the vector's own first element; the residual pointer moves with them)
            const uint32_t tile_base = tile * kTileElems - P.idx_bias;
            float* const residual_own = kBatched ? P.residual : P.residual + P.idx_bias;   // (batched: moved already)
#pragma unroll 4
            for (uint32_t q = dw * 32u + lane; q < cnt; q += 32u * kDrainWarps) {
                const uint32_t at = start + q;
                const uint2 ent = sm.ring[at < kRingEntries ? at : at - kRingEntries];
                const uint32_t local_eq = (ent.x >> 12) & 0xFFFu;
                place_survivor(tile_base + (ent.x & 0xFFFu), __uint_as_float(ent.y), (ent.x & kEqBit) != 0,
                               excl_gt + (q - local_eq), excl_eq + local_eq, P.budget, P.capacity, aborted, P.idx_out,
                               P.val_out, residual_own);
            }
            __syncwarp();                      // every lane has read its entries: the compute warps may overwrite them
            if (lane == 0) {
                sm.ring_tail[dw] = sm.slot_head[r];
                __threadfence_block();
                sm.drained[dw] = it + 1u;
            }
        }
    }

    // ===================== compute warps =================================================
    TileParams P;
    uint32_t cur_layer = 0xFFFFFFFFu;
    if (!kBatched) P = load_params(single, tile_state_base);
    bool healthy = true;
    uint32_t it = 0;
    uint32_t ring_head = 0;                   // running count of ring entries written by this CTA
    uint32_t ring_pos = 0;                    // the same modulo the size of the ring
    uint32_t ahead_upto = 0;                  // last iteration whose tile this warp has counted ahead of its turn
    uint32_t drained_seen = 0, tail_seen = 0; // what this warp last read of the drain warps' counters (they only grow)
    for (;; ++it) {
        const int s = it % kStages;
        const int r = it % kSlots;
        if (!named_barrier_all(1, kThreads,
                               mbar_wait_bounded(&sm.full[s], (it / kStages) & 1u, kMbarLimit, &sm.stop) &&
                                   !sm.stop)) {
            healthy = false;
            break;
        }
        const uint32_t tile = sm.tile[s];
        if (tile == kInvalidTile) break;
        if (kBatched && sm.layer[s] != cur_layer) {
            cur_layer = sm.layer[s];
            P = load_params(batch.layers[cur_layer], tile_state_base);
        }
        const uint32_t warp_base = tile * kTileElems + warp * kWarpElems;

        float w[kVecs * 4];
        {
            const float4* gs = reinterpret_cast<const float4*>(sm.g[s]) + warp * (kWarpElems / 4) + lane;
            const float4* es = reinterpret_cast<const float4*>(sm.e[s]) + warp * (kWarpElems / 4) + lane;
#pragma unroll
            for (int j = 0; j < kVecs; ++j) {
                const float4 g4 = gs[j * 32], e4 = es[j * 32];
                w[4 * j + 0] = __fadd_rn(g4.x, e4.x);
                w[4 * j + 1] = __fadd_rn(g4.y, e4.y);
                w[4 * j + 2] = __fadd_rn(g4.z, e4.z);
                w[4 * j + 3] = __fadd_rn(g4.w, e4.w);
            }
        }
        uint32_t gt_mask, eq_mask;
        flag_elements(w, P.tau_key, 0xFFFFu, gt_mask, eq_mask);
        const uint32_t flagged = gt_mask | eq_mask;
#pragma unroll
        for (int j = 0; j < kVecs; ++j) {
            float4 e;
            e.x = (flagged >> (4 * j + 0)) & 1u ? 0.0f : w[4 * j + 0];
            e.y = (flagged >> (4 * j + 1)) & 1u ? 0.0f : w[4 * j + 1];
            e.z = (flagged >> (4 * j + 2)) & 1u ? 0.0f : w[4 * j + 2];
            e.w = (flagged >> (4 * j + 3)) & 1u ? 0.0f : w[4 * j + 3];
            st_stream_f4(P.residual + warp_base + j * 128 + lane * 4, e);
        }
        const uint32_t warp_tot =
            __reduce_add_sync(0xFFFFFFFFu, (static_cast<uint32_t>(__popc(gt_mask)) << 16) | __popc(eq_mask));
        if (lane == 0) sm.warp_tot[it & 1u][warp] = warp_tot;
        named_barrier_sync(1, kThreads);          // every warp has read the stage and posted its counts
        uint32_t cta_tot = 0, before_warp = 0;
#pragma unroll
        for (int v = 0; v < kWarps; ++v) {
            const uint32_t t = sm.warp_tot[it & 1u][v];
            cta_tot += t;
            before_warp += (v < static_cast<int>(warp)) ? t : 0u;
        }
        const uint32_t cta_gt = cta_tot >> 16, cta_eq = cta_tot & 0xFFFFu;
        const uint32_t cnt = cta_gt + cta_eq;
        if (tid == 0) {
            mbar_arrive(&sm.empty[s]);
            // later tiles need these counts right now; the look-back warp adds the prefix when it gets here
            publish_tile_aggregate(P.tile_state, tile, cta_gt, cta_eq);
            sm.ahead[it & 3u] = 0;                // (whatever was counted ahead for this tile has served)
        }
        // The slot must have been drained (it normally was, long ago); the look-back may start as soon as the slot
        // holds the tile's counts, it does not need the ring entries.
        bool slot_ok = true;
        if (warp == 0) {
            const uint32_t need_drained = it + 1u - kSlots;
            if (static_cast<int32_t>(drained_seen - need_drained) < 0) {     // (else: seen to be free earlier)
                int32_t lead = 0x7FFFFFFF;
                if (lane < kDrainWarps) {         // one lane per drain warp
                    slot_ok = counter_wait_bounded(&sm.drained[lane], need_drained, kMbarLimit, &sm.stop);
                    lead = static_cast<int32_t>(sm.drained[lane] - need_drained);
                }
                slot_ok = __all_sync(0xFFFFFFFFu, slot_ok);
                drained_seen = need_drained + static_cast<uint32_t>(__reduce_min_sync(0xFFFFFFFFu, lead));
            }
            if (lane == 0 && slot_ok) {
                sm.slot_tile[r] = tile;
                sm.slot_layer[r] = cur_layer;
                sm.slot_agg[r] = cta_tot;
                sm.slot_start[r] = ring_pos;
                sm.slot_head[r] = ring_head + cnt;
                mbar_arrive(&sm.agg_ready[r]);
            }
        }
        // the tile's share of the ring must have been drained as well
        const uint32_t need_tail = ring_head + cnt - kRingEntries;
        auto least_tail = [&]() -> uint32_t {     // the least of the drain warps' counts (one lane per drain warp)
            const int32_t lead = lane < kDrainWarps ? static_cast<int32_t>(sm.ring_tail[lane] - need_tail) : 0x7FFFFFFF;
            return need_tail + static_cast<uint32_t>(__reduce_min_sync(0xFFFFFFFFu, lead));
        };
        bool room = static_cast<int32_t>(tail_seen - need_tail) >= 0;     // (seen to be free earlier)
        if (!room) {
            tail_seen = least_tail();
            room = static_cast<int32_t>(tail_seen - need_tail) >= 0;
        }
        if (!room) {
            // This warp has to wait for the drain warps, they for the look-back, and the look-back for the counts of
            // every earlier tile.  The CTA has taken tickets for the tiles in its other stages already; if their counts
            // came only after this wait, the CTAs behind those tiles would stop as well, each of them holding tickets
            // of its own, and the whole grid would advance one tile after the other.  So the warp first counts its span
            // of the tiles the CTA has taken and the last warp to do so publishes their counts.
            // (Only after a short while: most waits end by themselves before that.)
            uint32_t a = 1;
            for (uint32_t polls = 1;; ++polls) {
                tail_seen = least_tail();
                room = static_cast<int32_t>(tail_seen - need_tail) >= 0;
                if (room || polls >= kMbarLimit || ((polls & 63u) == 63u && sm.stop)) break;
                const uint32_t j = it + a;
                if (polls < kAheadGrace || a > static_cast<uint32_t>(kStages)) {
                    __nanosleep(100);          // leave the shared-memory pipe to the warps that are being waited for
                    continue;
                }
                ++a;
                if (j <= ahead_upto) continue;
                const int sa = j % kStages;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&sm.full[sa], (j / kStages) & 1u, kMbarLimit, &sm.stop)))
                    break;
                const uint32_t tile_a = sm.tile[sa];
                if (tile_a == kInvalidTile) {
                    a = kStages + 1;           // nothing follows
                    continue;
                }
                uint32_t tau_key_a = P.tau_key;
                uint64_t* tile_state_a = P.tile_state;
                if (kBatched && sm.layer[sa] != cur_layer) {
                    const LayerDesc& d = batch.layers[sm.layer[sa]];
                    tau_key_a = key_f32(*d.tau);
                    tile_state_a = tile_state_base + d.first_desc;
                }
                const float4* gs = reinterpret_cast<const float4*>(sm.g[sa]) + warp * (kWarpElems / 4) + lane;
                const float4* es = reinterpret_cast<const float4*>(sm.e[sa]) + warp * (kWarpElems / 4) + lane;
                uint32_t mine = 0;
#pragma unroll
                for (int v = 0; v < kVecs; ++v) {
                    const float4 g4 = gs[v * 32], e4 = es[v * 32];
                    const float wa[4] = {__fadd_rn(g4.x, e4.x), __fadd_rn(g4.y, e4.y), __fadd_rn(g4.z, e4.z),
                                         __fadd_rn(g4.w, e4.w)};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t kw = key_f32(wa[c]);
                        mine += (kw > tau_key_a ? (1u << 13) : 0u) + (kw == tau_key_a ? 1u : 0u);
                    }
                }
                mine = __reduce_add_sync(0xFFFFFFFFu, mine);
                if (lane == 0) {
                    const uint32_t all = atomicAdd(&sm.ahead[j & 3u], mine + (1u << 26)) + mine + (1u << 26);
                    if ((all >> 26) == static_cast<uint32_t>(kWarps))
                        publish_tile_aggregate(tile_state_a, tile_a, (all >> 13) & 0x1FFFu, all & 0x1FFFu);
                }
                ahead_upto = j;
            }
        }
        room = room && slot_ok;
        if (!room) sm.stop = 1;                   // seen by everybody at the next vote
        if (warp_tot != 0 && room && cta_eq == 0) {
            // no element of the tile equals tau (the usual case): one kind of entry, nothing to count before it
            const uint32_t first_off = warp * kWarpElems + lane * 4u;
            if (ring_pos + cnt <= kRingEntries) {
                uint2* ring = sm.ring + ring_pos;
                for_each_above(gt_mask, before_warp >> 16, [&](int b, uint32_t off, uint32_t local_gt) {
                    ring[local_gt] = make_uint2(first_off + off, __float_as_uint(w[b]));
                });
            } else {
                for_each_above(gt_mask, before_warp >> 16, [&](int b, uint32_t off, uint32_t local_gt) {
                    const uint32_t at = ring_pos + local_gt;
                    sm.ring[at < kRingEntries ? at : at - kRingEntries] = make_uint2(first_off + off, __float_as_uint(w[b]));
                });
            }
        } else if (warp_tot != 0 && room) {
            const uint32_t in_tile = warp * kWarpElems;
            for_each_flagged(gt_mask, eq_mask, in_tile, before_warp,
                             [&](int b, uint32_t off, uint32_t local_gt, uint32_t local_eq, bool is_eq) {
                                 const uint32_t at = ring_pos + local_gt + local_eq;
                                 sm.ring[at < kRingEntries ? at : at - kRingEntries] =
                                     make_uint2(off | (local_eq << 12) | (is_eq ? kEqBit : 0u), __float_as_uint(w[b]));
                             });
        }
        ring_head += cnt;
        ring_pos += cnt;
        ring_pos -= ring_pos >= kRingEntries ? kRingEntries : 0u;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.entries_ready[r]);
    }
    if (healthy) {
        // tell the other two warps that no more tiles follow
        const int r = it % kSlots;
        if (warp == 0) {
            bool slot_ok = true;
            if (lane < kDrainWarps)
                slot_ok = counter_wait_bounded(&sm.drained[lane], it + 1u - kSlots, kMbarLimit, &sm.stop);
            slot_ok = __all_sync(0xFFFFFFFFu, slot_ok);
            if (lane == 0 && slot_ok) {
                sm.slot_tile[r] = kInvalidTile;
                mbar_arrive(&sm.agg_ready[r]);
            }
        }
    } else if (tid == 0) {
        sm.stop = 1;
        atomicExch(&ctrl->abort, 1u);
        const LayerDesc& where = kBatched ? batch.layers[cur_layer < batch.num_layers ? cur_layer : 0] : single;
        atomicMax(&where.result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
    }
}

// ---- batched calls: many vectors (the layers of a model), one set of launches ------------------------
__global__ void dp_compress_batched_init_kernel(CompressCtrl* ctrl, uint64_t* tile_state, uint32_t total_tiles,
                                                const LayerDesc* layers, uint32_t num_layers) {
    chain_release_next();     // the streaming kernel may be scheduled; it waits for this grid (see dp_compress_init_kernel)
    const uint32_t stride = gridDim.x * blockDim.x;
    const uint32_t i0 = blockIdx.x * blockDim.x + threadIdx.x;
    for (uint32_t i = i0; i < total_tiles; i += stride) tile_state[i] = 0;
    for (uint32_t l = i0; l < num_layers; l += stride) {
        dct_result_t* r = layers[l].result;
        r->status = DCT_OK;
        r->reserved = 0;
        r->count = 0;
        r->needed = 0;
        r->n_gt = 0;
        r->n_eq = 0;
    }
    if (i0 == 0) {
        ctrl->ticket = 0;
        ctrl->abort = 0;
        ctrl->slow_ticket = 0;
    }
}

// The tiles the streaming kernel does not take: the ragged last tile of every aligned vector and all the
// tiles of vectors that are not 16-byte aligned.  Work items are handed out in table order by a ticket,
// so inside an unaligned vector a tile's predecessors have always been taken before it.
__global__ void __launch_bounds__(kThreads, kTileKernelMinBlocks)
dp_compress_tile_batched_kernel(const BatchTable batch, uint32_t total_slow, CompressCtrl* ctrl,
                                uint64_t* __restrict__ tile_state_base, uint32_t spin_limit) {
    __shared__ uint32_t s_work;
    if (threadIdx.x == 0) s_work = atomicAdd(&ctrl->slow_ticket, 1u);
    __syncthreads();
    const uint32_t work = s_work;
    if (work >= total_slow) return;
    uint32_t lo = 0, hi = batch.num_layers;            // the vector l with slow_prefix[l] <= work < slow_prefix[l + 1]
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (batch.slow_prefix[mid] <= work) lo = mid; else hi = mid;
    }
    const LayerDesc& d = batch.layers[lo];
    // an aligned vector contributes only its last tile; an unaligned one all of them
    const uint32_t tile = d.num_full + (work - batch.slow_prefix[lo]);
    compress_tile_body<false>(d.grad, d.residual, d.n, d.tau, d.tie_budget, d.idx_out, d.val_out, d.capacity,
                              d.result, ctrl, tile_state_base + d.first_desc, d.num_tiles, tile, spin_limit, d.idx_bias);
}

// The first tiles of the vectors that are worked on from the 16-byte boundary below them (LayerDesc::idx_bias != 0):
// they hold elements that are not the vector's, so the tile kernel's per-element path takes them -- before the streaming
// kernel, whose tiles of these vectors wait for their counts.  One CTA per such vector.
__global__ void __launch_bounds__(kThreads, kTileKernelMinBlocks)
dp_compress_heads_batched_kernel(const BatchTable batch, CompressCtrl* ctrl, uint64_t* __restrict__ tile_state_base,
                                 uint32_t spin_limit) {
    const LayerDesc& d = batch.layers[batch.head_layers[blockIdx.x]];
    compress_tile_body<false>(d.grad, d.residual, d.n, d.tau, d.tie_budget, d.idx_out, d.val_out, d.capacity,
                              d.result, ctrl, tile_state_base + d.first_desc, d.num_tiles, 0u, spin_limit, d.idx_bias);
}

}  // namespace

uint32_t dp_compress_num_tiles(uint64_t n) { return static_cast<uint32_t>((n + kTileElems - 1) / kTileElems); }

}  // namespace dct

using namespace dct;

extern "C" size_t dct_dp_compress_workspace_bytes(uint64_t n) {
    if (n == 0 || n > 0x7FFFFFFFull) return 0;
    // (+ 3: a vector that starts 4, 8 or 12 bytes past a 16-byte boundary is worked on from that boundary)
    const size_t bytes = kCtrlBytes + sizeof(uint64_t) * static_cast<size_t>(dp_compress_num_tiles(n + 3));
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
    // A gradient and a residual that sit the same 4, 8 or 12 bytes past a 16-byte boundary (views at the same offset
    // into two flat buffers) are worked on from that boundary: the `lead` elements before them lie in the same 16 bytes
    // of the same allocation, are read and never written, and the fast kernel's 16-byte accesses apply to all tiles but
    // the first.  (Any other misalignment: one CTA per tile with plain loads, about a quarter of the rate.)
    uint32_t lead = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(grad) & 15u) / 4u);
    if (lead != (reinterpret_cast<uintptr_t>(residual) & 15u) / 4u || n + lead > 0x7FFFFFFFull) lead = 0;
    grad -= lead;
    residual -= lead;
    const uint32_t n32 = static_cast<uint32_t>(n) + lead;
    const uint32_t num_tiles = dp_compress_num_tiles(n32);
    const uint32_t num_full = n32 / kTileElems;
    const uint32_t first_full = lead ? 1u : 0u;       // the first tile holds elements that are not the vector's
    const DebugConfig& dbg = debug_config();

    DCT_CUDA_TRY(launch_chained(dp_compress_init_kernel, (num_tiles + 1023) / 1024, 1024, stream, ctrl, tile_state, num_tiles,
                                result, dbg.first_ticket > first_full ? dbg.first_ticket : first_full,
                                static_cast<const uint32_t*>(nullptr)));
    const bool vec = aligned_to(grad, 16) && aligned_to(residual, 16);
    if (!vec) {
        const int sms_t = sm_count();
        if (sms_t <= 0) return DCT_ERR_CUDA;
        const uint32_t tile_grid = num_tiles < static_cast<uint32_t>(sms_t) * 8u ? num_tiles : static_cast<uint32_t>(sms_t) * 8u;
        dp_compress_tile_kernel<false><<<tile_grid, kThreads, 0, stream>>>(
            grad, residual, n32, tau, tie_budget, idx_out, val_out, capacity, result, ctrl, tile_state, num_tiles,
            kInvalidTile, dbg.spin_limit);
        DCT_CUDA_TRY(cudaGetLastError());
        return DCT_OK;
    }
    if (lead && num_full > 0) {   // the first tile, before the kernel whose tiles wait for its counts
        dp_compress_tile_kernel<true><<<1, kThreads, 0, stream>>>(
            grad, residual, n32, tau, tie_budget, idx_out, val_out, capacity, result, ctrl, tile_state, num_tiles, 0u,
            dbg.spin_limit, static_cast<const uint32_t*>(nullptr), lead);
        DCT_CUDA_TRY(cudaGetLastError());
    }
    if (num_full > first_full) {
        static thread_local int configured_device = -1;
        int dev = 0;
        DCT_CUDA_TRY(cudaGetDevice(&dev));
        if (configured_device != dev) {
            DCT_CUDA_TRY(cudaFuncSetAttribute(dp_compress_stream_kernel<false>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              static_cast<int>(sizeof(StreamSmem))));
            configured_device = dev;
        }
        const int sms = sm_count();
        if (sms <= 0) return DCT_ERR_CUDA;
        const uint32_t ctas_per_sm = 2;
        const uint32_t max_grid = static_cast<uint32_t>(sms) * ctas_per_sm;
        const uint32_t grid = num_full - first_full < max_grid ? num_full - first_full : max_grid;
        LayerDesc single{};
        single.grad = grad;
        single.residual = residual;
        single.tau = tau;
        single.tie_budget = tie_budget;
        single.idx_out = idx_out;
        single.val_out = val_out;
        single.result = result;
        single.capacity = capacity;
        single.n = n32;
        single.first_desc = 0;
        single.num_full = num_full;
        single.num_tiles = num_tiles;
        single.idx_bias = lead;
        DCT_CUDA_TRY(launch_chained_smem(dp_compress_stream_kernel<false>, grid, kStreamThreads, sizeof(StreamSmem), stream,
                                         single, BatchTable{}, num_full, ctrl, tile_state, dbg.spin_limit));
    }
    if (num_tiles > num_full) {   // ragged last tile
        dp_compress_tile_kernel<true><<<1, kThreads, 0, stream>>>(
            grad, residual, n32, tau, tie_budget, idx_out, val_out, capacity, result, ctrl, tile_state, num_tiles,
            num_full, dbg.spin_limit, static_cast<const uint32_t*>(nullptr), lead);
        DCT_CUDA_TRY(cudaGetLastError());
    }
    return DCT_OK;
}

// Algorithm 1, mask / compressed gradient / error steps on a vector that is already summed (w = g + e lies in
// `residual`), enqueued unconditionally but run only if *enabled != 0: the plain way of dct_dp_select_compress when
// its sample has misjudged the vector.  One CTA per tile with plain loads (the rare path need not be the fast one).
dct_status_t dct::compress_presummed_if(const uint32_t* enabled, float* residual, uint64_t n, const float* tau,
                                        const uint64_t* tie_budget, int32_t* idx_out, float* val_out, uint64_t capacity,
                                        dct_result_t* result, void* workspace, size_t workspace_bytes,
                                        cudaStream_t stream) {
    if (!workspace || !aligned_to(workspace, 256) || workspace_bytes < dct_dp_compress_workspace_bytes(n))
        return DCT_ERR_WORKSPACE;
    auto* ctrl = static_cast<CompressCtrl*>(workspace);
    auto* tile_state = reinterpret_cast<uint64_t*>(static_cast<char*>(workspace) + kCtrlBytes);
    const uint32_t n32 = static_cast<uint32_t>(n);
    const uint32_t num_tiles = dp_compress_num_tiles(n);
    const DebugConfig& dbg = debug_config();
    dp_compress_init_kernel<<<(num_tiles + 1023) / 1024, 1024, 0, stream>>>(ctrl, tile_state, num_tiles, result, 0u,
                                                                            enabled);
    DCT_CUDA_TRY(cudaGetLastError());
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint32_t tile_grid = num_tiles < static_cast<uint32_t>(sms) * 8u ? num_tiles : static_cast<uint32_t>(sms) * 8u;
    if (aligned_to(residual, 16))
        dp_compress_tile_kernel<true><<<tile_grid, kThreads, 0, stream>>>(
            nullptr, residual, n32, tau, tie_budget, idx_out, val_out, capacity, result, ctrl, tile_state, num_tiles,
            kInvalidTile, dbg.spin_limit, enabled);
    else
        dp_compress_tile_kernel<false><<<tile_grid, kThreads, 0, stream>>>(
            nullptr, residual, n32, tau, tie_budget, idx_out, val_out, capacity, result, ctrl, tile_state, num_tiles,
            kInvalidTile, dbg.spin_limit, enabled);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

// ------------------------------------------------------------------------------------------
// dct_dp_compress_batched: the layers of a model in one set of launches
// ------------------------------------------------------------------------------------------
namespace {

struct BatchLayout {
    size_t layers_off, full_off, slow_off, head_off, state_off, bytes;
    uint64_t total_tiles;
};
BatchLayout batch_layout(const uint64_t* n, uint32_t num_layers) {
    BatchLayout L{};
    uint64_t tiles = 0;
    // (+ 3: a vector that starts 4, 8 or 12 bytes past a 16-byte boundary is worked on from that boundary)
    for (uint32_t l = 0; l < num_layers; ++l) tiles += dp_compress_num_tiles(n[l] + 3);
    L.total_tiles = tiles;
    size_t off = kCtrlBytes;
    L.layers_off = off;
    off += sizeof(LayerDesc) * num_layers;
    off = (off + 15) & ~static_cast<size_t>(15);
    L.full_off = off;
    off += sizeof(uint32_t) * (num_layers + 1);
    L.slow_off = off;
    off += sizeof(uint32_t) * (num_layers + 1);
    L.head_off = off;
    off += sizeof(uint32_t) * num_layers;
    off = (off + 255) & ~static_cast<size_t>(255);
    L.state_off = off;
    off += sizeof(uint64_t) * tiles;
    L.bytes = (off + 255) & ~static_cast<size_t>(255);
    return L;
}

}  // namespace

extern "C" size_t dct_dp_compress_batched_workspace_bytes(const uint64_t* n, uint32_t num_layers) {
    if (!n || num_layers == 0) return 0;
    for (uint32_t l = 0; l < num_layers; ++l)
        if (n[l] == 0 || n[l] > 0x7FFFFFFFull) return 0;
    const BatchLayout L = batch_layout(n, num_layers);
    return L.total_tiles > 0xFFFFFFFFull ? 0 : L.bytes;
}

extern "C" dct_status_t dct_dp_compress_batched(const dct_dp_layer_t* layers, uint32_t num_layers, void* workspace,
                                                size_t workspace_bytes, dct_stream_t stream_) {
    if (!layers || num_layers == 0) return DCT_ERR_INVALID_ARG;
    if (stream_is_capturing(static_cast<cudaStream_t>(stream_))) return DCT_ERR_UNSUPPORTED;   // uploads a temporary table
    std::vector<uint64_t> sizes(num_layers);
    for (uint32_t l = 0; l < num_layers; ++l) {
        const dct_dp_layer_t& a = layers[l];
        if (!a.grad || !a.residual || !a.tau || !a.result || a.n == 0 || a.n > 0x7FFFFFFFull) return DCT_ERR_INVALID_ARG;
        if (a.capacity > 0 && (!a.idx_out || !a.val_out)) return DCT_ERR_INVALID_ARG;
        if (!aligned_to(a.grad, 4) || !aligned_to(a.residual, 4) || !aligned_to(a.tau, 4) || !aligned_to(a.result, 8) ||
            (a.tie_budget && !aligned_to(a.tie_budget, 8)) || !aligned_to(a.idx_out, 4) || !aligned_to(a.val_out, 4))
            return DCT_ERR_INVALID_ARG;
        const uintptr_t g0 = reinterpret_cast<uintptr_t>(a.grad), e0 = reinterpret_cast<uintptr_t>(a.residual);
        const uintptr_t bytes = static_cast<uintptr_t>(a.n) * 4;
        if (g0 < e0 + bytes && e0 < g0 + bytes) return DCT_ERR_INVALID_ARG;
        sizes[l] = a.n;
    }
    const BatchLayout L = batch_layout(sizes.data(), num_layers);
    if (L.total_tiles > 0xFFFFFFFFull) return DCT_ERR_UNSUPPORTED;
    if (!workspace || !aligned_to(workspace, 256) || workspace_bytes < L.bytes) return DCT_ERR_WORKSPACE;

    // the table the kernels read: descriptors of all vectors, and the two running work counts
    std::vector<unsigned char> table(L.state_off - L.layers_off);
    auto* descs = reinterpret_cast<LayerDesc*>(table.data());
    auto* full_prefix = reinterpret_cast<uint32_t*>(table.data() + (L.full_off - L.layers_off));
    auto* slow_prefix = reinterpret_cast<uint32_t*>(table.data() + (L.slow_off - L.layers_off));
    auto* head_layers = reinterpret_cast<uint32_t*>(table.data() + (L.head_off - L.layers_off));
    uint32_t first_desc = 0, total_full = 0, total_slow = 0, num_heads = 0;
    for (uint32_t l = 0; l < num_layers; ++l) {
        const dct_dp_layer_t& a = layers[l];
        LayerDesc& d = descs[l];
        // a gradient and a residual the same 4, 8 or 12 bytes past a 16-byte boundary (the usual state of a layer
        // inside two flat buffers) are worked on from that boundary: see dct_dp_compress
        uint32_t lead = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(a.grad) & 15u) / 4u);
        if (lead != (reinterpret_cast<uintptr_t>(a.residual) & 15u) / 4u || a.n + lead > 0x7FFFFFFFull) lead = 0;
        const uint32_t n32 = static_cast<uint32_t>(a.n) + lead;
        const bool vec = aligned_to(a.grad - lead, 16) && aligned_to(a.residual - lead, 16);
        d.grad = a.grad - lead;
        d.residual = a.residual - lead;
        d.idx_bias = lead;
        d.tau = a.tau;
        d.tie_budget = a.tie_budget;
        d.idx_out = a.idx_out;
        d.val_out = a.val_out;
        d.result = a.result;
        d.capacity = a.capacity;
        d.n = n32;
        d.first_desc = first_desc;
        d.num_tiles = dp_compress_num_tiles(n32);
        d.num_full = vec ? n32 / kTileElems : 0;
        // the first tile of a vector with leading elements goes to the tile kernel ahead of the streaming kernel
        const uint32_t head = lead && d.num_full > 0 ? 1u : 0u;
        if (head) head_layers[num_heads++] = l;
        full_prefix[l] = total_full;
        slow_prefix[l] = total_slow;
        total_full += d.num_full - head;
        total_slow += d.num_tiles - d.num_full;
        first_desc += d.num_tiles;
    }
    full_prefix[num_layers] = total_full;
    slow_prefix[num_layers] = total_slow;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    char* ws = static_cast<char*>(workspace);
    auto* ctrl = reinterpret_cast<CompressCtrl*>(ws);
    auto* tile_state = reinterpret_cast<uint64_t*>(ws + L.state_off);
    // pageable source: the runtime has staged the bytes by the time this returns, so `table` may go away
    DCT_CUDA_TRY(cudaMemcpyAsync(ws + L.layers_off, table.data(), table.size(), cudaMemcpyHostToDevice, stream));
    BatchTable batch;
    batch.layers = reinterpret_cast<const LayerDesc*>(ws + L.layers_off);
    batch.full_prefix = reinterpret_cast<const uint32_t*>(ws + L.full_off);
    batch.slow_prefix = reinterpret_cast<const uint32_t*>(ws + L.slow_off);
    batch.head_layers = reinterpret_cast<const uint32_t*>(ws + L.head_off);
    batch.num_layers = num_layers;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const DebugConfig& dbg = debug_config();
    {
        const uint64_t items = L.total_tiles > num_layers ? L.total_tiles : num_layers;
        const uint64_t blocks = (items + 1023) / 1024;
        const unsigned grid = static_cast<unsigned>(blocks < static_cast<uint64_t>(sms) * 4 ? blocks : sms * 4);
        dp_compress_batched_init_kernel<<<grid, 1024, 0, stream>>>(ctrl, tile_state,
                                                                   static_cast<uint32_t>(L.total_tiles), batch.layers,
                                                                   num_layers);
        DCT_CUDA_TRY(cudaGetLastError());
    }
    if (num_heads > 0) {
        dp_compress_heads_batched_kernel<<<num_heads, kThreads, 0, stream>>>(batch, ctrl, tile_state, dbg.spin_limit);
        DCT_CUDA_TRY(cudaGetLastError());
    }
    if (total_full > 0) {
        static thread_local int configured_device = -1;
        int dev = 0;
        DCT_CUDA_TRY(cudaGetDevice(&dev));
        if (configured_device != dev) {
            DCT_CUDA_TRY(cudaFuncSetAttribute(dp_compress_stream_kernel<true>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              static_cast<int>(sizeof(StreamSmem))));
            configured_device = dev;
        }
        const uint32_t ctas_per_sm = 2;
        const uint32_t max_grid = static_cast<uint32_t>(sms) * ctas_per_sm;
        const uint32_t grid = total_full < max_grid ? total_full : max_grid;
        DCT_CUDA_TRY(launch_chained_smem(dp_compress_stream_kernel<true>, grid, kStreamThreads, sizeof(StreamSmem), stream,
                                         LayerDesc{}, batch, total_full, ctrl, tile_state, dbg.spin_limit));
    }
    if (total_slow > 0) {
        dp_compress_tile_batched_kernel<<<total_slow, kThreads, 0, stream>>>(batch, total_slow, ctrl, tile_state,
                                                                           dbg.spin_limit);
        DCT_CUDA_TRY(cudaGetLastError());
    }
    return DCT_OK;
}

// ------------------------------------------------------------------------------------------
// dct_dp_compress_static: the same operator for callers that cannot hand over a workspace
// ------------------------------------------------------------------------------------------
// The tile descriptors and the ticket live in this file-scope device array instead of a caller
// buffer.  Every GPU that loads the library carries these 256.5 KiB until the process exits.
// In host code the array's name is only a stand-in: the device address is fetched once per device
// with cudaGetSymbolAddress (that device being current) and handed to the kernels like any workspace.
namespace {

constexpr uint64_t kStaticMaxElems = DCT_DP_COMPRESS_STATIC_MAX_N;
// (one descriptor more than whole tiles: a vector that starts past a 16-byte boundary is worked on from that boundary)
constexpr size_t kStaticScratchBytes = (kCtrlBytes + sizeof(uint64_t) * (kStaticMaxElems / kTileElems + 1) + 255) / 256 * 256;
static_assert(kStaticMaxElems % kTileElems == 0, "the static scratch is sized in whole tiles");

static __device__ __align__(256) unsigned char dct_static_scratch[kStaticScratchBytes];

// Device address of dct_static_scratch on the current device, looked up on first use.
cudaError_t static_scratch_address(void** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void* address[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (address[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, dct_static_scratch);   // resolves the symbol in the current device's copy
        if (e != cudaSuccess) return e;
        address[dev] = p;
    }
    *out = address[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" dct_status_t dct_dp_compress_static(const float* grad, float* residual, uint64_t n, const float* tau,
                                               const uint64_t* tie_budget, int32_t* idx_out, float* val_out,
                                               uint64_t capacity, dct_result_t* result, dct_stream_t stream) {
    if (n == 0) return DCT_ERR_INVALID_ARG;
    if (n > kStaticMaxElems) return DCT_ERR_UNSUPPORTED;   // the built-in scratch only covers DCT_DP_COMPRESS_STATIC_MAX_N
    void* scratch = nullptr;
    DCT_CUDA_TRY(static_scratch_address(&scratch));
    // dct_dp_compress resets the ticket and every descriptor it is going to use before the main
    // kernel runs, so whatever the previous call left in the array does not matter.
    return dct_dp_compress(grad, residual, n, tau, tie_budget, idx_out, val_out, capacity, result, scratch,
                           kStaticScratchBytes, stream);
}
