// dct_mp_topk_pack_fwd, rows of up to 512 bf16 or 256 fp32 columns: Algorithm 2 (DCT-MP) with the row held in
// registers and several samples per warp.  Two schemes:
//   * the count over the row in registers (narrow_slow_path, narrow_bisect_f32): tau_i bit by bit, every round a
//     count of the row's keys against a trial value by the G lanes that hold the row, then the ordered emit.  It
//     serves every k on bf16 rows of up to 128 columns and fp32 rows of up to 256, the denser k (more than an eighth
//     of the row) on bf16 rows of up to 256 columns, and the rows the second scheme gives up on;
//   * bound and candidates (mp_topk_fwd_bf16_narrow_kernel, bf16 rows of 129 to 512 columns, k up to an eighth of
//     the row), described next.
//
// For narrow rows the fixed cost per row of the shared-memory kernel (mp_pack.cu: bulk copy, barrier, bit
// table, bisection, linked walk) outweighs the work on the row itself, and so do the warp scans and votes
// when a whole warp serves one short row.  Here a row belongs to a group of G lanes (G = 8 or 16, so a
// warp works on 4 or 2 rows at once, every scan and vote serving all of them; G = 32 works too but is
// no faster than the shared-memory kernel and is not used); lane l of the group
// loads its E consecutive columns (E <= 32: at most four 16-byte loads) straight into registers, and the
// next rows are fetched while the current ones are worked on.  The candidate bits of a lane are one
// register word in column order, so one segmented scan ranks every candidate.  Steps per row:
//   A  bound: the previous row's tau_i minus a margin; if that leaves fewer than k or too many candidates,
//      the exact bound (the k-th largest maximum of the aligned 8-element leaves, found bit by bit) -- the
//      row is still in registers, so trying again costs no memory traffic.
//   B  candidates (key >= bound, ~1.3 k of them) go, in column order, to the group's list in shared memory;
//      their values are re-read from the row in global memory, which the loads above left in L1.
//   C  the list is dealt out evenly, at most 5 candidates to a lane; tau_i comes from a 64-bin histogram
//      just above the bound (else bit by bit over the candidates), and the ordered emit is that of the
//      wide kernel.
// Decisions that change the control flow (bound rejected, window missed, candidates do not fit) are taken
// for the warp as a whole, so all its lanes stay together; the slow path works on the rows in global memory.
#include "common.cuh"
#include "mp_warp.cuh"

namespace dct {
namespace {

constexpr int kNarrowWarps = 16;                 // warps per CTA
constexpr uint32_t kNarrowPerLaneFew = 5;        // candidates a lane holds in registers (8 for the denser k)
constexpr uint32_t kNarrowScratchWords = 320;    // per warp (G >= 8); a group's share holds its list / histogram / stage
// G = 4 (8 rows per warp): 8 shares of 64 + G words for the histogram
template <int G> __host__ __device__ constexpr uint32_t narrow_scratch_words() { return G >= 8 ? kNarrowScratchWords : (32u / G) * (64u + G); }

#pragma nv_diag_suppress 177   // (members that one instantiation or another does not use)
template <int G, int PLN = static_cast<int>(kNarrowPerLaneFew)> struct Group {
    static constexpr uint32_t kRows = 32u / G;                       // rows a warp works on at once
    static constexpr uint32_t kList = PLN * G;                       // candidates of a row that fit
    static constexpr uint32_t kShare = narrow_scratch_words<G>() / kRows;  // scratch words of one group: >= 64 + G, >= kList
    static constexpr uint32_t kBins = 64u / G;                       // window bins a lane looks after
    static_assert(kShare >= 64u + G && kShare >= kList, "scratch share too small");

    __device__ static __forceinline__ uint32_t inclusive_sum(uint32_t v, uint32_t gl) {
#pragma unroll
        for (int o = 1; o < G; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, v, o, G);
            if (gl >= static_cast<uint32_t>(o)) v += t;
        }
        return v;
    }
    __device__ static __forceinline__ uint32_t last(uint32_t v) { return __shfl_sync(0xFFFFFFFFu, v, G - 1, G); }
    __device__ static __forceinline__ uint32_t from(uint32_t v, uint32_t src) { return __shfl_sync(0xFFFFFFFFu, v, src, G); }
    __device__ static __forceinline__ uint32_t sum(uint32_t v) {
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o, G);
        return v;
    }
    // votes of the group's lanes, bit i = lane i of the group
    __device__ static __forceinline__ uint32_t ballot(bool p, uint32_t group_base) {
        const uint32_t all = __ballot_sync(0xFFFFFFFFu, p);
        return G == 32 ? all : (all >> group_base) & ((1u << (G & 31)) - 1u);
    }
};

// Slow path for the rows a warp holds: tau_i bit by bit by counting over the row (read again from global
// memory), then the ordered emit straight from the row.  Called by the whole warp; groups without a row
// (valid == false) run along on a row of their own that exists and store nothing.
template <int E8, int G>
__device__ __noinline__ void narrow_slow_path(const uint16_t* __restrict__ xr, uint32_t d, bool valid, uint32_t k,
                                              size_t out_base, uint32_t row, int16_t* __restrict__ cols_out,
                                              uint16_t* __restrict__ vals_out, int32_t* __restrict__ rows_out,
                                              uint16_t* __restrict__ tau_out) {
    using Gr = Group<G>;
    constexpr uint32_t E = E8 * 8u;
    const uint32_t gl = lane_id() & (G - 1);
    const uint4* mine = reinterpret_cast<const uint4*>(xr + gl * E);
    uint4 v[E8];                                   // (a lane past the end of the row holds zeros: the last columns)
#pragma unroll
    for (int c = 0; c < E8; ++c) v[c] = gl * E < d ? __ldg(mine + c) : make_uint4(0, 0, 0, 0);
    uint32_t tau_key = 0;
#pragma unroll 1
    for (int bit = 14; bit >= 0; --bit) {
        const uint32_t trial = tau_key | (1u << bit);
        uint32_t cnt = 0;
#pragma unroll
        for (int c = 0; c < E8; ++c) cnt += __popc(mask8_ge_exact(v[c], trial));
        if (Gr::sum(cnt) >= k) tau_key = trial;
    }
    uint32_t gt_mask = 0, eq_mask = 0;
#pragma unroll
    for (int c = 0; c < E8; ++c) {
        const uint32_t gt = mask8_ge_exact(v[c], tau_key + 1u);
        const uint32_t eq = mask8_ge_exact(v[c], tau_key) & ~gt;
        gt_mask |= gt << (8 * c);
        eq_mask |= eq << (8 * c);
    }
    const uint32_t n_gt_mine = __popc(gt_mask), n_eq_mine = __popc(eq_mask);
    const uint32_t incl = Gr::inclusive_sum(n_gt_mine, gl);
    const uint32_t take = k - Gr::last(incl);       // ties to keep, lowest columns first
    uint32_t g_at = incl - n_gt_mine;
    uint32_t e_at = Gr::inclusive_sum(n_eq_mine, gl) - n_eq_mine;
    uint32_t m = valid ? (gt_mask | eq_mask) : 0u;
    while (m) {
        const uint32_t j = __ffs(m) - 1;
        m &= m - 1;
        const bool is_eq = (eq_mask >> j) & 1u;
        if (!is_eq || e_at < take) {
            const size_t pos = out_base + g_at + (e_at < take ? e_at : take);
            cols_out[pos] = static_cast<int16_t>(gl * E + j);
            vals_out[pos] = xr[gl * E + j];
            if (rows_out) rows_out[pos] = static_cast<int32_t>(row);
        }
        g_at += is_eq ? 0u : 1u;
        e_at += is_eq ? 1u : 0u;
    }
    if (valid && gl == 0 && tau_out) tau_out[row] = static_cast<uint16_t>(tau_key);
}

template <int E8, int G, int PLN>
__global__ void __launch_bounds__(kNarrowWarps * 32)
mp_topk_fwd_bf16_narrow_kernel(const uint16_t* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                               int16_t* __restrict__ cols_out, uint16_t* __restrict__ vals_out,
                               int32_t* __restrict__ rows_out, uint16_t* __restrict__ tau_out,
                               dct_result_t* __restrict__ result) {
    using Gr = Group<G, PLN>;
    constexpr uint32_t kNarrowPerLane = PLN;       // candidates a lane holds in registers
    constexpr uint32_t E = E8 * 8u;                // columns per lane; the lane's candidate bits are one word
    constexpr uint32_t kRows = Gr::kRows;
    constexpr uint32_t kGuessMargin = 32;
    constexpr uint32_t kScratchWords = narrow_scratch_words<G>();
    __shared__ uint32_t s_scratch[kNarrowWarps][kScratchWords];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    const uint32_t gl = lane & (G - 1), group = lane / G, group_base = group * G;
    uint32_t* share = s_scratch[warp] + group * Gr::kShare;   // this group's list / histogram / stage, in turn

    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }
    // Row bundles (kRows consecutive rows) are dealt out CTA by CTA, then warp by warp.
    const uint32_t warps = blockDim.x >> 5;
    const uint64_t bundles = (static_cast<uint64_t>(rows) + kRows - 1) / kRows;
    const uint64_t first_bundle = blockIdx.x + static_cast<uint64_t>(gridDim.x) * warp;
    const uint64_t bundle_step = static_cast<uint64_t>(gridDim.x) * warps;
    // a group past the last row reads the last row instead (and stores nothing)
    auto row_of = [&](uint64_t bundle) -> uint64_t {
        const uint64_t r = bundle * kRows + group;
        return r < rows ? r : rows - 1;
    };
    // A row of d <= G E columns (d a multiple of E): the lanes past its end hold zeros, which lie below every bound
    // and, being the last columns, lose every tie.
    const bool lane_in = gl * E < d;
    auto load_row = [&](uint64_t r, uint4 (&v)[E8]) {
        const uint4* src = reinterpret_cast<const uint4*>(x + r * ld + gl * E);
#pragma unroll
        for (int c = 0; c < E8; ++c) v[c] = lane_in ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
    };
    uint4 cur[E8], nxt[E8];
    if (first_bundle < bundles) load_row(row_of(first_bundle), nxt);

    uint32_t guess_low = 0;                         // bound guessed from the group's previous row (0: none)
    const bool have_bound = k <= d / 8u;            // at least k leaves in a row
    for (uint64_t bundle = first_bundle; bundle < bundles; bundle += bundle_step) {
        const bool valid = bundle * kRows + group < rows;
        const uint64_t row64 = row_of(bundle);
        const uint32_t row = static_cast<uint32_t>(row64);
#pragma unroll
        for (int c = 0; c < E8; ++c) cur[c] = nxt[c];
        if (bundle + bundle_step < bundles) load_row(row_of(bundle + bundle_step), nxt);   // in flight meanwhile
        const uint16_t* xr = x + row64 * ld;
        const size_t out_base = static_cast<size_t>(row) * k;

        // ---- B (with A): candidate bits of the lane, one word in column order -------------------------
        uint32_t mask = 0, incl = 0, n_cand = 0;
        auto build_mask = [&](uint32_t bound) {
            mask = 0;
#pragma unroll
            for (int c = 0; c < E8; ++c) mask |= mask8_ge_exact(cur[c], bound) << (8 * c);
            incl = Gr::inclusive_sum(__popc(mask), gl);
            n_cand = Gr::last(incl);
        };
        uint32_t low = guess_low;
        bool settled = false;
        if (have_bound && __all_sync(0xFFFFFFFFu, guess_low != 0)) {
            build_mask(low);
            settled = __all_sync(0xFFFFFFFFu, n_cand >= k && n_cand <= Gr::kList);
        }
        if (!settled) {
            // exact bound: the k-th largest of the row's leaf maxima, bit by bit
            uint32_t leaf[E8];
#pragma unroll
            for (int c = 0; c < E8; ++c) {
                const __nv_bfloat162 m2 = __hmax2(__hmax2(__habs2(as_bf162(cur[c].x)), __habs2(as_bf162(cur[c].y))),
                                                  __hmax2(__habs2(as_bf162(cur[c].z)), __habs2(as_bf162(cur[c].w))));
                const uint32_t m = as_u32(m2);
                leaf[c] = max(m & 0xFFFFu, m >> 16);
            }
            low = 0;
            if (have_bound) {
#pragma unroll 1
                for (int bit = 14; bit >= 0; --bit) {
                    const uint32_t trial = low | (1u << bit);
                    uint32_t cnt = 0;
#pragma unroll
                    for (int c = 0; c < E8; ++c) cnt += leaf[c] >= trial ? 1u : 0u;
                    if (Gr::sum(cnt) >= k) low = trial;
                }
            }
            build_mask(low);
        }
        if (!have_bound || __any_sync(0xFFFFFFFFu, n_cand > Gr::kList || low == 0)) {
            narrow_slow_path<E8, G>(xr, d, valid, k, out_base, row, cols_out, vals_out, rows_out, tau_out);
            continue;
        }

        // candidates into the group's list, column order: entry = value | column << 16
        __syncwarp();                                   // whatever used the scratch before is done
        {
            uint32_t at = incl - __popc(mask);
            uint32_t m = mask;
            while (m) {
                const uint32_t col = gl * E + (__ffs(m) - 1);
                m &= m - 1;
                share[at++] = __ldg(xr + col) | (col << 16);
            }
        }
        __syncwarp();
        uint32_t ent[kNarrowPerLane];                   // 0: unused slot (a key below the bound, which is >= 1)
        const uint32_t per_lane = (n_cand + G - 1) / G;
#pragma unroll
        for (int i = 0; i < static_cast<int>(kNarrowPerLane); ++i) {
            const uint32_t r = gl * per_lane + i;
            ent[i] = (static_cast<uint32_t>(i) < per_lane && r < n_cand) ? share[r] : 0u;
        }
        __syncwarp();                                   // the list is in registers: its words become the histogram

        // ---- C: k-th largest of the candidates --------------------------------------------------
        uint32_t tau_key = 0, take = 0;
        bool found = false;
        {
            // 64 bins just above the bound, G private overflow bins behind them
            const uint32_t drop = n_cand - k;
            for (uint32_t b = gl; b < 64u + G; b += G) share[b] = 0;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < static_cast<int>(kNarrowPerLane); ++i) {
                const uint32_t rel = (ent[i] & 0x7FFFu) - low;
                atomicAdd(&share[rel < 64u ? rel : 64u + gl], 1u);
            }
            __syncwarp();
            uint32_t h[Gr::kBins], own = 0;             // the lane looks after bins gl kBins .. gl kBins + kBins - 1
#pragma unroll
            for (int j = 0; j < static_cast<int>(Gr::kBins); ++j) {
                h[j] = share[gl * Gr::kBins + j];
                own += h[j];
            }
            uint32_t before = Gr::inclusive_sum(own, gl) - own;
            uint32_t my_tau = 0, my_take = 0;
            bool mine = false;
#pragma unroll
            for (int j = 0; j < static_cast<int>(Gr::kBins); ++j) {
                if (before <= drop && drop < before + h[j]) {
                    mine = true;
                    my_tau = low + gl * Gr::kBins + j;
                    my_take = h[j] - (drop - before);
                }
                before += h[j];
            }
            const uint32_t who = Gr::ballot(mine, group_base);
            const uint32_t src = who ? __ffs(who) - 1 : 0u;
            tau_key = Gr::from(my_tau, src);
            take = Gr::from(my_take, src);
            found = who != 0;
            __syncwarp();
        }
        if (__any_sync(0xFFFFFFFFu, !found)) {
            // tau_i beyond the window for some row: the k-th largest candidate key, bit by bit (every group
            // recomputes; where the window had the answer this gives the same one)
            uint32_t t = 0;
#pragma unroll 1
            for (int bit = 14; bit >= 0; --bit) {
                const uint32_t trial = t | (1u << bit);
                uint32_t cnt = 0;
#pragma unroll
                for (int i = 0; i < static_cast<int>(kNarrowPerLane); ++i) cnt += (ent[i] & 0x7FFFu) >= trial ? 1u : 0u;
                if (Gr::sum(cnt) >= k) t = trial;
            }
            uint32_t above = 0;
#pragma unroll
            for (int i = 0; i < static_cast<int>(kNarrowPerLane); ++i) above += (ent[i] & 0x7FFFu) > t ? 1u : 0u;
            tau_key = t;
            take = k - Gr::sum(above);
        }
        if (valid && gl == 0 && tau_out) tau_out[row] = static_cast<uint16_t>(tau_key);
        guess_low = tau_key > kGuessMargin ? tau_key - kGuessMargin : 0u;

        // ---- D: ordered emit ------------------------------------------------------------------------
        {
            uint32_t counts = 0;                              // (gt << 16) | eq of this lane's entries
#pragma unroll
            for (int i = 0; i < static_cast<int>(kNarrowPerLane); ++i) {
                const uint32_t key = ent[i] & 0x7FFFu;
                counts += key > tau_key ? 0x10000u : (key == tau_key ? 1u : 0u);
            }
            const uint32_t before = Gr::inclusive_sum(counts, gl) - counts;
            uint32_t e_at = before & 0xFFFFu;
            uint32_t pos = (before >> 16) + (e_at < take ? e_at : take);
#pragma unroll
            for (int i = 0; i < static_cast<int>(kNarrowPerLane); ++i) {
                const uint32_t key = ent[i] & 0x7FFFu;
                const bool is_eq = key == tau_key;
                const bool keep = key > tau_key || (is_eq && e_at < take);
                if (keep) share[pos] = ent[i];
                pos += keep ? 1u : 0u;
                e_at += is_eq ? 1u : 0u;
            }
        }
        __syncwarp();
        if (valid) {
            for (uint32_t p = gl; p < k; p += G) {
                const uint32_t e = share[p];
                cols_out[out_base + p] = static_cast<int16_t>(e >> 16);
                vals_out[out_base + p] = static_cast<uint16_t>(e & 0xFFFFu);
                if (rows_out) rows_out[out_base + p] = static_cast<int32_t>(row);
            }
        }
        __syncwarp();
    }
}

template <int E8, int G, int PLN>
dct_status_t launch_narrow(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                           void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result,
                           cudaStream_t stream) {
    auto kernel = mp_topk_fwd_bf16_narrow_kernel<E8, G, PLN>;
    int per_sm = 0;
    DCT_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kNarrowWarps * 32, 0));
    if (per_sm < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t bundles = (static_cast<uint64_t>(rows) + Group<G>::kRows - 1) / Group<G>::kRows;
    const uint64_t ctas_needed = (bundles + kNarrowWarps - 1) / kNarrowWarps;
    const uint64_t max_grid = static_cast<uint64_t>(sms) * per_sm;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < max_grid ? ctas_needed : max_grid);
    kernel<<<grid, kNarrowWarps * 32, 0, stream>>>(static_cast<const uint16_t*>(x_act), rows, d, ld, k, cols_out,
                                                   static_cast<uint16_t*>(vals_out), rows_out,
                                                   static_cast<uint16_t*>(tau_out), result);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

// The largest 15-bit value t with "at least k of the row's keys are >= t", by counting (count_ge(t): the lane's keys
// >= t; the G lanes of the group are summed here).  With a guess (the value the group found for its previous row;
// 0: none) the search first tries the 256 values around it: two counts to see that the answer lies among them, then
// 8 halvings; otherwise, or if a group of the warp finds its guess off, 15 rounds bit by bit.  The control flow is
// the warp's (the sums are shuffles of all 32 lanes), so one group with a bad guess takes the others along.
template <int G, typename CountGe>
__device__ __forceinline__ uint32_t narrow_search15(CountGe&& count_ge, uint32_t k, uint32_t guess) {
    using Gr = Group<G>;
    constexpr uint32_t kHalf = 128;                  // one binade of bf16 keys on either side
    uint32_t lo = guess > kHalf ? guess - kHalf : 0u, hi = guess + kHalf < 0x8000u ? guess + kHalf : 0x8000u;
    bool ok = guess != 0;
    if (__any_sync(0xFFFFFFFFu, ok)) {               // (no group has a guess: skip the two counts)
        const uint32_t at_lo = Gr::sum(count_ge(lo)), at_hi = Gr::sum(count_ge(hi));   // (nothing is >= 0x8000)
        // (the sums are shuffles of all 32 lanes: they stay outside every condition that a lane can fail)
        ok = ok && at_lo >= k && at_hi < k;
    }
    if (__all_sync(0xFFFFFFFFu, ok)) {
#pragma unroll 1
        for (int round = 0; round < 8; ++round) {    // hi - lo <= 256: 8 halvings leave one value
            const uint32_t mid = lo + ((hi - lo) >> 1);
            if (Gr::sum(count_ge(mid)) >= k) lo = mid; else hi = mid;
        }
        return lo;
    }
    uint32_t key = 0;
#pragma unroll 1
    for (int bit = 14; bit >= 0; --bit) {
        const uint32_t trial = key | (1u << bit);
        if (Gr::sum(count_ge(trial)) >= k) key = trial;
    }
    return key;
}

// One bf16 row of a group by the count over the row in registers: narrow_slow_path with the search started from the
// group's previous tau_i (`guess`, updated).
// kAligned == false: rows of any width up to 32 G columns at any address (16-bit loads, columns past the end read as
// zeros, which lie below every bound and, being the last columns, lose every tie).
template <int E8, int G, bool kAligned = true>
__device__ __forceinline__ void narrow_count_path(const uint16_t* __restrict__ xr, uint32_t d, bool valid, uint32_t k,
                                                  size_t out_base, uint32_t row, int16_t* __restrict__ cols_out,
                                                  uint16_t* __restrict__ vals_out, int32_t* __restrict__ rows_out,
                                                  uint16_t* __restrict__ tau_out, uint32_t& guess) {
    using Gr = Group<G>;
    constexpr uint32_t E = E8 * 8u;
    const uint32_t gl = lane_id() & (G - 1);
    uint4 v[E8];                                   // (a lane past the end of the row holds zeros: the last columns)
    if constexpr (kAligned) {
        const uint4* mine = reinterpret_cast<const uint4*>(xr + gl * E);
#pragma unroll
        for (int c = 0; c < E8; ++c) v[c] = gl * E < d ? __ldg(mine + c) : make_uint4(0, 0, 0, 0);
    } else {
        auto pair = [&](uint32_t col) -> uint32_t {
            const uint32_t a = col < d ? __ldg(xr + col) : 0u, b = col + 1 < d ? __ldg(xr + col + 1) : 0u;
            return a | (b << 16);
        };
#pragma unroll
        for (int c = 0; c < E8; ++c) {
            const uint32_t col = gl * E + 8u * c;
            v[c] = make_uint4(pair(col), pair(col + 2), pair(col + 4), pair(col + 6));
        }
    }
    const uint32_t tau_key = narrow_search15<G>([&](uint32_t t) {
        uint32_t cnt = 0;
#pragma unroll
        for (int c = 0; c < E8; ++c) cnt += __popc(mask8_ge_exact(v[c], t));
        return cnt;
    }, k, guess);
    guess = tau_key;
    uint32_t gt_mask = 0, eq_mask = 0;
#pragma unroll
    for (int c = 0; c < E8; ++c) {
        const uint32_t gt = mask8_ge_exact(v[c], tau_key + 1u);
        const uint32_t eq = mask8_ge_exact(v[c], tau_key) & ~gt;
        gt_mask |= gt << (8 * c);
        eq_mask |= eq << (8 * c);
    }
    const uint32_t n_gt_mine = __popc(gt_mask), n_eq_mine = __popc(eq_mask);
    const uint32_t incl = Gr::inclusive_sum(n_gt_mine, gl);
    const uint32_t take = k - Gr::last(incl);       // ties to keep, lowest columns first
    uint32_t g_at = incl - n_gt_mine;
    uint32_t e_at = Gr::inclusive_sum(n_eq_mine, gl) - n_eq_mine;
    uint32_t m = valid ? (gt_mask | eq_mask) : 0u;
    while (m) {
        const uint32_t j = __ffs(m) - 1;
        m &= m - 1;
        const bool is_eq = (eq_mask >> j) & 1u;
        if (!is_eq || e_at < take) {
            const size_t pos = out_base + g_at + (e_at < take ? e_at : take);
            cols_out[pos] = static_cast<int16_t>(gl * E + j);
            vals_out[pos] = xr[gl * E + j];
            if (rows_out) rows_out[pos] = static_cast<int32_t>(row);
        }
        g_at += is_eq ? 0u : 1u;
        e_at += is_eq ? 1u : 0u;
    }
    if (valid && gl == 0 && tau_out) tau_out[row] = static_cast<uint16_t>(tau_key);
}

// Denser k (more than an eighth of the row: no leaf bound applies): every row takes the bit-by-bit count over the
// row in registers, 15 rounds for a bf16 key, and the ordered emit from the row.  The warp kernels and the general
// kernel pay their fixed cost per row for these short rows; here a warp serves 32 / G rows at once.
template <int E8, int G, bool kAligned>
__global__ void __launch_bounds__(kNarrowWarps * 32)
mp_topk_fwd_bf16_narrow_dense_kernel(const uint16_t* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                     int16_t* __restrict__ cols_out, uint16_t* __restrict__ vals_out,
                                     int32_t* __restrict__ rows_out, uint16_t* __restrict__ tau_out,
                                     dct_result_t* __restrict__ result) {
    constexpr uint32_t kRows = 32u / G;
    const uint32_t warp = threadIdx.x >> 5, group = lane_id() / G;
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }
    const uint64_t bundles = (static_cast<uint64_t>(rows) + kRows - 1) / kRows;
    const uint64_t bundle_step = static_cast<uint64_t>(gridDim.x) * (blockDim.x >> 5);
    uint32_t guess = 0;                              // tau_i of the group's previous row
    for (uint64_t bundle = blockIdx.x + static_cast<uint64_t>(gridDim.x) * warp; bundle < bundles; bundle += bundle_step) {
        const uint64_t r = bundle * kRows + group;
        const bool valid = r < rows;
        const uint64_t row64 = valid ? r : rows - 1;     // a group past the last row runs along on the last row
        narrow_count_path<E8, G, kAligned>(x + row64 * ld, d, valid, k, static_cast<size_t>(row64) * k, static_cast<uint32_t>(row64),
                                 cols_out, vals_out, rows_out, tau_out, guess);
    }
}

template <int E8, int G, bool kAligned = true>
dct_status_t launch_narrow_dense(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                                 void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result,
                                 cudaStream_t stream) {
    auto kernel = mp_topk_fwd_bf16_narrow_dense_kernel<E8, G, kAligned>;
    int per_sm = 0;
    DCT_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kNarrowWarps * 32, 0));
    if (per_sm < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t bundles = (static_cast<uint64_t>(rows) + (32u / G) - 1) / (32u / G);
    const uint64_t ctas_needed = (bundles + kNarrowWarps - 1) / kNarrowWarps;
    const uint64_t max_grid = static_cast<uint64_t>(sms) * per_sm;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < max_grid ? ctas_needed : max_grid);
    kernel<<<grid, kNarrowWarps * 32, 0, stream>>>(static_cast<const uint16_t*>(x_act), rows, d, ld, k, cols_out,
                                                   static_cast<uint16_t*>(vals_out), rows_out,
                                                   static_cast<uint16_t*>(tau_out), result);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

// ------------------------------------------------------------------------------------------
// fp32 rows of up to 256 columns: the count over the row in registers, on two levels
// ------------------------------------------------------------------------------------------
// The paper's recommendation model runs in fp32.  A key has 31 bits; as in the other fp32 kernels the first level
// works on its upper 15 bits (the bucket: the bf16 truncation of |x|), which gives the bucket of tau_i and how many
// of its members belong to the top k; the members (usually one) are then ranked by their lower 16 bits.  A lane
// holds 32 consecutive columns (eight 16-byte loads), a group of G = 2, 4 or 8 lanes a row.
// tau_i bit by bit by counting over the row in registers, then the ordered emit straight from the
// row.  The upper 15 key bits (the bucket) take 15 rounds on the packed upper halves, eight columns per exact flag
// step as in the bf16 kernels; the lower 16 bits come from the bucket's members: the smallest of them if all are
// needed (the usual case: one member), the largest if one is, else 16 more rounds over the row's keys.  Called by the
// whole warp; groups without a row run along and store nothing.
template <int G, bool kAligned = true>
__device__ __forceinline__ void narrow_bisect_f32(const uint32_t* __restrict__ xr, uint32_t d, bool valid, uint32_t k,
                                                  size_t out_base, uint32_t row, int16_t* __restrict__ cols_out,
                                                  uint32_t* __restrict__ vals_out, int32_t* __restrict__ rows_out,
                                                  uint32_t* __restrict__ tau_out, uint32_t& guess) {
    using Gr = Group<G>;
    constexpr uint32_t E = 32u;
    const uint32_t gl = lane_id() & (G - 1);
    uint32_t key[E];
    uint4 up[4];                                   // upper halves of the lane's 32 columns, eight to a register quad
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint4 v;
        if constexpr (kAligned) {
            v = gl * E < d ? __ldg(reinterpret_cast<const uint4*>(xr + gl * E) + c) : make_uint4(0, 0, 0, 0);
        } else {                               // any width, any address: columns past the end read as zeros
            const uint32_t col = gl * E + 4u * c;
            v.x = col < d ? __ldg(xr + col) : 0u;
            v.y = col + 1 < d ? __ldg(xr + col + 1) : 0u;
            v.z = col + 2 < d ? __ldg(xr + col + 2) : 0u;
            v.w = col + 3 < d ? __ldg(xr + col + 3) : 0u;
        }
        key[4 * c] = v.x & 0x7FFFFFFFu;
        key[4 * c + 1] = v.y & 0x7FFFFFFFu;
        key[4 * c + 2] = v.z & 0x7FFFFFFFu;
        key[4 * c + 3] = v.w & 0x7FFFFFFFu;
        if (c & 1) {
            up[c / 2].z = upper_halves(v.x, v.y);
            up[c / 2].w = upper_halves(v.z, v.w);
        } else {
            up[c / 2].x = upper_halves(v.x, v.y);
            up[c / 2].y = upper_halves(v.z, v.w);
        }
    }
    const uint32_t bucket = narrow_search15<G>([&](uint32_t t) {
        uint32_t cnt = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) cnt += __popc(mask8_ge_exact(up[c], t));
        return cnt;
    }, k, guess);
    guess = bucket;                                // (the group's next row starts its search around this bucket)
    uint32_t above = 0, members = 0;               // columns of the lane above the bucket / inside it
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t gt = mask8_ge_exact(up[c], bucket + 1u);
        above |= gt << (8 * c);
        members |= (mask8_ge_exact(up[c], bucket) & ~gt) << (8 * c);
    }
    const uint32_t need = k - Gr::sum(__popc(above));      // members of the bucket that belong to the top k: >= 1
    const uint32_t in_bucket = Gr::sum(__popc(members));
    uint32_t tau_key = bucket << 16;
    if (__all_sync(0xFFFFFFFFu, need == in_bucket || need == 1u)) {
        uint32_t lo = 0xFFFFFFFFu, hi = 0;
        for (uint32_t m = members; m; m &= m - 1) {
            // (a lane past the end of the row holds zeros: nothing of its own to read)
            const uint32_t col = gl * E + __ffs(m) - 1;
            const uint32_t v = col < d ? xr[col] & 0x7FFFFFFFu : 0u;
            lo = v < lo ? v : lo;
            hi = v > hi ? v : hi;
        }
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) {
            const uint32_t a = __shfl_xor_sync(0xFFFFFFFFu, lo, o, G), b = __shfl_xor_sync(0xFFFFFFFFu, hi, o, G);
            lo = a < lo ? a : lo;
            hi = b > hi ? b : hi;
        }
        tau_key = need == in_bucket ? lo : hi;
    } else {
#pragma unroll 1
        for (int bit = 15; bit >= 0; --bit) {
            const uint32_t trial = tau_key | (1u << bit);
            uint32_t cnt = 0;
#pragma unroll
            for (int j = 0; j < static_cast<int>(E); ++j) cnt += key[j] >= trial ? 1u : 0u;
            if (Gr::sum(cnt) >= k) tau_key = trial;
        }
    }
    uint32_t gt_mask = 0, eq_mask = 0;
#pragma unroll
    for (int j = 0; j < static_cast<int>(E); ++j) {
        gt_mask |= key[j] > tau_key ? 1u << j : 0u;
        eq_mask |= key[j] == tau_key ? 1u << j : 0u;
    }
    const uint32_t n_gt_mine = __popc(gt_mask), n_eq_mine = __popc(eq_mask);
    const uint32_t incl = Gr::inclusive_sum(n_gt_mine, gl);
    const uint32_t take = k - Gr::last(incl);       // ties to keep, lowest columns first
    uint32_t g_at = incl - n_gt_mine;
    uint32_t e_at = Gr::inclusive_sum(n_eq_mine, gl) - n_eq_mine;
    uint32_t m = valid ? (gt_mask | eq_mask) : 0u;
    while (m) {
        const uint32_t j = __ffs(m) - 1;
        m &= m - 1;
        const bool is_eq = (eq_mask >> j) & 1u;
        if (!is_eq || e_at < take) {
            const size_t pos = out_base + g_at + (e_at < take ? e_at : take);
            cols_out[pos] = static_cast<int16_t>(gl * E + j);
            vals_out[pos] = xr[gl * E + j];
            if (rows_out) rows_out[pos] = static_cast<int32_t>(row);
        }
        g_at += is_eq ? 0u : 1u;
        e_at += is_eq ? 1u : 0u;
    }
    if (valid && gl == 0 && tau_out) tau_out[row] = tau_key;
}

// Denser k, fp32: the two-level bit-by-bit count over the row in registers (narrow_bisect_f32), for every row.
template <int G, bool kAligned>
__global__ void __launch_bounds__(kNarrowWarps * 32, 2)
mp_topk_fwd_f32_narrow_dense_kernel(const uint32_t* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                    int16_t* __restrict__ cols_out, uint32_t* __restrict__ vals_out,
                                    int32_t* __restrict__ rows_out, uint32_t* __restrict__ tau_out,
                                    dct_result_t* __restrict__ result) {
    constexpr uint32_t kRows = 32u / G;
    const uint32_t warp = threadIdx.x >> 5, group = lane_id() / G;
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }
    const uint64_t bundles = (static_cast<uint64_t>(rows) + kRows - 1) / kRows;
    const uint64_t bundle_step = static_cast<uint64_t>(gridDim.x) * (blockDim.x >> 5);
    uint32_t guess = 0;                              // bucket of tau_i of the group's previous row
    for (uint64_t bundle = blockIdx.x + static_cast<uint64_t>(gridDim.x) * warp; bundle < bundles; bundle += bundle_step) {
        const uint64_t r = bundle * kRows + group;
        const bool valid = r < rows;
        const uint64_t row64 = valid ? r : rows - 1;
        narrow_bisect_f32<G, kAligned>(x + row64 * ld, d, valid, k, static_cast<size_t>(row64) * k, static_cast<uint32_t>(row64),
                             cols_out, vals_out, rows_out, tau_out, guess);
    }
}

template <int G, bool kAligned = true>
dct_status_t launch_narrow_dense_f32(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                     int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                     dct_result_t* result, cudaStream_t stream) {
    auto kernel = mp_topk_fwd_f32_narrow_dense_kernel<G, kAligned>;
    int per_sm = 0;
    DCT_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kNarrowWarps * 32, 0));
    if (per_sm < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t bundles = (static_cast<uint64_t>(rows) + (32u / G) - 1) / (32u / G);
    const uint64_t ctas_needed = (bundles + kNarrowWarps - 1) / kNarrowWarps;
    const uint64_t max_grid = static_cast<uint64_t>(sms) * per_sm;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < max_grid ? ctas_needed : max_grid);
    kernel<<<grid, kNarrowWarps * 32, 0, stream>>>(static_cast<const uint32_t*>(x_act), rows, d, ld, k, cols_out,
                                                   static_cast<uint32_t*>(vals_out), rows_out,
                                                   static_cast<uint32_t*>(tau_out), result);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

}  // namespace

// *handled = false: not a shape of this path; the caller goes on to the other kernels.
// The list of a row holds 5 candidates per lane of its group and must take the ~1.3 k candidates (1.45 k at
// the 99th percentile) the bound leaves: k <= 3.4 lanes.
dct_status_t launch_fwd_bf16_narrow(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                    int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                    dct_result_t* result, cudaStream_t stream, bool* handled) {
    *handled = false;
    const bool odd = !aligned_to(x_act, 16) || (static_cast<size_t>(ld) * 2) % 16 != 0 || d % 8 != 0;
    if (odd || (d <= 256 && d % 32 != 0)) {
        // Rows the 16-byte loads of every other fast kernel cannot take (odd widths, odd strides, odd addresses): up to
        // 1024 columns they take the count over the row with 16-bit loads, for every k (the general kernel: 0.1 to 0.4
        // TB/s).  So do short rows that are not whole lanes of 32 columns (100, 200 columns: the warp-per-row kernels
        // spend a warp on a few hundred bytes).
        if (d > 1024) return DCT_OK;
        *handled = true;
        if (d > 512) return launch_narrow_dense<4, 32, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        if (d <= 64) return launch_narrow_dense<4, 2, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        if (d <= 128) return launch_narrow_dense<4, 4, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        if (d <= 256) return launch_narrow_dense<4, 8, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        return launch_narrow_dense<4, 16, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    }
    *handled = true;
    // The count over the row in registers, for every row (15 rounds): the denser k on rows of up to 256 columns, and
    // every k on rows of up to 128 columns, where it beats the bound-and-candidates kernel as well (1572864 rows of 64
    // columns, k = 3: 0.133 against 0.322 ms; 786432 x 128, k = 6: 0.141 against 0.174 ms; 256 columns, k = 2: 0.136
    // against 0.123 ms).
    if (d % 32 == 0 && d <= 64) return launch_narrow_dense<4, 2>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    if (d % 32 == 0 && d <= 128) return launch_narrow_dense<4, 4>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    if (k > d / 8) {
        if (d % 32 == 0 && d <= 256) return launch_narrow_dense<4, 8>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        *handled = false;
        return DCT_OK;
    }
    // 5 candidates per lane up to k = 2.5 lanes of the group, 8 up to 4.25 lanes (the bound leaves ~1.3 k candidates,
    // 1.45 k at the 99th percentile)
#define DCT_NARROW(E8, G, K5, K8)                                                                                          \
    if (k <= K5) return launch_narrow<E8, G, 5>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream); \
    if (k <= K8) return launch_narrow<E8, G, 8>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream)
    // (k <= d / 8 was checked above: the bound needs k leaves of 8 columns; rows narrower than the group's 32 G
    // columns, in whole lanes of 32, leave the lanes past their end empty)
    if (d % 32 == 0 && d <= 256) {
        DCT_NARROW(4, 8, 20, 32);
    } else if (d % 32 == 0 && d <= 512) {  // (k = 51 with 8 candidates per lane: 0.125 ms for 131072 rows of 512, the warp-per-row kernel 0.104)
        DCT_NARROW(4, 16, 40, 40);
    }
#undef DCT_NARROW
    *handled = false;
    return DCT_OK;
}

// fp32 rows of up to 256 columns (whole lanes of 32), any k: the two-level count over the row in registers.  It beat
// the bound-and-candidates kernel this file used to have for fp32 at every width it served (786432 rows of 64 columns,
// k = 3: 0.100 against 0.252 ms; 393216 x 128, k = 6: 0.107 against 0.152; 196608 x 256, k = 12: 0.112 against 0.120)
// and serves the denser k the warp-per-row kernels leave to the general one (128 columns, k = 32: 0.159 against 0.98 ms).
// Rows of 512 columns stay with the warp-per-row kernels (0.084 against 0.110 ms at k = 5).
dct_status_t launch_fwd_f32_narrow(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                   int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                   dct_result_t* result, cudaStream_t stream, bool* handled) {
    *handled = false;
    const bool odd = !aligned_to(x_act, 16) || (static_cast<size_t>(ld) * 4) % 16 != 0 || d % 4 != 0;
    if (odd || (d <= 256 && d % 32 != 0)) {
        // rows the 16-byte loads cannot take: up to 1024 columns, the count over the row with 32-bit loads, for every k;
        // so do short rows that are not whole lanes of 32 columns
        if (d > 1024) return DCT_OK;
        *handled = true;
        if (d > 512) return launch_narrow_dense_f32<32, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        if (d <= 64) return launch_narrow_dense_f32<2, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        if (d <= 128) return launch_narrow_dense_f32<4, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        if (d <= 256) return launch_narrow_dense_f32<8, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
        return launch_narrow_dense_f32<16, false>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    }
    if (d % 32 != 0) return DCT_OK;
    // 288 to 480 columns, the denser k: 16 lanes per row (the bounds-and-bit-tables kernel of the 512-column buffer
    // is crowded by rows that fill only part of it: 320 columns, k = 80: 0.47 TB/s)
    if (d > 256 && d < 512 && fwd_candidates_per_lane(d, k) == 0) {
        *handled = true;
        return launch_narrow_dense_f32<16>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    }
    if (d > 256) return DCT_OK;
    *handled = true;
    if (d <= 64) return launch_narrow_dense_f32<2>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    if (d <= 128) return launch_narrow_dense_f32<4>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    return launch_narrow_dense_f32<8>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
}

}  // namespace dct
