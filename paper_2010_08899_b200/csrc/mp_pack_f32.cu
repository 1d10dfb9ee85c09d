// dct_mp_topk_pack_fwd, fp32 fast path: Algorithm 2 (DCT-MP), one warp per sample (row).
//
// The structure is that of the bf16 warp-per-row kernel (mp_pack.cu); what differs is how a 31-bit key is
// handled with the same 15-bit machinery:
//   * every step up to and including the select works on the upper 15 bits of the key (the bf16
//     truncation of |x|): the bound, the candidate bits, the windowed histogram.  Packed bf16 compares
//     run on the upper halves of two fp32 words gathered into one register by a byte permute.
//   * that select yields the 15-bit bucket that holds tau_i and how many of its members belong to the
//     top k.  The members (a handful: the candidates are about two per bucket near the threshold) are
//     then ranked by their full keys, which gives the exact 31-bit tau_i and the number of ties to keep.
//   * the candidates carry their full 32-bit value from the row buffer, so the emit needs nothing else.
// Rows are 16-byte aligned, d <= 4096 a multiple of 4 (held zero-padded in a buffer of 256 * E8 columns),
// k <= 224 and k <= d/8 (10
// candidates per lane) or k <= 448 and k <= d/4 (20 per lane); everything else takes the general kernel.
#include "common.cuh"
#include "mp_warp.cuh"

namespace dct {
namespace {

template <int E8> struct RowLayoutF32 {
    static constexpr uint32_t E = E8 * 8u, D = E * 32u;
    static constexpr uint32_t kRowBytes = D * 4u;             // the row lies in shared memory as it does in HBM
    static constexpr uint32_t kRowWords = 8u * E8;            // 32-bit candidate-bit words of a row (one bit per column)
    static constexpr uint32_t kMaskWords = (E8 + 3) / 4;      // bit words a lane looks after
    static constexpr uint32_t kTableWords = 32u * kMaskWords;
    // per warp: row | scratch | mbarrier.  The scratch is, in turn: leaf histogram; bit table; linked table;
    // select histogram; member list; the staged columns [0, kpad) and values [kpad, 2 kpad).
    __host__ __device__ static constexpr uint32_t kpad(uint32_t k) { return (k + 3u) & ~3u; }
    __host__ __device__ static constexpr uint32_t scratch_words(uint32_t k) {
        uint32_t w = 2u * kTableWords > kHistWords ? 2u * kTableWords : kHistWords;
        return w > 2u * kpad(k) ? w : 2u * kpad(k);
    }
    __host__ __device__ static constexpr uint32_t warp_bytes(uint32_t k) {
        return kRowBytes + scratch_words(k) * 4u + 16u;
    }
};

constexpr uint32_t kMaxMembers = 64;      // bucket members ranked through the list; more take the bit-serial route

// exact key >= low on 31-bit keys, 4 elements
__device__ __forceinline__ uint32_t mask4_ge_exact(uint4 v, uint32_t low) {
    return ((v.x & 0x7FFFFFFFu) >= low ? 1u : 0u) | ((v.y & 0x7FFFFFFFu) >= low ? 2u : 0u) |
           ((v.z & 0x7FFFFFFFu) >= low ? 4u : 0u) | ((v.w & 0x7FFFFFFFu) >= low ? 8u : 0u);
}

// General slow path for one row (rare): tau_i bit by bit over the 31 key bits by counting over the row, then
// everything above tau_i and the first ties, in column order, straight from the row.  Lane l owns the
// E consecutive columns from l E on.
template <int E8>
__device__ __noinline__ void mp_row_slow_path_f32(const unsigned char* span, uint32_t k, size_t out_base, uint32_t row,
                                                  int16_t* __restrict__ cols_out, uint32_t* __restrict__ vals_out,
                                                  int32_t* __restrict__ rows_out, uint32_t* __restrict__ tau_out) {
    constexpr uint32_t E = E8 * 8u;
    constexpr int kMaskWords = (E8 + 3) / 4;
    const uint32_t lane = lane_id();
    uint32_t tau_key = 0;
#pragma unroll 1
    for (int bit = 30; bit >= 0; --bit) {
        const uint32_t trial = tau_key | (1u << bit);
        uint32_t cnt = 0;
#pragma unroll 4
        for (int c = 0; c < 2 * E8; ++c)
            cnt += __popc(mask4_ge_exact(*reinterpret_cast<const uint4*>(span + c * 16), trial));
        if (__reduce_add_sync(0xFFFFFFFFu, cnt) >= k) tau_key = trial;
    }
    uint32_t gt_masks[kMaskWords], eq_masks[kMaskWords];
    uint32_t n_gt_mine = 0, n_eq_mine = 0;
#pragma unroll
    for (int i = 0; i < kMaskWords; ++i) gt_masks[i] = eq_masks[i] = 0;
#pragma unroll
    for (int c = 0; c < 2 * E8; ++c) {
        const uint4 v = *reinterpret_cast<const uint4*>(span + c * 16);
        const uint32_t gt = tau_key == 0x7FFFFFFFu ? 0u : mask4_ge_exact(v, tau_key + 1u);
        const uint32_t eq = mask4_ge_exact(v, tau_key) & ~gt;
        gt_masks[c / 8] |= gt << (4 * (c % 8));
        eq_masks[c / 8] |= eq << (4 * (c % 8));
        n_gt_mine += __popc(gt);
        n_eq_mine += __popc(eq);
    }
    const uint32_t incl = warp_inclusive_sum(n_gt_mine);
    const uint32_t take = k - __shfl_sync(0xFFFFFFFFu, incl, 31);   // ties to keep, lowest columns first
    uint32_t g_at = incl - n_gt_mine;
    uint32_t e_at = warp_inclusive_sum(n_eq_mine) - n_eq_mine;
#pragma unroll
    for (int wd = 0; wd < kMaskWords; ++wd) {
        uint32_t m = gt_masks[wd] | eq_masks[wd];
        while (m) {
            const uint32_t bit = __ffs(m) - 1;
            m &= m - 1;
            const bool is_eq = (eq_masks[wd] >> bit) & 1u;
            if (!is_eq || e_at < take) {
                const uint32_t j = wd * 32 + bit;
                const size_t pos = out_base + g_at + (e_at < take ? e_at : take);
                cols_out[pos] = static_cast<int16_t>(lane * E + j);
                vals_out[pos] = *reinterpret_cast<const uint32_t*>(span + j * 4);
                if (rows_out) rows_out[pos] = static_cast<int32_t>(row);
            }
            g_at += is_eq ? 0u : 1u;
            e_at += is_eq ? 1u : 0u;
        }
    }
    if (lane == 0 && tau_out) tau_out[row] = tau_key;
}

// Warps of a CTA at most: 32 for rows of up to 1024 columns (4 KB: shared memory has room for them, and the
// kernel fits the 64 registers that allows; 9 to 10 % faster than 24), else what the registers of the variant allow.
template <int E8, int PL> constexpr int fwd_f32_max_warps() {
    return (E8 <= 4 && PL <= 10) ? 32 : FwdVariant<PL>::kMaxWarps;
}

template <int E8, int PL>
__global__ void __launch_bounds__(fwd_f32_max_warps<E8, PL>() * 32)
mp_topk_fwd_f32_warp_kernel(const uint32_t* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                            int16_t* __restrict__ cols_out, uint32_t* __restrict__ vals_out,
                            int32_t* __restrict__ rows_out, uint32_t* __restrict__ tau_out,
                            dct_result_t* __restrict__ result) {
    using Lay = RowLayoutF32<E8>;
    constexpr int kMaskWords = Lay::kMaskWords;
    constexpr uint32_t kPerLane = PL, kRound = 32u * kPerLane;
    constexpr bool kFineLeaves = FwdVariant<PL>::kFineLeaves;
    constexpr int kLeaves = kFineLeaves ? 2 * E8 : E8;           // leaves per lane (4 or 8 elements each)
    constexpr uint32_t kGuessMargin = 32;                         // 15-bit keys below the previous tau_i
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned char* base = smem_raw + warp * Lay::warp_bytes(k);
    unsigned char* span = base + lane * (Lay::E * 4u);        // the slow path's view: E consecutive columns per lane
    uint32_t* scratch = reinterpret_cast<uint32_t*>(base + Lay::kRowBytes);
    uint32_t* mask_tab = scratch;                             // one bit per column (upper key bits >= bound), column order
    uint2* table = reinterpret_cast<uint2*>(scratch);        // per bit word: {mask, running count and link}
    uint32_t* hist = scratch;
    uint32_t* stage_col = scratch;
    uint32_t* stage_val = scratch + Lay::kpad(k);
    uint64_t* bar = reinterpret_cast<uint64_t*>(scratch + Lay::scratch_words(k));
    __shared__ uint32_t s_stop;
    __shared__ uint32_t s_next;                               // rows of this CTA handed out so far
    __shared__ uint32_t s_hint;                               // the latest bound any warp of this CTA guessed from a tau_i

    if (threadIdx.x == 0) {
        s_stop = 0;
        s_next = blockDim.x >> 5;
        s_hint = 0;
    }
    if (lane == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
        fence_proxy_async_all();
    }
    // A row of d <= D columns (d a multiple of 4) fills the first d columns of the buffer; the rest is zeroed
    // once and never written again: zeros lie below every bound and, being the last columns, lose every tie.
    const uint32_t row_bytes = d * 4u;
    for (uint32_t b = row_bytes + lane * 16u; b < Lay::kRowBytes; b += 512u)
        *reinterpret_cast<uint4*>(base + b) = make_uint4(0, 0, 0, 0);
    __syncthreads();
    chain_wait_previous();          // set-up above; inputs and outputs only below (see the bf16 kernel in mp_pack.cu)
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }

    // rows are dealt out CTA by CTA (row mod grid = CTA); inside the CTA a warp takes the CTA's next row whenever
    // it lets go of one (see the bf16 kernel in mp_pack.cu)
    const uint32_t warp_global = blockIdx.x + gridDim.x * warp;             // this warp's first row
    auto request_row = [&](uint32_t r) {          // one bulk copy brings the whole row
        if (lane == 0) {
            mbar_arrive_expect_tx(bar, row_bytes);
            bulk_load(base, x + static_cast<size_t>(r) * ld, row_bytes, bar);
        }
    };
    uint64_t next_row = 0;
    auto release_row = [&]() {               // the row buffer is no longer needed: request the CTA's next row
        __syncwarp();
        fence_proxy_async_smem();
        uint32_t j = 0;
        if (lane == 0) j = atomicAdd(&s_next, 1u);
        j = __shfl_sync(0xFFFFFFFFu, j, 0);
        next_row = blockIdx.x + static_cast<uint64_t>(gridDim.x) * j;
        if (next_row < rows) request_row(static_cast<uint32_t>(next_row));
    };
    // In the passes over the whole row lane l reads the 32-byte pieces l, l + 32, ... (8 columns each, one byte
    // of the bit table).  The two 16-byte halves of a piece are read in an order that depends on the lane, so
    // that the eight lanes served together touch eight different bank groups.
    const uint32_t swap = (lane >> 2) & 1u;                   // 1: this lane reads columns 4..7 of a piece first
    const unsigned char* piece_first = base + lane * 32u + swap * 16u;
    const unsigned char* piece_second = base + lane * 32u + (swap ^ 1u) * 16u;
    // where the flags of the two reads go in the byte of the piece (bit j = column j of the piece)
    const uint32_t w_first = swap ? 0x80C0E0F0u : 0xF8FCFEFFu;      // dot-product weights -2^j of the columns a read holds
    const uint32_t w_second = swap ? 0xF8FCFEFFu : 0x80C0E0F0u;
    if (warp_global < rows) request_row(warp_global);

    uint32_t use = 0;
    uint32_t guess_low = 0;                         // 15-bit bound guessed from the previous row (0: none)
    for (uint64_t row64 = warp_global; row64 < rows; row64 = next_row, ++use) {
        const uint32_t row = static_cast<uint32_t>(row64);
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(bar, use & 1u, 1u << 24, &s_stop))) {
            s_stop = 1;
            if (lane == 0 && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
            return;
        }
        const size_t out_base = static_cast<size_t>(row) * k;

        // ---- A: a lower bound for the upper 15 bits of tau_i -----------------------------------------
        uint32_t row_max = 0x7FFFu;                  // only the exact bound computes the true maximum
        const bool have_bound = k <= 32u * kLeaves;
        auto exact_bound = [&]() -> uint32_t {
            uint32_t leaf[kLeaves];
            uint32_t top = 0;
#pragma unroll
            for (int c = 0; c < E8; ++c) {
                const uint4 a = *reinterpret_cast<const uint4*>(piece_first + c * 1024);
                const uint4 b = *reinterpret_cast<const uint4*>(piece_second + c * 1024);
                const __nv_bfloat162 ma = __hmax2(__habs2(as_bf162(upper_halves(a.x, a.y))),
                                                  __habs2(as_bf162(upper_halves(a.z, a.w))));
                const __nv_bfloat162 mb = __hmax2(__habs2(as_bf162(upper_halves(b.x, b.y))),
                                                  __habs2(as_bf162(upper_halves(b.z, b.w))));
                if (kFineLeaves) {
                    const uint32_t ua = as_u32(ma), ub = as_u32(mb);
                    leaf[2 * c] = max(ua & 0xFFFFu, ua >> 16);
                    leaf[2 * c + 1] = max(ub & 0xFFFFu, ub >> 16);
                    top = max(top, max(leaf[2 * c], leaf[2 * c + 1]));
                } else {
                    const uint32_t m = as_u32(__hmax2(ma, mb));
                    leaf[c] = max(m & 0xFFFFu, m >> 16);
                    top = max(top, leaf[c]);
                }
            }
            row_max = __reduce_max_sync(0xFFFFFFFFu, top);
            if (!have_bound) return 0u;
            // histogram of the leaf maxima in bins of 8 keys counted down from the row maximum; the bound is the
            // lowest key of the bin in which the count reaches k
            reinterpret_cast<uint4*>(hist)[lane] = make_uint4(0, 0, 0, 0);
            reinterpret_cast<uint4*>(hist)[lane + 32] = make_uint4(0, 0, 0, 0);
            __syncwarp();
#pragma unroll
            for (int c = 0; c < kLeaves; ++c) {
                const uint32_t rel = (row_max - leaf[c]) >> 3;
                atomicAdd(&hist[rel < 255u ? rel : 255u], 1u);
            }
            __syncwarp();
            uint32_t need = k, bin = 255;
#pragma unroll 1
            for (uint32_t first = 0; first < 256; first += 32) {
                const uint32_t c = hist[first + lane];
                const uint32_t inc = warp_inclusive_sum(c);
                const uint32_t hit = __ballot_sync(0xFFFFFFFFu, inc >= need);
                if (hit) {
                    bin = first + (__ffs(hit) - 1);
                    break;
                }
                need -= __shfl_sync(0xFFFFFFFFu, inc, 31);
            }
            __syncwarp();
            const uint32_t span_keys = bin * 8u + 7u;
            return (bin < 255u && row_max > span_keys) ? row_max - span_keys : 0u;
        };

        // ---- B: candidate bits (upper key bits >= bound), in column order ------------------------------
        uint32_t masks[kMaskWords];
        uint32_t n_mine = 0, incl = 0, n_cand = 0;
        auto build_masks = [&](uint32_t bound, bool probe) -> bool {
            const uint32_t low2 = bound | (bound << 16);
            unsigned char* tab8 = reinterpret_cast<unsigned char*>(mask_tab) + lane;
            {
                const uint4 a = *reinterpret_cast<const uint4*>(piece_first);
                const uint4 b = *reinterpret_cast<const uint4*>(piece_second);
                const uint32_t m0 = piece_flags(a, b, low2, w_first, w_second);
                tab8[0] = static_cast<unsigned char>(m0);
                // a guessed bound is probed on the first piece of every lane (1 / E8 of the row) before the rest of
                // the pass is made for it (see the bf16 kernel, mp_pack.cu)
                if (E8 >= 8 && probe) {
                    const uint32_t sample = __reduce_add_sync(0xFFFFFFFFu, __popc(m0)) * E8;
                    if (8u * sample < 5u * k || 5u * sample > 8u * kRound) {
                        n_cand = 0;
                        return false;
                    }
                }
            }
#pragma unroll
            for (int c = 1; c < E8; ++c) {
                const uint4 a = *reinterpret_cast<const uint4*>(piece_first + c * 1024);
                const uint4 b = *reinterpret_cast<const uint4*>(piece_second + c * 1024);
                tab8[c * 32] = static_cast<unsigned char>(piece_flags(a, b, low2, w_first, w_second));
            }
            __syncwarp();
            if (kMaskWords == 4) {
                const uint4 t = reinterpret_cast<const uint4*>(mask_tab)[lane];
                masks[0] = t.x; masks[1 % kMaskWords] = t.y; masks[2 % kMaskWords] = t.z; masks[3 % kMaskWords] = t.w;
            } else if (kMaskWords == 2) {
                const uint2 t = reinterpret_cast<const uint2*>(mask_tab)[lane];
                masks[0] = t.x; masks[1 % kMaskWords] = t.y;
            } else {
#pragma unroll
                for (int i = 0; i < kMaskWords; ++i) masks[i] = mask_tab[lane * kMaskWords + i];
            }
            if (Lay::kRowWords != Lay::kTableWords) {
#pragma unroll
                for (int i = 0; i < kMaskWords; ++i)
                    if (lane * kMaskWords + i >= Lay::kRowWords) masks[i] = 0u;
            }
            n_mine = 0;
#pragma unroll
            for (int i = 0; i < kMaskWords; ++i) n_mine += __popc(masks[i]);
            incl = warp_inclusive_sum(n_mine);
            n_cand = __shfl_sync(0xFFFFFFFFu, incl, 31);
            return true;
        };

        uint32_t low = 0;
        if (guess_low == 0) guess_low = *reinterpret_cast<volatile uint32_t*>(&s_hint);   // none of its own: the CTA's latest
        bool use_guess = have_bound && guess_low != 0;
#pragma unroll 1
        while (true) {
            low = use_guess ? guess_low : exact_bound();
            const bool built = build_masks(low, use_guess);
            if (!use_guess || (built && n_cand >= k && n_cand <= kRound)) break;
            use_guess = false;
        }
        if (!have_bound || n_cand > kRound || low == 0) {
            mp_row_slow_path_f32<E8>(span, k, out_base, row, cols_out, vals_out, rows_out, tau_out);
            release_row();
            continue;
        }

        // ---- C: candidates into registers, evenly (linked table, branch-free walk) ----------------------
        uint32_t first_word;
        {
            const uint32_t wbase = lane * kMaskWords;
            uint32_t my_first = Lay::kTableWords;
#pragma unroll
            for (int i = kMaskWords - 1; i >= 0; --i)
                if (masks[i]) my_first = wbase + i;
            const uint32_t holders = __ballot_sync(0xFFFFFFFFu, n_mine != 0);
            const uint32_t later = holders & (0xFFFFFFFEu << lane);
            first_word = __shfl_sync(0xFFFFFFFFu, my_first, __ffs(holders) - 1);
            uint32_t link = __shfl_sync(0xFFFFFFFFu, my_first, __ffs(later ? later : holders) - 1);
            uint32_t next_of[kMaskWords];
#pragma unroll
            for (int i = kMaskWords - 1; i >= 0; --i) {
                next_of[i] = link;
                if (masks[i]) link = wbase + i;
            }
            uint32_t before = incl - n_mine;
            if (kMaskWords == 4) {
                uint32_t y[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    y[i] = (before << 16) | next_of[i % kMaskWords];
                    before += __popc(masks[i % kMaskWords]);
                }
                uint4* t4 = reinterpret_cast<uint4*>(table + wbase);
                t4[0] = make_uint4(masks[0], y[0], masks[1 % kMaskWords], y[1]);
                t4[1] = make_uint4(masks[2 % kMaskWords], y[2], masks[3 % kMaskWords], y[3]);
            } else {
#pragma unroll
                for (int i = 0; i < kMaskWords; ++i) {
                    table[wbase + i] = make_uint2(masks[i], (before << 16) | next_of[i]);
                    before += __popc(masks[i]);
                }
            }
        }
        __syncwarp();
        // the rest runs over the slots a lane holds, instantiated for the slot counts rows mostly need (see the bf16
        // kernel in mp_pack.cu); only for rows of up to 2048 columns (4 to 8 % faster there; at 4096 columns the
        // three copies made the kernel 70 % slower)
        const uint32_t per_lane = (n_cand + 31u) >> 5;
        auto finish_row = [&](auto trips_tag) {
            constexpr uint32_t kTrips = decltype(trips_tag)::value;
            uint32_t ent_val[kTrips];      // the candidate's 32 bits (0: unused slot, a key below every bound)
            uint32_t ent_col[kTrips];
            const uint32_t first = lane * per_lane;
            const uint32_t nvalid = first >= n_cand ? 0u : (n_cand - first < per_lane ? n_cand - first : per_lane);
            {
                uint32_t word = 0, m = 0, link = first_word;
                if (kMaskWords == 4) {
                    // the lane whose words hold rank `first`: the last one with (candidates before it) <= first, found
                    // by a binary search over the lanes' running counts (every lane takes part in the shuffles)
                    const uint32_t excl = incl - n_mine;
                    const uint32_t pc = __popc(masks[0]) | (__popc(masks[1 % kMaskWords]) << 8) | (__popc(masks[2 % kMaskWords]) << 16);
                    uint32_t owner = 0, owner_excl = 0;
#pragma unroll
                    for (int step = 16; step > 0; step >>= 1) {
                        const uint32_t v = __shfl_sync(0xFFFFFFFFu, excl, owner + step);
                        if (v <= first) {
                            owner += step;
                            owner_excl = v;
                        }
                    }
                    const uint32_t opc = __shfl_sync(0xFFFFFFFFu, pc, owner);
                    if (nvalid) {
                        const uint32_t r = first - owner_excl;          // rank inside the owner's four words
                        const uint32_t p0 = opc & 0xFFu, p01 = p0 + ((opc >> 8) & 0xFFu), p012 = p01 + (opc >> 16);
                        const uint32_t i = (r >= p0 ? 1u : 0u) + (r >= p01 ? 1u : 0u) + (r >= p012 ? 1u : 0u);
                        const uint2 e = table[owner * 4u + i];
                        word = owner * 4u + i;
                        m = e.x;
                        link = e.y & 0xFFFFu;
                        for (uint32_t skip = r - (i == 0 ? 0u : (i == 1 ? p0 : (i == 2 ? p01 : p012))); skip; --skip) m &= m - 1;
                    }
                } else if (nvalid) {
                    uint32_t lo = 0, hi = Lay::kTableWords - 1;
                    const uint32_t limit = (first + 1u) << 16;
                    while (lo < hi) {
                        const uint32_t mid = (lo + hi + 1) >> 1;
                        if (table[mid].y < limit) lo = mid; else hi = mid - 1;
                    }
                    const uint2 e = table[lo];
                    word = lo;
                    m = e.x;
                    link = e.y & 0xFFFFu;
                    for (uint32_t skip = first - (e.y >> 16); skip; --skip) m &= m - 1;
                }
                uint2 ahead = table[link];
                const uint32_t table_addr = smem_addr(table);
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const bool advance = (m == 0);
                    m = advance ? ahead.x : m;
                    word = advance ? link : word;
                    link = advance ? (ahead.y & 0xFFFFu) : link;
                    lds64_if(ahead, table_addr + link * 8u, advance);
                    const uint32_t col = word * 32u + (__ffs(m) - 1);
                    m &= m - 1;
                    const uint32_t v = reinterpret_cast<const uint32_t*>(base)[col];
                    const bool live = static_cast<uint32_t>(i) < nvalid;
                    ent_val[i] = live ? v : 0u;
                    ent_col[i] = live ? col : 0u;
                }
            }
            release_row();

            // ---- D: the 15-bit bucket of tau_i and how many of its members are kept -------------------------
            uint32_t tau15 = 0, take15 = 0;
            bool found = false;
            {
                const uint32_t drop = n_cand - k;                 // candidates to discard, smallest first
                hist[lane] = 0;
                hist[lane + 32] = 0;
                hist[lane + 64] = 0;
                __syncwarp();
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t rel = ((ent_val[i] >> 16) & 0x7FFFu) - low;
                    atomicAdd(&hist[rel < 64u ? rel : 64u + lane], 1u);
                }
                __syncwarp();
                const uint2 h = reinterpret_cast<const uint2*>(hist)[lane];   // lane owns bins 2 lane, 2 lane + 1
                const uint32_t own = h.x + h.y;
                const uint32_t before = warp_inclusive_sum(own) - own;
                uint32_t my_tau = 0xFFFFFFFFu, my_take = 0;
                if (before <= drop && drop < before + h.x) {
                    my_tau = low + 2u * lane;
                    my_take = h.x - (drop - before);
                } else if (before + h.x <= drop && drop < before + own) {
                    my_tau = low + 2u * lane + 1u;
                    my_take = h.y - (drop - before - h.x);
                }
                const uint32_t who = __ballot_sync(0xFFFFFFFFu, my_tau != 0xFFFFFFFFu);
                if (who) {
                    const int src = __ffs(who) - 1;
                    tau15 = __shfl_sync(0xFFFFFFFFu, my_tau, src);
                    take15 = __shfl_sync(0xFFFFFFFFu, my_take, src);
                    found = true;
                }
                __syncwarp();
            }
            if (!found) {
                // general case: radix select over the candidates' upper 15 bits, exponent byte then mantissa
                uint32_t k_rem = k;
                reinterpret_cast<uint4*>(hist)[lane] = make_uint4(0, 0, 0, 0);
                reinterpret_cast<uint4*>(hist)[lane + 32] = make_uint4(0, 0, 0, 0);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i)
                    if (static_cast<uint32_t>(i) < nvalid) atomicAdd(&hist[(ent_val[i] >> 23) & 0xFFu], 1u);
                __syncwarp();
                const uint32_t exp_bin = pick_exponent(hist, row_max >> 7, k_rem);
                __syncwarp();
                reinterpret_cast<uint4*>(hist)[lane] = make_uint4(0, 0, 0, 0);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t key15 = (ent_val[i] >> 16) & 0x7FFFu;
                    if (static_cast<uint32_t>(i) < nvalid && (key15 >> 7) == exp_bin) atomicAdd(&hist[key15 & 0x7Fu], 1u);
                }
                __syncwarp();
                tau15 = (exp_bin << 7) | pick_mantissa(hist, k_rem, take15);
                __syncwarp();
            }
            guess_low = tau15 > kGuessMargin ? tau15 - kGuessMargin : 0u;
            if (lane == 0) *reinterpret_cast<volatile uint32_t*>(&s_hint) = guess_low;

            // ---- D': exact tau_i among the members of that bucket: the take15-th largest full key ------------
            uint32_t tau_key = 0, take = 0;
            {
                uint32_t* n_members = scratch;                 // the histogram is dead
                uint32_t* members = scratch + 1;
                if (lane == 0) *n_members = 0;
                __syncwarp();
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t key = ent_val[i] & 0x7FFFFFFFu;
                    if ((key >> 16) == tau15) {
                        const uint32_t slot = atomicAdd(n_members, 1u);
                        if (slot < kMaxMembers) members[slot] = key;
                    }
                }
                __syncwarp();
                const uint32_t n_mem = *n_members;             // >= take15 >= 1
                if (n_mem <= kMaxMembers) {
                    // lane j ranks members j and j + 32 among all of them
                    for (uint32_t j = lane; j < ((n_mem + 31u) & ~31u); j += 32) {
                        const bool have = j < n_mem;
                        const uint32_t mine = have ? members[j] : 0u;
                        uint32_t greater = 0, equal = 0;
                        for (uint32_t i = 0; i < n_mem; ++i) {
                            const uint32_t other = members[i];
                            greater += other > mine ? 1u : 0u;
                            equal += other == mine ? 1u : 0u;
                        }
                        const uint32_t hit = __ballot_sync(0xFFFFFFFFu, have && greater < take15 && take15 <= greater + equal);
                        if (hit) {
                            const int src = __ffs(hit) - 1;
                            tau_key = __shfl_sync(0xFFFFFFFFu, mine, src);
                            take = take15 - __shfl_sync(0xFFFFFFFFu, greater, src);
                        }
                    }
                } else {
                    // many members (ties, coarse data): the take15-th largest, bit by bit over the lower 16 bits
                    uint32_t prefix = tau15 << 16;
#pragma unroll 1
                    for (int bit = 15; bit >= 0; --bit) {
                        const uint32_t trial = prefix | (1u << bit);
                        uint32_t cnt = 0;
#pragma unroll
                        for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                            const uint32_t key = ent_val[i] & 0x7FFFFFFFu;
                            cnt += ((key >> 16) == tau15 && key >= trial) ? 1u : 0u;
                        }
                        if (__reduce_add_sync(0xFFFFFFFFu, cnt) >= take15) prefix = trial;
                    }
                    tau_key = prefix;
                    uint32_t above = 0;
#pragma unroll
                    for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                        const uint32_t key = ent_val[i] & 0x7FFFFFFFu;
                        above += ((key >> 16) == tau15 && key > tau_key) ? 1u : 0u;
                    }
                    take = take15 - __reduce_add_sync(0xFFFFFFFFu, above);
                }
            }
            if (lane == 0 && tau_out) tau_out[row] = tau_key;

            // ---- E: ordered emit ------------------------------------------------------------------------
            __syncwarp();                                         // the member list is dead: its words become the stage
            {
                uint32_t counts = 0;                              // (gt << 16) | eq of this lane's entries
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t key = ent_val[i] & 0x7FFFFFFFu;
                    counts += key > tau_key ? 0x10000u : (key == tau_key ? 1u : 0u);
                }
                const uint32_t before = warp_inclusive_sum(counts) - counts;
                uint32_t e_at = before & 0xFFFFu;                 // ties before this entry
                uint32_t pos = (before >> 16) + (e_at < take ? e_at : take);   // kept entries before it
#pragma unroll
                for (int i = 0; i < static_cast<int>(kTrips); ++i) {
                    const uint32_t key = ent_val[i] & 0x7FFFFFFFu;
                    const bool is_eq = key == tau_key;
                    const bool keep = key > tau_key || (is_eq && e_at < take);
                    if (keep) {
                        stage_col[pos] = ent_col[i];
                        stage_val[pos] = ent_val[i];
                    }
                    pos += keep ? 1u : 0u;
                    e_at += is_eq ? 1u : 0u;
                }
            }
            __syncwarp();
            for (uint32_t p = lane; p < k; p += 32) {
                cols_out[out_base + p] = static_cast<int16_t>(stage_col[p]);
                vals_out[out_base + p] = stage_val[p];
                if (rows_out) rows_out[out_base + p] = static_cast<int32_t>(row);
            }
            __syncwarp();
        };
        if constexpr (E8 <= 8) {
            if (per_lane <= FwdTrips<PL>::kFew)
                finish_row(std::integral_constant<uint32_t, FwdTrips<PL>::kFew>{});
            else if (per_lane <= FwdTrips<PL>::kSome)
                finish_row(std::integral_constant<uint32_t, FwdTrips<PL>::kSome>{});
            else
                finish_row(std::integral_constant<uint32_t, PL>{});
        } else {
            finish_row(std::integral_constant<uint32_t, PL>{});
        }
    }
    chain_release_next();           // no row left for this warp: the next kernel may be scheduled as this one's CTAs retire
}

template <int E8, int PL>
dct_status_t launch_variant(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                            void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result,
                            cudaStream_t stream) {
    using Lay = RowLayoutF32<E8>;
    auto kernel = mp_topk_fwd_f32_warp_kernel<E8, PL>;
    constexpr int kMaxWarps = fwd_f32_max_warps<E8, PL>();
    constexpr size_t kSmemBudget = 220 * 1024;            // of the 227 KiB a CTA may use
    static thread_local int configured_device = -1;
    int dev = 0;
    DCT_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        DCT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(kSmemBudget)));
        configured_device = dev;
    }
    const size_t per_warp = Lay::warp_bytes(k);
    size_t warps = kSmemBudget / per_warp;                 // one CTA per SM with as many row slots as fit
    if (warps > static_cast<size_t>(kMaxWarps)) warps = kMaxWarps;
    if (warps < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    warps = warps_for_rows(warps, rows, sms);
    const uint64_t ctas_needed = (static_cast<uint64_t>(rows) + warps - 1) / warps;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < static_cast<uint64_t>(sms) ? ctas_needed : sms);
    DCT_CUDA_TRY(launch_chained_smem(kernel, grid, static_cast<unsigned>(warps * 32), warps * per_warp, stream,
                                     static_cast<const uint32_t*>(x_act), rows, d, ld, k, cols_out,
                                     static_cast<uint32_t*>(vals_out), rows_out, static_cast<uint32_t*>(tau_out), result));
    return DCT_OK;
}

template <int E8>
dct_status_t launch_width(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                          void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result, cudaStream_t stream) {
    const int per_lane = fwd_candidates_per_lane(d, k);
    if constexpr (E8 <= 4) {
        if (per_lane == 5)
            return launch_variant<E8, 5>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    }
    if (per_lane == 10)
        return launch_variant<E8, 10>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
    return launch_variant<E8, 20>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream);
}

// ------------------------------------------------------------------------------------------
// fp32, dense k (up to half the row): one warp per row
// ------------------------------------------------------------------------------------------
// As the dense bf16 kernel (mp_pack.cu), on the upper 15 key bits: two bit tables, upper bits >= low and
// >= low + 64, pin the 15-bit bucket of tau_i inside a 64-bucket window; a 64-bin histogram of the window
// elements gives the bucket and how many of its members are kept; the members (a handful) are ranked by
// their full keys, which gives the exact 31-bit tau_i and the ties to keep; then every lane walks its
// candidate bits in column order and keeps what the full key says.  Kept entries go through staging slots
// (16-bit column, 32-bit value) to coalesced stores.
constexpr uint32_t kDenseWindowF32 = 64;
constexpr uint32_t kDenseMaxKF32 = 1280;
constexpr int kDenseMaxWarpsF32 = 32;
constexpr int kDenseRetriesF32 = 6;

template <int E8> struct DenseLayoutF32 {
    using Row = RowLayoutF32<E8>;
    static constexpr uint32_t kTabWords = 128;
    // per warp: row | low table | high table | histogram (64) + member list (1 + 64) | staged values (k) | staged columns (k/2) | mbarrier
    __host__ __device__ static constexpr uint32_t kpad(uint32_t k) { return (k + 7u) & ~7u; }   // keeps every part a multiple of 16 bytes
    __host__ __device__ static constexpr uint32_t scratch_words(uint32_t k) {
        return 2u * kTabWords + 64u + 68u + kpad(k) + kpad(k) / 2u;
    }
    __host__ __device__ static constexpr uint32_t warp_bytes(uint32_t k) { return Row::kRowBytes + scratch_words(k) * 4u + 16u; }
};

template <int E8>
__global__ void __launch_bounds__(kDenseMaxWarpsF32 * 32)
mp_topk_fwd_f32_dense_kernel(const uint32_t* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                             int16_t* __restrict__ cols_out, uint32_t* __restrict__ vals_out,
                             int32_t* __restrict__ rows_out, uint32_t* __restrict__ tau_out,
                             dct_result_t* __restrict__ result) {
    using Lay = RowLayoutF32<E8>;
    using Den = DenseLayoutF32<E8>;
    constexpr int kMaskWords = Lay::kMaskWords;
    constexpr uint32_t kGuessMargin = 32;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned char* base = smem_raw + warp * Den::warp_bytes(k);
    unsigned char* span = base + lane * (Lay::E * 4u);
    uint32_t* scratch = reinterpret_cast<uint32_t*>(base + Lay::kRowBytes);
    uint32_t* tab_low = scratch;
    uint32_t* tab_high = scratch + Den::kTabWords;
    uint32_t* hist = scratch + 2u * Den::kTabWords;            // 64 bins
    uint32_t* n_members = hist + 64;                           // 1 word, then up to 64 member keys
    uint32_t* members = n_members + 1;
    uint32_t* stage_val = hist + 64 + 68;
    uint16_t* stage_col = reinterpret_cast<uint16_t*>(stage_val + Den::kpad(k));
    uint64_t* bar = reinterpret_cast<uint64_t*>(scratch + Den::scratch_words(k));
    const uint32_t* row32 = reinterpret_cast<const uint32_t*>(base);
    __shared__ uint32_t s_stop;
    __shared__ uint32_t s_next;                               // rows of this CTA handed out so far

    if (threadIdx.x == 0) {
        s_stop = 0;
        s_next = blockDim.x >> 5;
    }
    if (lane == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
        fence_proxy_async_all();
    }
    const uint32_t row_bytes = d * 4u;                         // the tail of the buffer stays zero
    for (uint32_t b = row_bytes + lane * 16u; b < Lay::kRowBytes; b += 512u)
        *reinterpret_cast<uint4*>(base + b) = make_uint4(0, 0, 0, 0);
    __syncthreads();
    chain_wait_previous();          // set-up above; inputs and outputs only below (see the bf16 kernel in mp_pack.cu)
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }

    const uint32_t warp_global = blockIdx.x + gridDim.x * warp;
    auto request_row = [&](uint32_t r) {
        if (lane == 0) {
            mbar_arrive_expect_tx(bar, row_bytes);
            bulk_load(base, x + static_cast<size_t>(r) * ld, row_bytes, bar);
        }
    };
    uint64_t next_row = 0;
    auto release_row = [&]() {               // the row buffer is no longer needed: request the CTA's next row
        __syncwarp();
        fence_proxy_async_smem();
        uint32_t j = 0;
        if (lane == 0) j = atomicAdd(&s_next, 1u);
        j = __shfl_sync(0xFFFFFFFFu, j, 0);
        next_row = blockIdx.x + static_cast<uint64_t>(gridDim.x) * j;
        if (next_row < rows) request_row(static_cast<uint32_t>(next_row));
    };
    // 32-byte pieces (8 columns, one table byte), halves read in a lane-dependent order: see the sparse kernel
    const uint32_t swap = (lane >> 2) & 1u;
    const unsigned char* piece_first = base + lane * 32u + swap * 16u;
    const unsigned char* piece_second = base + lane * 32u + (swap ^ 1u) * 16u;
    const uint32_t w_first = swap ? 0x80C0E0F0u : 0xF8FCFEFFu;      // dot-product weights -2^j of the columns a read holds
    const uint32_t w_second = swap ? 0xF8FCFEFFu : 0x80C0E0F0u;
    if (warp_global < rows) request_row(warp_global);

    uint32_t use = 0;
    uint32_t guess_low = 0;
    for (uint64_t row64 = warp_global; row64 < rows; row64 = next_row, ++use) {
        const uint32_t row = static_cast<uint32_t>(row64);
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(bar, use & 1u, 1u << 24, &s_stop))) {
            s_stop = 1;
            if (lane == 0 && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
            return;
        }
        const size_t out_base = static_cast<size_t>(row) * k;

        // ---- A: bounds around the upper 15 bits of tau_i ------------------------------------------------
        uint32_t low = guess_low;
        if (low == 0) {
            // no previous row: a conservative (k/d)-quantile of up to 128 samples (column 0 of up to four pieces)
            constexpr int kSamples = E8 < 4 ? E8 : 4;
            uint32_t sample[kSamples];
#pragma unroll
            for (int c = 0; c < kSamples; ++c)
                sample[c] = (*reinterpret_cast<const uint32_t*>(base + lane * 32u + c * 1024) >> 16) & 0x7FFFu;
            const uint32_t n_samples = 32u * kSamples;
            uint32_t rank = (n_samples * k + d - 1) / d;
            rank += 2u * static_cast<uint32_t>(__fsqrt_rn(static_cast<float>(rank))) + 2u;
            if (rank > n_samples) rank = n_samples;
#pragma unroll 1
            for (int bit = 14; bit >= 0; --bit) {
                const uint32_t trial = low | (1u << bit);
                uint32_t cnt = 0;
#pragma unroll
                for (int c = 0; c < kSamples; ++c) cnt += sample[c] >= trial ? 1u : 0u;
                if (__reduce_add_sync(0xFFFFFFFFu, cnt) >= rank) low = trial;
            }
            if (low == 0) low = 1;
        }
        uint32_t geL[kMaskWords], geH[kMaskWords];
        uint32_t n_low = 0, n_high = 0, before_packed = 0;
        bool pinned = false;
        uint32_t step = kDenseWindowF32;
        int last_move = 0;
#pragma unroll 1
        for (int attempt = 0; attempt < kDenseRetriesF32; ++attempt) {
            const uint32_t high = low + kDenseWindowF32;
            unsigned char* tl = reinterpret_cast<unsigned char*>(tab_low) + lane;
            unsigned char* th = reinterpret_cast<unsigned char*>(tab_high) + lane;
            __syncwarp();
            {
                const uint32_t low2 = low * 0x10001u, high2 = high * 0x10001u;
#pragma unroll
                for (int c = 0; c < E8; ++c) {
                    const uint4 a = *reinterpret_cast<const uint4*>(piece_first + c * 1024);
                    const uint4 b = *reinterpret_cast<const uint4*>(piece_second + c * 1024);
                    tl[c * 32] = static_cast<unsigned char>(piece_flags(a, b, low2, w_first, w_second));
                    th[c * 32] = static_cast<unsigned char>(piece_flags(a, b, high2, w_first, w_second));
                }
            }
            __syncwarp();
            uint32_t mine = 0;
#pragma unroll
            for (int i = 0; i < kMaskWords; ++i) {
                const uint32_t w = lane * kMaskWords + i;
                const bool real = Lay::kRowWords == Lay::kTableWords || w < Lay::kRowWords;
                geL[i] = real ? tab_low[w] : 0u;
                geH[i] = real ? tab_high[w] : 0u;
                mine += (__popc(geL[i]) << 16) | __popc(geH[i]);
            }
            const uint32_t incl = warp_inclusive_sum(mine);
            const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
            n_low = total >> 16;
            n_high = total & 0xFFFFu;
            before_packed = incl - mine;
            if (n_high < k && k <= n_low) {
                pinned = true;
                break;
            }
            const int move = n_low < k ? -1 : 1;
            if (attempt > 0) step = (move == last_move) ? step * 2u : (step > kDenseWindowF32 ? step / 2u : kDenseWindowF32);
            last_move = move;
            if (move < 0) {
                if (low == 1) break;
                low = low > step ? low - step : 1u;
            } else {
                low = low + step < 0x7F80u ? low + step : 0x7F80u;
            }
        }
        if (!pinned) {
            mp_row_slow_path_f32<E8>(span, k, out_base, row, cols_out, vals_out, rows_out, tau_out);
            release_row();
            continue;
        }

        // ---- B: the bucket of tau_i, then tau_i among its members ------------------------------------------
        hist[lane] = 0;
        hist[lane + 32] = 0;
        if (lane == 0) *n_members = 0;
        __syncwarp();
#pragma unroll
        for (int i = 0; i < kMaskWords; ++i) {
            uint32_t m = geL[i] & ~geH[i];
            const uint32_t col0 = (lane * kMaskWords + i) * 32u;
            while (m) {
                const uint32_t col = col0 + (__ffs(m) - 1);
                m &= m - 1;
                atomicAdd(&hist[(((row32[col] >> 16) & 0x7FFFu) - low) & 63u], 1u);
            }
        }
        __syncwarp();
        uint32_t tau15, take15;
        {
            const uint32_t drop = n_low - k;
            const uint2 h = reinterpret_cast<const uint2*>(hist)[lane];
            const uint32_t own = h.x + h.y;
            const uint32_t before = warp_inclusive_sum(own) - own;
            uint32_t my_tau = 0, my_take = 0;
            bool mine = false;
            if (before <= drop && drop < before + h.x) {
                mine = true;
                my_tau = low + 2u * lane;
                my_take = h.x - (drop - before);
            } else if (before + h.x <= drop && drop < before + own) {
                mine = true;
                my_tau = low + 2u * lane + 1u;
                my_take = h.y - (drop - before - h.x);
            }
            const uint32_t who = __ballot_sync(0xFFFFFFFFu, mine);
            const int src = who ? __ffs(who) - 1 : 0;
            tau15 = __shfl_sync(0xFFFFFFFFu, my_tau, src);
            take15 = __shfl_sync(0xFFFFFFFFu, my_take, src);
        }
        guess_low = tau15 > kGuessMargin ? tau15 - kGuessMargin : 1u;
        // members of the bucket: full keys into the list
#pragma unroll
        for (int i = 0; i < kMaskWords; ++i) {
            uint32_t m = geL[i] & ~geH[i];
            const uint32_t col0 = (lane * kMaskWords + i) * 32u;
            while (m) {
                const uint32_t col = col0 + (__ffs(m) - 1);
                m &= m - 1;
                const uint32_t key = row32[col] & 0x7FFFFFFFu;
                if ((key >> 16) == tau15) {
                    const uint32_t slot = atomicAdd(n_members, 1u);
                    if (slot < 64u) members[slot] = key;
                }
            }
        }
        __syncwarp();
        const uint32_t n_mem = *n_members;
        if (n_mem > 64u) {                                     // too many to rank here (coarse or tied data)
            mp_row_slow_path_f32<E8>(span, k, out_base, row, cols_out, vals_out, rows_out, tau_out);
            release_row();
            continue;
        }
        uint32_t tau_key = 0, take = 0;
        for (uint32_t j = lane; j < ((n_mem + 31u) & ~31u); j += 32) {
            const bool have = j < n_mem;
            const uint32_t mine = have ? members[j] : 0u;
            uint32_t greater = 0, equal = 0;
            for (uint32_t i = 0; i < n_mem; ++i) {
                const uint32_t other = members[i];
                greater += other > mine ? 1u : 0u;
                equal += other == mine ? 1u : 0u;
            }
            const uint32_t hit = __ballot_sync(0xFFFFFFFFu, have && greater < take15 && take15 <= greater + equal);
            if (hit) {
                const int src = __ffs(hit) - 1;
                tau_key = __shfl_sync(0xFFFFFFFFu, mine, src);
                take = take15 - __shfl_sync(0xFFFFFFFFu, greater, src);
            }
        }
        if (lane == 0 && tau_out) tau_out[row] = tau_key;

        // ---- C: ordered emit ------------------------------------------------------------------------
        uint32_t counts = (before_packed & 0xFFFFu) << 16;         // kept for sure (high table) before this lane
        {
            uint32_t mine = 0;                                     // (window elements > tau << 16) | window elements == tau
#pragma unroll
            for (int i = 0; i < kMaskWords; ++i) {
                uint32_t m = geL[i] & ~geH[i];
                const uint32_t col0 = (lane * kMaskWords + i) * 32u;
                while (m) {
                    const uint32_t col = col0 + (__ffs(m) - 1);
                    m &= m - 1;
                    const uint32_t key = row32[col] & 0x7FFFFFFFu;
                    mine += key > tau_key ? 0x10000u : (key == tau_key ? 1u : 0u);
                }
            }
            counts += warp_inclusive_sum(mine) - mine;
        }
        {
            uint32_t e_at = counts & 0xFFFFu;
            uint32_t pos = (counts >> 16) + (e_at < take ? e_at : take);
#pragma unroll
            for (int i = 0; i < kMaskWords; ++i) {
                uint32_t m = geL[i];
                const uint32_t col0 = (lane * kMaskWords + i) * 32u;
                while (m) {
                    const uint32_t col = col0 + (__ffs(m) - 1);
                    m &= m - 1;
                    const uint32_t v = row32[col];
                    const uint32_t key = v & 0x7FFFFFFFu;
                    const bool is_eq = key == tau_key;
                    const bool keep = key > tau_key || (is_eq && e_at < take);
                    if (keep) {
                        stage_val[pos] = v;
                        stage_col[pos] = static_cast<uint16_t>(col);
                    }
                    pos += keep ? 1u : 0u;
                    e_at += is_eq ? 1u : 0u;
                }
            }
        }
        release_row();
        for (uint32_t p = lane; p < k; p += 32) {
            cols_out[out_base + p] = static_cast<int16_t>(stage_col[p]);
            vals_out[out_base + p] = stage_val[p];
            if (rows_out) rows_out[out_base + p] = static_cast<int32_t>(row);
        }
        __syncwarp();
    }
    chain_release_next();           // no row left for this warp
}

template <int E8>
dct_status_t launch_dense(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                          void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result, cudaStream_t stream) {
    using Den = DenseLayoutF32<E8>;
    auto kernel = mp_topk_fwd_f32_dense_kernel<E8>;
    constexpr size_t kSmemBudget = 220 * 1024;
    static thread_local int configured_device = -1;
    int dev = 0;
    DCT_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        DCT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(kSmemBudget)));
        configured_device = dev;
    }
    const size_t per_warp = Den::warp_bytes(k);
    size_t warps = kSmemBudget / per_warp;
    if (warps > static_cast<size_t>(kDenseMaxWarpsF32)) warps = kDenseMaxWarpsF32;
    if (warps < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    warps = warps_for_rows(warps, rows, sms);
    const uint64_t ctas_needed = (static_cast<uint64_t>(rows) + warps - 1) / warps;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < static_cast<uint64_t>(sms) ? ctas_needed : sms);
    DCT_CUDA_TRY(launch_chained_smem(kernel, grid, static_cast<unsigned>(warps * 32), warps * per_warp, stream,
                                     static_cast<const uint32_t*>(x_act), rows, d, ld, k, cols_out,
                                     static_cast<uint32_t*>(vals_out), rows_out, static_cast<uint32_t*>(tau_out), result));
    return DCT_OK;
}

}  // namespace

// *handled = false: the shape is not one of the fast path's; the caller runs the general kernel.
dct_status_t launch_fwd_f32_warp(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                 int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                 dct_result_t* result, cudaStream_t stream, bool* handled) {
    *handled = false;
    if (!aligned_to(x_act, 16) || (static_cast<size_t>(ld) * 4) % 16 != 0 || d % 4 != 0 || d > 4096) return DCT_OK;
    if (fwd_candidates_per_lane(d, k) == 0) {
        // dense k (beyond the candidate registers, up to half the row) on rows of up to 512 columns: bounds + bit
        // tables.  (From 513 columns on the CTA-per-row kernel of mp_pack_f32_wide.cu is 1.5 to 2.4 times faster up
        // to k = 3d/8, and beyond that the general kernel is: 65536x1024, k = 512: 0.49 against 2.05 ms.)
        if (k > kDenseMaxKF32 || k > d / 2 || d > 512) return DCT_OK;
        *handled = true;
#define DCT_F32_DENSE(E8) \
    if (d <= 256u * E8)   \
        return launch_dense<E8>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream)
        DCT_F32_DENSE(1);
        DCT_F32_DENSE(2);
#undef DCT_F32_DENSE
        *handled = false;
        return DCT_OK;
    }
    *handled = true;
#define DCT_F32_WIDTH(E8) \
    if (d <= 256u * E8)   \
        return launch_width<E8>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream)
    // the smallest instantiated buffer of 256 * E8 columns that holds the row
    DCT_F32_WIDTH(1);
    DCT_F32_WIDTH(2);
    DCT_F32_WIDTH(3);
    DCT_F32_WIDTH(4);
    DCT_F32_WIDTH(5);
    DCT_F32_WIDTH(6);
    DCT_F32_WIDTH(7);
    DCT_F32_WIDTH(8);
    DCT_F32_WIDTH(10);
    DCT_F32_WIDTH(12);
    DCT_F32_WIDTH(14);
    DCT_F32_WIDTH(16);
#undef DCT_F32_WIDTH
    *handled = false;
    return DCT_OK;
}

}  // namespace dct
