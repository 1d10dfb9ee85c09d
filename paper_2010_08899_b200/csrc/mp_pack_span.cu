// dct_mp_topk_pack_fwd, bf16, k from about a tenth to 3/8 of the row (the 75 % sparsity level of the paper's DCT-MP
// tables and the denser part of its 90 % level), rows of up to 3072 columns on 16-byte boundaries: Algorithm 2 (DCT-MP), forward pass -- one warp
// per row, every lane looking after one contiguous span of the row.
//
// The row arrives by one bulk copy (TMA engine) into shared memory exactly as it lies in HBM.  Lane l owns the
// columns [l E, (l + 1) E), E = d_buffer / 32, so "column order" is "lane order, then bit order inside the lane":
// every lane can write its own kept entries, in order, at an offset that one warp scan provides.
//   A  two bounds around tau_i, low and high = low + window: low is the previous row's tau_i minus half a window
//      (a warp without a previous row borrows the latest of its CTA, or takes a quantile of 128 samples of the row).
//   B  one pass over the lane's own 16-byte units gives two flags per column, key >= low and key >= high, as 2 E
//      bits in registers.  Exact integer compares; the 8 flags of a unit come out of a byte permutation and two
//      dot-product instructions.  The units are read in a lane-dependent (XOR-swizzled) order so that the 128-bit
//      shared-memory reads of a quarter warp fall into different banks although the lanes' spans are a multiple of
//      128 bytes apart; a byte permutation puts the flags back in column order.  If the counts satisfy
//      n_high < k <= n_low, tau_i lies inside the window; otherwise the window moves and the pass is repeated.
//   C  the elements inside the window (a few per lane) are read one by one: their keys go into a histogram, which
//      gives tau_i and the number of ties to keep, and into a short list per lane, from which the lane then adds
//      the window elements above tau_i and its share of the ties (lowest columns first) to its `high` flags:
//      the kept columns of its span, as bits.
//   D  one warp scan over the kept counts gives every lane its offset in the row's output; the lane walks its
//      kept bits and stages {column, value} in shared memory.
//   E  the staged entries leave in pairs, as 4-byte stores to either output (the staging index is shifted by the
//      parity of the row's first output element), while the row buffer already receives the warp's next row.
// A row with fewer than k non-zeros (tau_i = 0) keeps its non-zeros and fills up with its first zeros.  Rows for
// which the window does not settle take the bit-serial slow path of mp_warp.cuh.  The result never depends on the
// guesses.
#include "common.cuh"
#include "mp_warp.cuh"

namespace dct {
namespace {

constexpr int gcd8(int e8) { return (e8 % 8 == 0) ? 8 : (e8 % 4 == 0) ? 4 : (e8 % 2 == 0) ? 2 : 1; }
constexpr uint32_t kSpanMaxK = 2048;             // staging: 2 x 2 bytes per kept entry
constexpr uint32_t kSpanWindow = 64;             // widest window, in keys (= histogram bins)
constexpr uint32_t kSpanListLen = 24;            // window elements a lane can take
constexpr uint32_t kSpanListStride = 25;         // words between the lanes' lists (odd: no bank conflicts)
constexpr int kSpanRetries = 8;
template <int E8> constexpr int span_max_warps() { return E8 <= 2 ? 32 : 24; }   // (narrow rows need few registers)

template <int E8> struct SpanLayout {
    static constexpr uint32_t E = E8 * 8u;                  // columns per lane
    static constexpr uint32_t kSpanBytes = E8 * 16u;        // bytes per lane
    static constexpr uint32_t kRowBytes = 32u * kSpanBytes;
    static constexpr int kWords = (E8 + 3) / 4;             // 32-bit flag words per lane
    static constexpr int kGroup = gcd8(E8);                 // units whose read order is swizzled among themselves
    static constexpr uint32_t kHistBytes = 128u * 4u;       // 64 bins (+ padding)
    static constexpr uint32_t kListBytes = 32u * kSpanListStride * 4u;
    // per warp: row | histogram | window lists / staging (the same bytes, one after the other).  A multiple of 128
    // bytes, so that every row buffer starts on a 128-byte boundary (the swizzled reads rely on it).
    __host__ __device__ static constexpr uint32_t stage_bytes(uint32_t k) { return 2u * ((2u * (k + 8u) + 15u) & ~15u); }
    __host__ __device__ static constexpr uint32_t warp_bytes(uint32_t k) {
        const uint32_t u = kListBytes > stage_bytes(k) ? kListBytes : stage_bytes(k);
        return (kRowBytes + kHistBytes + u + 127u) & ~127u;
    }
};

// The flags key >= low and key >= high of the 8 bf16 of one 16-byte unit, element j at bit 7 - j (the walks over
// the flags run from the highest bit down, i.e. from the first column on).  Integer compares on the keys, exact for
// every bit pattern: per 16-bit half, bit 15 of ((x | 0x8000) - bound) is set iff key(x) >= bound, and no borrow
// crosses the halves (bound <= 0x8000).  low2 / high2 = the bound in both halves.
__device__ __forceinline__ void flags8_two(uint4 v, uint32_t low2, uint32_t high2, uint32_t& f_low, uint32_t& f_high) {
    const uint32_t x0 = v.x | 0x80008000u, x1 = v.y | 0x80008000u, x2 = v.z | 0x80008000u, x3 = v.w | 0x80008000u;
    // bytes 1, 3 of either word, the sign bit replicated over the byte: 0xFF (= -1) or 0 for elements 0..3 / 4..7;
    // (-1) * (-2^(7-j)) = 2^(7-j): two signed dot products add up the eight weights
    f_low = static_cast<uint32_t>(dp4a_ss(prmt(x2 - low2, x3 - low2, 0xFDB9u), 0xFFFEFCF8u,
                                          dp4a_ss(prmt(x0 - low2, x1 - low2, 0xFDB9u), 0xF0E0C080u, 0)));
    f_high = static_cast<uint32_t>(dp4a_ss(prmt(x2 - high2, x3 - high2, 0xFDB9u), 0xFFFEFCF8u,
                                           dp4a_ss(prmt(x0 - high2, x1 - high2, 0xFDB9u), 0xF0E0C080u, 0)));
}

template <int E8>
__global__ void __launch_bounds__(span_max_warps<E8>() * 32)
mp_topk_fwd_bf16_span_kernel(const uint16_t* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                             int16_t* __restrict__ cols_out, uint16_t* __restrict__ vals_out,
                             int32_t* __restrict__ rows_out, uint16_t* __restrict__ tau_out,
                             dct_result_t* __restrict__ result) {
    using Lay = SpanLayout<E8>;
    constexpr int kWords = Lay::kWords;
    constexpr int kGroup = Lay::kGroup;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned char* base = smem_raw + warp * Lay::warp_bytes(k);
    const unsigned char* own = base + lane * Lay::kSpanBytes;
    uint32_t* hist = reinterpret_cast<uint32_t*>(base + Lay::kRowBytes);
    uint32_t* lists = hist + Lay::kHistBytes / 4;              // window elements {position << 16 | key}, one list per lane
    uint32_t* stage = lists;                                   // the k kept entries {column << 16 | value} (after the lists)
    __shared__ uint64_t s_bar[32];                             // one mbarrier per warp: its row has arrived
    uint64_t* bar = &s_bar[warp];
    __shared__ uint32_t s_stop;
    __shared__ uint32_t s_next;                                // rows of this CTA handed out so far
    __shared__ uint32_t s_hint;                                // the latest low bound any warp of the CTA derived from a tau_i

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
    // A row of d <= 256 E8 columns (d a multiple of 8) fills the first d columns of the buffer; the rest is zeroed
    // once and never written again: zeros lie below every bound and, being the last columns, lose every tie.
    const uint32_t row_bytes = d * 2u;
    for (uint32_t b = row_bytes + lane * 16u; b < Lay::kRowBytes; b += 512u)
        *reinterpret_cast<uint4*>(base + b) = make_uint4(0, 0, 0, 0);
    __syncthreads();
    chain_wait_previous();          // set-up above; inputs and outputs only below (see the sparse kernel in mp_pack.cu)
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }

    // Read order of the lane's units: unit (c ^ swz) at step c, inside aligned groups of kGroup units.  The spans of
    // consecutive lanes are E8 * 16 bytes apart; the swizzle makes the 8 lanes of a quarter warp hit the 8 different
    // 16-byte bank groups at every step.
    const uint32_t swz = kGroup == 1 ? 0u : (lane / (8u / kGroup)) % kGroup;
    const uint32_t fix_sel = 0x3210u ^ (0x1111u * (swz & 3u));    // byte permutation that undoes the swizzle in a flag word
    uint32_t unit_base[kGroup];                              // address of the unit read at step c < kGroup
#pragma unroll
    for (int c = 0; c < kGroup; ++c) unit_base[c] = smem_addr(own) ^ (16u * (swz ^ static_cast<uint32_t>(c)));
    const uint32_t row_addr = smem_addr(base);

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
    if (warp_global < rows) request_row(warp_global);

    uint32_t use = 0;
    uint32_t guess_low = 0;
    // Width of the window in keys.  A wide window rarely misses tau_i, but every element inside it is looked at one
    // by one: it is halved (down to 16 keys) while rows find more than 96 elements in it, at once when a lane's list
    // would overflow, and doubled again when a row needs a second pass.
    uint32_t window = kSpanWindow;
    for (uint64_t row64 = warp_global; row64 < rows; row64 = next_row, ++use) {
        const uint32_t row = static_cast<uint32_t>(row64);
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(bar, use & 1u, 1u << 24, &s_stop))) {
            s_stop = 1;
            if (lane == 0 && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
            return;
        }
        const size_t out_base = static_cast<size_t>(row) * k;

        // ---- A: bounds around tau_i ------------------------------------------------------------------
        if (guess_low == 0) guess_low = *reinterpret_cast<volatile uint32_t*>(&s_hint);
        uint32_t low = guess_low;
        if (low == 0) {
            // no row behind this warp or its CTA: the (k/d)-quantile of up to 128 samples (the first element of up
            // to four units of every lane), taken a little low, found bit by bit
            constexpr int kSamples = E8 < 4 ? E8 : 4;
            uint32_t sample[kSamples];
#pragma unroll
            for (int c = 0; c < kSamples; ++c) sample[c] = *reinterpret_cast<const uint16_t*>(own + c * 16) & 0x7FFFu;
            const uint32_t n_samples = 32u * kSamples;
            uint32_t rank = (n_samples * k + d - 1) / d;                   // expected rank of tau_i among the samples
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
        if (low > 0x7F80u) low = 0x7F80u;

        // ---- B: two flags per column of the lane's span ---------------------------------------------------
        uint32_t ge_low[kWords], ge_high[kWords];
        uint32_t n_low = 0, n_high = 0;
        bool pinned = false, moved = false, crowded = false, tau_zero = false;
#pragma unroll 1
        for (int attempt = 0; attempt < kSpanRetries; ++attempt) {
            const uint32_t high = low + window;                    // low <= 0x7F80: stays within the 2^15 keys
            const uint32_t low2 = low * 0x10001u, high2 = high * 0x10001u;
#pragma unroll
            for (int i = 0; i < kWords; ++i) ge_low[i] = ge_high[i] = 0;
            static_for<E8>([&](auto c_tag) {
                constexpr int c = decltype(c_tag)::value;
                uint32_t f_low, f_high;
                flags8_two(lds128<16 * kGroup * (c / kGroup)>(unit_base[c % kGroup]), low2, high2, f_low, f_high);
                // unit c (in read order) is byte 3 - c % 4 of word c / 4: column j of the word at bit 31 - j
                constexpr uint32_t sel = c % 4 == 1 ? 0x3410u : (c % 4 == 2 ? 0x3240u : 0x3214u);
                ge_low[c / 4] = (c % 4 == 0) ? (f_low << 24) : prmt(ge_low[c / 4], f_low, sel);
                ge_high[c / 4] = (c % 4 == 0) ? (f_high << 24) : prmt(ge_high[c / 4], f_high, sel);
            });
            // back to column order: unit (c ^ swz) was read at step c
            if (kGroup == 8) {
#pragma unroll
                for (int h = 0; h + 1 < kWords; h += 2) {
                    const uint32_t l0 = ge_low[h], l1 = ge_low[h + 1], h0 = ge_high[h], h1 = ge_high[h + 1];
                    ge_low[h] = (swz & 4u) ? l1 : l0;
                    ge_low[h + 1] = (swz & 4u) ? l0 : l1;
                    ge_high[h] = (swz & 4u) ? h1 : h0;
                    ge_high[h + 1] = (swz & 4u) ? h0 : h1;
                }
            }
            if (kGroup > 1) {
#pragma unroll
                for (int i = 0; i < kWords; ++i) {
                    ge_low[i] = prmt(ge_low[i], 0u, fix_sel);
                    ge_high[i] = prmt(ge_high[i], 0u, fix_sel);
                }
            }
            uint32_t mine = 0;
#pragma unroll
            for (int i = 0; i < kWords; ++i) mine += (__popc(ge_low[i]) << 16) | __popc(ge_high[i]);
            const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, mine);     // both counts stay below 2^16
            n_low = total >> 16;
            n_high = total & 0xFFFFu;
            if (n_high < k && k <= n_low) {
                const uint32_t in_window = (mine >> 16) - (mine & 0xFFFFu);
                if (__reduce_max_sync(0xFFFFFFFFu, in_window) <= kSpanListLen) {
                    pinned = true;
                    break;
                }
                if (window <= 8u) break;                           // cannot be narrowed further: slow path
                window >>= 1;                                      // a lane's list would overflow: same low, narrower window
                crowded = true;
                continue;
            }
            // Move the window to where the counts say tau_i is: the window holds n_low - n_high elements, i.e. so many
            // per key around here; tau_i lies (n_high - k) elements above high, or (k - n_low) below low.  The estimate
            // goes to the middle of the new window; a move never is shorter than half a window.
            const uint32_t per_key_x16 = max(((n_low - n_high) << 4) / window, 4u);        // elements per key, times 16
            moved = true;
            if (n_low < k) {
                if (low == 1) {                                    // tau_i = 0: the row has fewer than k non-zeros
                    tau_zero = true;
                    break;
                }
                const uint32_t below = max(((k - n_low) << 4) / per_key_x16 + window / 2u, window / 2u);
                low = low > below ? low - below : 1u;
            } else {
                const uint32_t above = ((n_high - k + 1u) << 4) / per_key_x16 + window / 2u;
                low = low + above < 0x7F80u ? low + above : 0x7F80u;
            }
        }
        uint32_t keep[kWords];                                 // the kept columns of the lane's span, as bits
        if (tau_zero) {
            // Every non-zero is kept (ge_low holds key >= 1 here), and the first k - n_low zeros in column order fill
            // the row's slots up; the padding columns behind the row are the last zeros and are never reached.
            const uint32_t fill = k - n_low;
            uint32_t zeros[kWords], n_zeros = 0;
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                const uint32_t valid = (E8 % 4 != 0 && i == kWords - 1) ? 0xFFFFFFFFu << (32 - 8 * (E8 % 4)) : 0xFFFFFFFFu;
                zeros[i] = ~ge_low[i] & valid;
                n_zeros += __popc(zeros[i]);
            }
            const uint32_t zeros_before = warp_inclusive_sum(n_zeros) - n_zeros;
            uint32_t room = zeros_before < fill ? fill - zeros_before : 0u;     // zeros this lane still takes
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t z = zeros[i];
                const uint32_t n = __popc(z);
                if (n > room) {
                    for (uint32_t extra = n - room; extra; --extra) z &= z - 1u;   // the highest columns go (lowest bits)
                    room = 0;
                } else {
                    room -= n;
                }
                keep[i] = ge_low[i] | z;
            }
            if (lane == 0 && tau_out) tau_out[row] = 0;
            guess_low = 0;
            __syncwarp();
        } else if (!pinned) {
            mp_row_slow_path<E8>(own, k, out_base, row, cols_out, vals_out, rows_out, tau_out);
            guess_low = 0;
            release_row();
            continue;
        } else {
            // ---- C: tau_i from the elements inside the window; the kept columns as bits ------------------------------
            hist[lane] = 0;
            hist[lane + 32] = 0;
            __syncwarp();                                          // (also: the previous row's staged output has been read)
            uint32_t* my_list = lists + lane * kSpanListStride;
            uint32_t n_list = 0;
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t m = ge_low[i] & ~ge_high[i];
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    const uint32_t col = lane * Lay::E + 32u * i + 31u - q;
                    uint32_t v;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(row_addr + 2u * col));
                    const uint32_t key = v & 0x7FFFu;
                    atomicAdd(&hist[key - low], 1u);               // low <= key < low + window <= low + 64
                    my_list[n_list++] = ((32u * i + q) << 16) | key;
                }
            }
            __syncwarp();
            uint32_t tau_key, take;
            {
                const uint32_t drop = n_low - k;                   // window elements to discard, smallest first
                const uint2 h = reinterpret_cast<const uint2*>(hist)[lane];   // lane owns bins 2 lane, 2 lane + 1
                const uint32_t own_cnt = h.x + h.y;
                const uint32_t before = warp_inclusive_sum(own_cnt) - own_cnt;
                uint32_t my_tau = 0, my_take = 0;
                bool mine = false;
                if (before <= drop && drop < before + h.x) {
                    mine = true;
                    my_tau = low + 2u * lane;
                    my_take = h.x - (drop - before);
                } else if (before + h.x <= drop && drop < before + own_cnt) {
                    mine = true;
                    my_tau = low + 2u * lane + 1u;
                    my_take = h.y - (drop - before - h.x);
                }
                const uint32_t who = __ballot_sync(0xFFFFFFFFu, mine);        // exactly one lane: n_high < k <= n_low
                const int src = who ? __ffs(who) - 1 : 0;
                tau_key = __shfl_sync(0xFFFFFFFFu, my_tau, src);
                take = __shfl_sync(0xFFFFFFFFu, my_take, src);
            }
            if (lane == 0 && tau_out) tau_out[row] = static_cast<uint16_t>(tau_key);
            if (crowded) {
                // the window stays narrow
            } else if (moved) {
                window = window < kSpanWindow ? window * 2u : kSpanWindow;
            } else if (n_low - n_high > 96u && window > 16u) {
                window >>= 1;
            }
            guess_low = tau_key > window / 2u ? tau_key - window / 2u : 1u;
            if (lane == 0) *reinterpret_cast<volatile uint32_t*>(&s_hint) = guess_low;

            // kept = above the window, plus the window elements above tau_i, plus the first `take` ties (the lists are in
            // column order, and so are the lanes)
#pragma unroll
            for (int i = 0; i < kWords; ++i) keep[i] = ge_high[i];
            {
                uint32_t n_ties = 0;
                for (uint32_t j = 0; j < n_list; ++j) n_ties += (my_list[j] & 0xFFFFu) == tau_key ? 1u : 0u;
                const uint32_t ties_before = warp_inclusive_sum(n_ties) - n_ties;
                uint32_t room = ties_before < take ? take - ties_before : 0u;   // ties this lane may still keep
                for (uint32_t j = 0; j < n_list; ++j) {
                    const uint32_t e = my_list[j];
                    const uint32_t key = e & 0xFFFFu;
                    bool add = key > tau_key;
                    if (key == tau_key && room > 0u) {
                        add = true;
                        --room;
                    }
                    const uint32_t bit = add ? 1u << ((e >> 16) & 31u) : 0u;
                    const uint32_t word = e >> 21;
#pragma unroll
                    for (int i = 0; i < kWords; ++i) keep[i] |= word == static_cast<uint32_t>(i) ? bit : 0u;
                }
            }

        }

        // ---- D: every lane writes its kept entries, in column order, at its offset of the row's output ---------
        // (staged as {column << 16 | value}; the index is shifted by the parity of the row's first output element, so
        // that pairs of staged entries are pairs of 4-byte aligned output elements)
        const uint32_t shift = static_cast<uint32_t>(out_base) & 1u;
        {
            uint32_t kept_mine = 0;
#pragma unroll
            for (int i = 0; i < kWords; ++i) kept_mine += __popc(keep[i]);
            const uint32_t before = warp_inclusive_sum(kept_mine) - kept_mine;
            __syncwarp();                                      // every lane is done with its list: the words become the stage
            uint32_t at = smem_addr(stage) + 4u * (shift + before);
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t m = keep[i];
                const uint32_t colb = lane * Lay::E + 32u * i + 31u;           // column of bit q: colb - q
                const uint32_t trips = __reduce_max_sync(0xFFFFFFFFu, static_cast<uint32_t>(__popc(m)));
#pragma unroll 2
                for (uint32_t t = 0; t < trips; ++t) {
                    // branch-free: a lane whose word has run out loads from the row's first column and stores nothing
                    const uint32_t some = m != 0u ? 1u : 0u;
                    const uint32_t q = bfind(m) & 31u;
                    m &= ~(some << q);
                    const uint32_t col = some ? colb - q : 0u;
                    uint32_t v;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(row_addr + 2u * col));
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p st.shared.u32 [%0], %1;\n\t}"
                                 ::"r"(at), "r"(prmt(v, col, 0x5410u)), "r"(some) : "memory");
                    at += 4u * some;
                }
            }
        }
        release_row();                                         // (starts with a warp barrier: the stage is complete)

        // ---- E: the staged entries leave in pairs: 4-byte stores to either output ------------------------------
        {
            const size_t pair_base = out_base - shift;         // even: cols_out / vals_out + pair_base are 4-byte aligned
            const uint32_t last = shift + k;                    // staged entries live at [shift, last)
            for (uint32_t p = 2u * lane; p < last; p += 64u) {
                const uint2 e = *reinterpret_cast<const uint2*>(stage + p);
                const bool first = p >= shift, second = p + 1u < last;
                if (first && second) {
                    *reinterpret_cast<uint32_t*>(cols_out + pair_base + p) = prmt(e.x, e.y, 0x7632u);
                    *reinterpret_cast<uint32_t*>(vals_out + pair_base + p) = prmt(e.x, e.y, 0x5410u);
                } else if (first) {
                    cols_out[pair_base + p] = static_cast<int16_t>(e.x >> 16);
                    vals_out[pair_base + p] = static_cast<uint16_t>(e.x & 0xFFFFu);
                } else if (second) {
                    cols_out[pair_base + p + 1u] = static_cast<int16_t>(e.y >> 16);
                    vals_out[pair_base + p + 1u] = static_cast<uint16_t>(e.y & 0xFFFFu);
                }
            }
            if (rows_out)
                for (uint32_t p = lane; p < k; p += 32) rows_out[out_base + p] = static_cast<int32_t>(row);
        }
        __syncwarp();
    }
    chain_release_next();           // no row left for this warp: the next kernel may be scheduled as this one's CTAs retire
}

template <int E8>
dct_status_t launch_span(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                         void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result, cudaStream_t stream) {
    using Lay = SpanLayout<E8>;
    auto kernel = mp_topk_fwd_bf16_span_kernel<E8>;
    constexpr size_t kSmemBudget = 226 * 1024;             // of the 227 KiB a CTA may use (a few static words besides)
    static thread_local int configured_device = -1;
    int dev = 0;
    DCT_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        DCT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(kSmemBudget)));
        configured_device = dev;
    }
    const size_t per_warp = Lay::warp_bytes(k);
    size_t warps = kSmemBudget / per_warp;
    if (warps > static_cast<size_t>(span_max_warps<E8>())) warps = span_max_warps<E8>();
    if (warps < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    warps = warps_for_rows(warps, rows, sms);
    const uint64_t ctas_needed = (static_cast<uint64_t>(rows) + warps - 1) / warps;
    const uint32_t grid = static_cast<uint32_t>(ctas_needed < static_cast<uint64_t>(sms) ? ctas_needed : sms);
    DCT_CUDA_TRY(launch_chained_smem(kernel, grid, static_cast<unsigned>(warps * 32), warps * per_warp, stream,
                                     static_cast<const uint16_t*>(x_act), rows, d, ld, k, cols_out,
                                     static_cast<uint16_t*>(vals_out), rows_out, static_cast<uint16_t*>(tau_out), result));
    return DCT_OK;
}


// ------------------------------------------------------------------------------------------
// rows of more than 3072 columns (up to 32768): W warps per row, one row per CTA at a time
// ------------------------------------------------------------------------------------------
// The same steps as above with a CTA in the place of the warp: lane l of warp w looks after the 32 KW columns from
// (32 w + l) 32 KW on (KW = 2 for rows of up to 8192 columns, 4 beyond), counts and offsets are summed over the warps
// through shared memory, and
// the histogram of the window elements is the CTA's.  No lists: a lane walks the window bits of its span twice, once
// for the histogram and once, with tau_i known, to add the elements above tau_i to its kept bits and to mark the
// ties; one scan over the CTA then gives every lane its offset in the row's output and its share of the ties.
// Several CTAs share an SM, so one CTA's load overlaps another's work.  A row whose window does not settle is not
// handed to another routine: its threshold is found bit by bit (15 counting passes) and the row is then packed
// with a window of one key, whose elements all tie at tau_i.
constexpr uint32_t kWideMaxK = 12288;            // 3/8 of the widest row (staging: 4 bytes per kept entry)
constexpr int kWideRetries = 6;
constexpr uint32_t kWideShrink = 3;               // window elements per lane (on average) from which the window narrows

template <int W, int KW> struct WideLayout {             // KW: flag words (32 columns each) of a lane, 2 or 4
    static constexpr uint32_t kSegBytes = 2048u * KW;        // one warp's 1024 KW columns
    static constexpr uint32_t kRowBytes = W * kSegBytes;
    static constexpr uint32_t kHistBytes = 256u;
    __host__ __device__ static constexpr uint32_t cta_bytes(uint32_t k) {
        return (kRowBytes + kHistBytes + 4u * (k + 2u) + 127u) & ~127u;
    }
};

template <int W, int KW>
__global__ void __launch_bounds__(W * 32)
mp_topk_fwd_bf16_wide_kernel(const uint16_t* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                             int16_t* __restrict__ cols_out, uint16_t* __restrict__ vals_out,
                             int32_t* __restrict__ rows_out, uint16_t* __restrict__ tau_out,
                             dct_result_t* __restrict__ result) {
    using Lay = WideLayout<W, KW>;
    constexpr int kWords = KW;                                 // 32 KW columns per lane
    constexpr uint32_t kLaneCols = 32u * KW;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned char* base = smem_raw;
    const unsigned char* own = base + warp * Lay::kSegBytes + lane * (2u * kLaneCols);
    uint32_t* hist = reinterpret_cast<uint32_t*>(base + Lay::kRowBytes);
    uint32_t* stage = hist + Lay::kHistBytes / 4;
    __shared__ uint64_t s_bar;
    __shared__ uint32_t s_stop;
    __shared__ uint32_t s_cnt[2][W];                           // per-warp packed counts (double-buffered across passes)
    __shared__ uint32_t s_sum[2][W];                           // per-warp totals of the row's scan (double-buffered across rows)
    __shared__ uint32_t s_guess;

    if (threadIdx.x == 0) {
        s_stop = 0;
        mbar_init(&s_bar, 1);
        mbar_init_fence();
        fence_proxy_async_all();
    }
    const uint32_t row_bytes = d * 2u;                         // the tail of the buffer stays zero
    for (uint32_t b = row_bytes + threadIdx.x * 16u; b < Lay::kRowBytes; b += W * 512u)
        *reinterpret_cast<uint4*>(base + b) = make_uint4(0, 0, 0, 0);
    __syncthreads();
    chain_wait_previous();                                     // set-up done: the inputs may come from the previous kernel
    if (blockIdx.x == 0 && threadIdx.x == 0 && result) {
        result->status = DCT_OK;
        result->reserved = 0;
        result->count = 0;
        result->needed = 0;
        result->n_gt = 0;
        result->n_eq = 0;
    }
    const uint32_t swz = lane & 7u;
    const uint32_t fix_sel = 0x3210u ^ (0x1111u * (swz & 3u));
    uint32_t unit_base[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) unit_base[c] = smem_addr(own) ^ (16u * (swz ^ static_cast<uint32_t>(c)));
    const uint32_t row_addr = smem_addr(base);
    const uint32_t col0 = (warp * 32u + lane) * kLaneCols;     // first column of the lane's span
    const bool emit = cols_out != nullptr;                     // (thresholds only, for the diagnostics, if not)

    auto request_row = [&](uint64_t r) {
        if (threadIdx.x == 0) {
            fence_proxy_async_smem();
            mbar_arrive_expect_tx(&s_bar, row_bytes);
            bulk_load(base, x + static_cast<size_t>(r) * ld, row_bytes, &s_bar);
        }
    };
    // sum of one packed word per warp over the CTA (and optionally the part before this warp)
    auto cta_sum = [&](uint32_t (*slot)[W], uint32_t parity, uint32_t warp_total, uint32_t& before) -> uint32_t {
        if (lane == 0) slot[parity][warp] = warp_total;
        __syncthreads();
        uint32_t total = 0;
        before = 0;
#pragma unroll
        for (int w = 0; w < W; ++w) {
            const uint32_t t = slot[parity][w];
            total += t;
            before += static_cast<uint32_t>(w) < warp ? t : 0u;
        }
        return total;
    };

    // both flag sets of the lane's span for the bounds (low, high); returns the lane's packed counts
    uint32_t ge_low[kWords], ge_high[kWords];
    auto flag_pass = [&](uint32_t low, uint32_t high) -> uint32_t {
        const uint32_t low2 = low * 0x10001u, high2 = high * 0x10001u;
#pragma unroll
        for (int i = 0; i < kWords; ++i) ge_low[i] = ge_high[i] = 0;
        static_for<4 * KW>([&](auto c_tag) {
            constexpr int c = decltype(c_tag)::value;
            uint32_t f_low, f_high;
            flags8_two(lds128<128 * (c / 8)>(unit_base[c % 8]), low2, high2, f_low, f_high);
            constexpr uint32_t sel = c % 4 == 1 ? 0x3410u : (c % 4 == 2 ? 0x3240u : 0x3214u);
            ge_low[c / 4] = (c % 4 == 0) ? (f_low << 24) : prmt(ge_low[c / 4], f_low, sel);
            ge_high[c / 4] = (c % 4 == 0) ? (f_high << 24) : prmt(ge_high[c / 4], f_high, sel);
        });
#pragma unroll
        for (int h = 0; h < kWords; h += 2) {
            const uint32_t l0 = ge_low[h], l1 = ge_low[h + 1], h0 = ge_high[h], h1 = ge_high[h + 1];
            ge_low[h] = (swz & 4u) ? l1 : l0;
            ge_low[h + 1] = (swz & 4u) ? l0 : l1;
            ge_high[h] = (swz & 4u) ? h1 : h0;
            ge_high[h + 1] = (swz & 4u) ? h0 : h1;
        }
        uint32_t mine = 0;
#pragma unroll
        for (int i = 0; i < kWords; ++i) {
            ge_low[i] = prmt(ge_low[i], 0u, fix_sel);
            ge_high[i] = prmt(ge_high[i], 0u, fix_sel);
            mine += (__popc(ge_low[i]) << 16) | __popc(ge_high[i]);
        }
        return mine;
    };

    if (blockIdx.x < rows) request_row(blockIdx.x);
    uint32_t use = 0, pass_no = 0;
    uint32_t guess_low = 0;
    uint32_t window = kSpanWindow;
    for (uint64_t row64 = blockIdx.x; row64 < rows; row64 += gridDim.x, ++use) {
        const uint32_t row = static_cast<uint32_t>(row64);
        if (!__syncthreads_and(mbar_wait_bounded(&s_bar, use & 1u, 1u << 24, &s_stop) ? 1 : 0)) {
            s_stop = 1;
            if (threadIdx.x == 0 && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
            return;
        }
        const size_t out_base = static_cast<size_t>(row) * k;

        // ---- A: bounds around tau_i ------------------------------------------------------------------
        uint32_t low = guess_low;
        if (low == 0) {
            // the (k/d)-quantile of 128 samples of the first warp's columns, taken a little low, found bit by bit
            if (warp == 0) {
                uint32_t sample[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) sample[c] = *reinterpret_cast<const uint16_t*>(own + c * 16) & 0x7FFFu;
                uint32_t rank = (128u * k + d - 1) / d;
                rank += 2u * static_cast<uint32_t>(__fsqrt_rn(static_cast<float>(rank))) + 2u;
                if (rank > 128u) rank = 128u;
                uint32_t q = 0;
#pragma unroll 1
                for (int bit = 14; bit >= 0; --bit) {
                    const uint32_t trial = q | (1u << bit);
                    uint32_t cnt = 0;
#pragma unroll
                    for (int c = 0; c < 4; ++c) cnt += sample[c] >= trial ? 1u : 0u;
                    if (__reduce_add_sync(0xFFFFFFFFu, cnt) >= rank) q = trial;
                }
                if (lane == 0) s_guess = q ? q : 1u;
            }
            __syncthreads();
            low = s_guess;
        }
        if (low > 0x7F80u) low = 0x7F80u;

        // ---- B: the window ---------------------------------------------------------------------------
        uint32_t n_low = 0, n_high = 0;
        bool pinned = false, moved = false, tau_zero = false;
        if (threadIdx.x < 64) hist[threadIdx.x] = 0;           // (a barrier follows in the first pass)
#pragma unroll 1
        for (int attempt = 0; attempt < kWideRetries; ++attempt) {
            const uint32_t mine = flag_pass(low, low + window);
            uint32_t before;
            const uint32_t total = cta_sum(s_cnt, pass_no & 1u, __reduce_add_sync(0xFFFFFFFFu, mine), before);
            ++pass_no;
            n_low = total >> 16;
            n_high = total & 0xFFFFu;
            if (n_high < k && k <= n_low) {
                pinned = true;
                break;
            }
            const uint32_t per_key_x16 = max(((n_low - n_high) << 4) / window, 4u);
            moved = true;
            if (n_low < k) {
                if (low == 1) {                                    // fewer than k non-zeros: tau_i = 0
                    tau_zero = true;
                    break;
                }
                const uint32_t below = max(((k - n_low) << 4) / per_key_x16 + window / 2u, window / 2u);
                low = low > below ? low - below : 1u;
            } else {
                const uint32_t above = ((n_high - k + 1u) << 4) / per_key_x16 + window / 2u;
                low = low + above < 0x7F80u ? low + above : 0x7F80u;
            }
        }

        // ---- C: tau_i; the columns above it (kept for certain) and the ties at it, as bits ------------------------
        uint32_t tau_key = 0;
        uint32_t keep[kWords], ties[kWords];
        if (pinned) {
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t m = ge_low[i] & ~ge_high[i];
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    uint32_t v;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(row_addr + 2u * (col0 + 32u * i + 31u - q)));
                    atomicAdd(&hist[(v & 0x7FFFu) - low], 1u);
                }
            }
            __syncthreads();
            {
                // the (k - n_high)-th largest window element: lane l owns the bins 63 - 2 l (h.y) and 62 - 2 l
                const uint32_t r = k - n_high;
                const uint2 h = reinterpret_cast<const uint2*>(hist)[31u - lane];
                const uint32_t own_cnt = h.x + h.y;
                const uint32_t before = warp_inclusive_sum(own_cnt) - own_cnt;
                uint32_t my_bin = 0;
                bool mine = false;
                if (before < r && r <= before + h.y) {
                    mine = true;
                    my_bin = 63u - 2u * lane;
                } else if (before + h.y < r && r <= before + own_cnt) {
                    mine = true;
                    my_bin = 62u - 2u * lane;
                }
                const uint32_t who = __ballot_sync(0xFFFFFFFFu, mine);
                tau_key = low + __shfl_sync(0xFFFFFFFFu, my_bin, who ? __ffs(who) - 1 : 0);
            }
            if (moved) {
                window = window < kSpanWindow ? window * 2u : kSpanWindow;
            } else if (n_low - n_high > kWideShrink * 32u * W && window > 4u) {
                window >>= 1;                                      // many window elements per lane: a narrower one next time
            }
            guess_low = tau_key > window / 2u ? tau_key - window / 2u : 1u;
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t m = ge_low[i] & ~ge_high[i];
                keep[i] = ge_high[i];
                ties[i] = 0;
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    uint32_t v;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(row_addr + 2u * (col0 + 32u * i + 31u - q)));
                    v &= 0x7FFFu;
                    keep[i] |= v > tau_key ? 1u << q : 0u;
                    ties[i] |= v == tau_key ? 1u << q : 0u;
                }
            }
        } else {
            // exact mode: the largest v with #{key >= v} >= k, bit by bit (0 if the window ended there); then a window
            // of one key at it (v = 0: every column, the padding behind the row included, is >= 0)
            uint32_t v = 0;
            if (!tau_zero) {
#pragma unroll 1
                for (int bit = 14; bit >= 0; --bit) {
                    const uint32_t trial = v | (1u << bit);
                    const uint32_t mine = flag_pass(trial, trial);
                    uint32_t before;
                    const uint32_t total = cta_sum(s_cnt, pass_no & 1u, __reduce_add_sync(0xFFFFFFFFu, mine), before);
                    ++pass_no;
                    if ((total >> 16) >= k) v = trial;
                }
            }
            tau_key = v;
            flag_pass(v, v + 1u);
            guess_low = 0;
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                keep[i] = ge_high[i];
                ties[i] = ge_low[i] & ~ge_high[i];
            }
        }
        if (threadIdx.x == 0 && tau_out) tau_out[row] = static_cast<uint16_t>(tau_key);

        // ---- D: every lane stages its kept entries at its offset of the row's output ----------------------------
        // One scan of (#certain << 16 | #ties) over the CTA: the ties are taken in column order until k is reached.
        const uint32_t shift = static_cast<uint32_t>(out_base) & 1u;
        if (emit) {
            uint32_t packed = 0;
#pragma unroll
            for (int i = 0; i < kWords; ++i) packed += (__popc(keep[i]) << 16) | __popc(ties[i]);
            const uint32_t incl = warp_inclusive_sum(packed);
            uint32_t warps_before;
            const uint32_t total = cta_sum(s_sum, use & 1u, __shfl_sync(0xFFFFFFFFu, incl, 31), warps_before);
            const uint32_t ties_to_take = k - (total >> 16);
            const uint32_t mine_before = warps_before + incl - packed;
            const uint32_t ties_before = mine_before & 0xFFFFu;
            uint32_t room = ties_before < ties_to_take ? ties_to_take - ties_before : 0u;
            uint32_t at = smem_addr(stage) +
                          4u * (shift + (mine_before >> 16) + (ties_before < ties_to_take ? ties_before : ties_to_take));
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t z = ties[i];
                const uint32_t n = __popc(z);
                if (n > room) {
                    for (uint32_t extra = n - room; extra; --extra) z &= z - 1u;   // the highest columns go (lowest bits)
                    room = 0;
                } else {
                    room -= n;
                }
                uint32_t m = keep[i] | z;
                const uint32_t colb = col0 + 32u * i + 31u;
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    const uint32_t col = colb - q;
                    uint32_t v;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(row_addr + 2u * col));
                    asm volatile("st.shared.u32 [%0], %1;" ::"r"(at), "r"(prmt(v, col, 0x5410u)) : "memory");
                    at += 4u;
                }
            }
        }
        fence_proxy_async_smem();                              // this thread's reads of the row come before the next bulk copy into it
        __syncthreads();                                       // the stage is complete, the row buffer free
        if (row64 + gridDim.x < rows) request_row(row64 + gridDim.x);

        // ---- E: the staged entries leave in pairs ------------------------------------------------------------------
        if (emit) {
            const size_t pair_base = out_base - shift;
            const uint32_t last = shift + k;
            for (uint32_t p = 2u * threadIdx.x; p < last; p += 2u * W * 32u) {
                const uint2 e = *reinterpret_cast<const uint2*>(stage + p);
                const bool first = p >= shift, second = p + 1u < last;
                if (first && second) {
                    *reinterpret_cast<uint32_t*>(cols_out + pair_base + p) = prmt(e.x, e.y, 0x7632u);
                    *reinterpret_cast<uint32_t*>(vals_out + pair_base + p) = prmt(e.x, e.y, 0x5410u);
                } else if (first) {
                    cols_out[pair_base + p] = static_cast<int16_t>(e.x >> 16);
                    vals_out[pair_base + p] = static_cast<uint16_t>(e.x & 0xFFFFu);
                } else if (second) {
                    cols_out[pair_base + p + 1u] = static_cast<int16_t>(e.y >> 16);
                    vals_out[pair_base + p + 1u] = static_cast<uint16_t>(e.y & 0xFFFFu);
                }
            }
            if (rows_out)
                for (uint32_t p = threadIdx.x; p < k; p += W * 32u) rows_out[out_base + p] = static_cast<int32_t>(row);
        }
        __syncthreads();                                       // the stage has been read: the next row may fill it
    }
    chain_release_next();
}

template <int W, int KW>
dct_status_t launch_wide(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                         void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result, cudaStream_t stream) {
    using Lay = WideLayout<W, KW>;
    auto kernel = mp_topk_fwd_bf16_wide_kernel<W, KW>;
    const size_t smem = Lay::cta_bytes(k);
    static thread_local int configured_device = -1;
    int dev = 0;
    DCT_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        DCT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
        configured_device = dev;
    }
    int per_sm = 0;
    DCT_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, W * 32, smem));
    if (per_sm < 1) return DCT_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    const uint64_t max_grid = static_cast<uint64_t>(sms) * per_sm;
    const uint32_t grid = static_cast<uint32_t>(rows < max_grid ? rows : max_grid);
    DCT_CUDA_TRY(launch_chained_smem(kernel, grid, static_cast<unsigned>(W * 32), smem, stream,
                                     static_cast<const uint16_t*>(x_act), rows, d, ld, k, cols_out,
                                     static_cast<uint16_t*>(vals_out), rows_out, static_cast<uint16_t*>(tau_out), result));
    return DCT_OK;
}

}  // namespace

// The per-row thresholds alone (tau_out[row], nothing packed), by the CTA-per-row kernel: for the threshold
// diagnostics.  *handled = false: not a shape of this kernel.
dct_status_t launch_tau_bf16_wide(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, void* tau_out,
                                  cudaStream_t stream, bool* handled) {
    *handled = false;
    if (d <= 3072 || d > 32768 || d % 8 != 0 || k > kWideMaxK || 8ull * k > 3ull * d || !aligned_to(x_act, 16) ||
        (static_cast<size_t>(ld) * 2) % 16 != 0)
        return DCT_OK;
    *handled = true;
#define DCT_WIDE_WARPS(W, KW) \
    if (d <= 1024u * KW * W)  \
        return launch_wide<W, KW>(x_act, rows, d, ld, k, nullptr, nullptr, nullptr, tau_out, nullptr, stream)
    DCT_WIDE_WARPS(2, 2);
    DCT_WIDE_WARPS(3, 2);
    DCT_WIDE_WARPS(4, 2);
    DCT_WIDE_WARPS(3, 4);
    DCT_WIDE_WARPS(4, 4);
    DCT_WIDE_WARPS(5, 4);
    DCT_WIDE_WARPS(6, 4);
    DCT_WIDE_WARPS(7, 4);
    DCT_WIDE_WARPS(8, 4);
#undef DCT_WIDE_WARPS
    *handled = false;
    return DCT_OK;
}

dct_status_t launch_fwd_bf16_span(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                  int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                  dct_result_t* result, cudaStream_t stream, bool* handled) {
    *handled = false;
    // Rows of more than 3072 columns: one CTA per row (rows of 3073..8192 columns with 64 columns per lane, wider ones
    // with 128).  Measured against the warp-per-row kernel below, which served rows of up to 8192 columns before:
    // 16384x4096, k = 1024: 66.6 against 73.3 us; 8192x8192, k = 1280: 52.3 against 77.0 us; k = 2048: 69.0 against
    // 97.8 us; and widths that kernel is not instantiated for (5120, 6144 columns in its 8192-column buffer) three
    // times faster.  64 columns per lane on rows beyond 8192 columns: 4 to 9 % slower than 128.
    if (d > 3072 && d <= 32768 && d % 8 == 0 && k <= kWideMaxK && 8ull * k <= 3ull * d && aligned_to(x_act, 16) &&
        (static_cast<size_t>(ld) * 2) % 16 == 0 && aligned_to(cols_out, 4) && aligned_to(vals_out, 4)) {
        *handled = true;
        // as many warps as the row has segments of 2048 (4096) columns, the last one zero-padded
#define DCT_WIDE_WARPS(W, KW) \
    if (d <= 1024u * KW * W)  \
        return launch_wide<W, KW>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream)
        DCT_WIDE_WARPS(2, 2);
        DCT_WIDE_WARPS(3, 2);
        DCT_WIDE_WARPS(4, 2);
        DCT_WIDE_WARPS(3, 4);
        DCT_WIDE_WARPS(4, 4);
        DCT_WIDE_WARPS(5, 4);
        DCT_WIDE_WARPS(6, 4);
        DCT_WIDE_WARPS(7, 4);
        DCT_WIDE_WARPS(8, 4);
#undef DCT_WIDE_WARPS
    }
    // (beyond 3/8 of the row a post-ReLU row's threshold is next to zero, where keys are sparse and the window
    // rarely settles: the general kernel serves those)
    if (d > 3072 || d % 8 != 0 || k > kSpanMaxK || 8ull * k > 3ull * d) return DCT_OK;
    if (!aligned_to(x_act, 16) || (static_cast<size_t>(ld) * 2) % 16 != 0) return DCT_OK;
    if (!aligned_to(cols_out, 4) || !aligned_to(vals_out, 4)) return DCT_OK;   // the paired stores need 4-byte aligned outputs
    *handled = true;
    // The smallest buffer of 256 * E8 columns that holds the row, every E8 up to 12: a lane's span is 8 E8 columns, and
    // a row that fills only part of the lanes crowds their lists (43690x1536, k = 576 in the 2048-column buffer: 0.98 ms,
    // nearly every row on the slow path; in its own buffer 0.095 ms).
#define DCT_SPAN_WIDTH(E8) \
    if (d <= 256u * E8) return launch_span<E8>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream)
    DCT_SPAN_WIDTH(1);
    DCT_SPAN_WIDTH(2);
    DCT_SPAN_WIDTH(3);
    DCT_SPAN_WIDTH(4);
    DCT_SPAN_WIDTH(5);
    DCT_SPAN_WIDTH(6);
    DCT_SPAN_WIDTH(7);
    DCT_SPAN_WIDTH(8);
    DCT_SPAN_WIDTH(9);
    DCT_SPAN_WIDTH(10);
    DCT_SPAN_WIDTH(11);
    DCT_SPAN_WIDTH(12);
#undef DCT_SPAN_WIDTH
    *handled = false;
    return DCT_OK;
}

}  // namespace dct
