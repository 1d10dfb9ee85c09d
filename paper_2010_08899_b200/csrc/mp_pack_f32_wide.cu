// dct_mp_topk_pack_fwd, fp32, rows of more than 512 columns (up to 32768) that the warp-per-row kernels do not serve:
// Algorithm 2 (DCT-MP), forward pass -- one CTA of W warps per row, warp w looking after the columns
// [1024 w, 1024 w + 1024) and lane l of it after 32 of them (KW = 1; twice that with KW = 2).
//
// The row arrives by one bulk copy (TMA engine) into shared memory as it lies in HBM.  The steps are those of the
// bf16 kernel for wide rows (mp_pack_span.cu), on two levels, because a key has 31 bits and the packed compares 15:
//   A  two bounds around the *bucket* of tau_i (a bucket = the upper 15 bits of the key, the bf16 truncation of |x|):
//      the previous row's bucket minus half a window, or a quantile of 128 samples of the row.
//   B  one pass over the lane's eight (sixteen) 16-byte units gives two flags per column (bucket >= low, bucket >= high) as
//      bits in registers: the upper halves of the fp32 words are gathered by byte permutes, the compares are integer
//      subtractions on the packed halves, and a byte permutation plus two dot-product instructions collect 8 flags.
//      The units are read in an XOR-swizzled order (no bank conflicts although the lanes' spans are a multiple of
//      128 bytes apart); a byte permutation puts the flags back in column order.  Counts are summed over the CTA; the window
//      moves until n_high < k <= n_low.
//   C  a radix select over the window elements: their buckets go into a 64-bin histogram, which gives the bucket of
//      tau_i and how many of its members belong to the top k; the members' lower 16 key bits follow in digits of
//      6, 6 and 4 bits (a round is skipped as soon as one member is left), which gives the exact 31-bit tau_i.
//   D  kept are the columns above the bucket, the members above tau_i and the first ties in column order.  One scan
//      over the CTA gives every lane its offset in the row's output and its share of the ties; it stages column
//      and value.
//   E  the staged entries leave as coalesced stores while the row buffer already receives the CTA's next row.
// A row whose window does not settle finds its bucket bit by bit (15 counting passes) and goes on from C's second
// half; a row with fewer than k elements outside bucket 0 starts there.  The result never depends on the guesses.
#include "common.cuh"
#include "mp_warp.cuh"

namespace dct {
namespace {

constexpr uint32_t kWideWindowF32 = 64;           // widest window, in buckets (= histogram bins)
constexpr uint32_t kWideMaxKF32 = 12288;        // 3/8 of the widest row (staging: 6 bytes per kept entry)
constexpr int kWideRetriesF32 = 6;

template <int W, int KW> struct WideLayoutF32 {
    static constexpr uint32_t kSegBytes = 4096u * KW;        // one warp's 1024 KW columns
    static constexpr uint32_t kRowBytes = W * kSegBytes;
    static constexpr uint32_t kHistBytes = 1024u;            // four tables of 64 bins
    __host__ __device__ static constexpr uint32_t vals_bytes(uint32_t k) { return 4u * k; }
    __host__ __device__ static constexpr uint32_t cta_bytes(uint32_t k) {
        return (kRowBytes + kHistBytes + vals_bytes(k) + 2u * (k + 2u) + 127u) & ~127u;
    }
};

// upper halves of two fp32 words in one register, with bit 15 of either half set: (hi16(b) << 16) | hi16(a) | 0x80008000
__device__ __forceinline__ uint32_t upper_halves_set(uint32_t a, uint32_t b) {
    return prmt(a, b, 0x7632u) | 0x80008000u;
}

template <int W, int KW>
__global__ void __launch_bounds__(W * 32)
mp_topk_fwd_f32_wide_kernel(const float* __restrict__ x, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                            int16_t* __restrict__ cols_out, uint32_t* __restrict__ vals_out,
                            int32_t* __restrict__ rows_out, uint32_t* __restrict__ tau_out,
                            dct_result_t* __restrict__ result) {
    using Lay = WideLayoutF32<W, KW>;
    constexpr int kWords = KW;                                 // 32 KW columns per lane
    constexpr uint32_t kLaneCols = 32u * KW;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    unsigned char* base = smem_raw;
    const unsigned char* own = base + warp * Lay::kSegBytes + lane * (4u * kLaneCols);
    uint32_t* hist = reinterpret_cast<uint32_t*>(base + Lay::kRowBytes);
    uint32_t* stage_vals = hist + Lay::kHistBytes / 4;
    uint16_t* stage_cols = reinterpret_cast<uint16_t*>(stage_vals + k);
    __shared__ uint64_t s_bar;
    __shared__ uint32_t s_stop;
    __shared__ uint32_t s_cnt[2][W];                           // per-warp packed counts (double-buffered across passes)
    __shared__ uint32_t s_sum[2][W];                           // per-warp totals for the two prefix sums of a row
    __shared__ uint32_t s_guess;

    if (threadIdx.x == 0) {
        s_stop = 0;
        mbar_init(&s_bar, 1);
        mbar_init_fence();
        fence_proxy_async_all();
    }
    const uint32_t row_bytes = d * 4u;                         // the tail of the buffer stays zero
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
    // Step c of a pass reads the unit (swz ^ c % 8) + 8 (c / 8) of the lane's 8 KW; steps 2p and 2p + 1 make up the
    // 32-byte piece (p % 4 ^ swz / 2) + 4 (p / 4), its upper half first if swz is odd.
    const uint32_t swz = lane & 7u;
    const uint32_t fix_sel = 0x3210u ^ (0x1111u * (swz >> 1));
    const uint32_t w_first = (swz & 1u) ? 0xFFFEFCF8u : 0xF0E0C080u;     // column j of a piece at bit 7 - j
    const uint32_t w_second = (swz & 1u) ? 0xF0E0C080u : 0xFFFEFCF8u;
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
    // sum of one packed word per warp over the CTA, and the part of it that belongs to the warps before this one
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

    // Both flag sets of the lane's span for the bucket bounds (low, high): column 32 i + j of the span at bit 31 - j of
    // word i.  Returns the lane's counts, (#low << 16) | #high.  Exact for every bit pattern: per 16-bit half, bit 15
    // of ((bucket | 0x8000) - bound) is set iff bucket >= bound, and no borrow crosses the halves (bound <= 0x8000).
    uint32_t ge_low[kWords], ge_high[kWords];
    auto flag_pass = [&](uint32_t low, uint32_t high) -> uint32_t {
        const uint32_t low2 = low * 0x10001u, high2 = high * 0x10001u;
#pragma unroll
        for (int i = 0; i < kWords; ++i) ge_low[i] = ge_high[i] = 0;
        static_for<4 * KW>([&](auto p_tag) {
            constexpr int p = decltype(p_tag)::value;
            const uint4 a = lds128<128 * (p / 4)>(unit_base[(2 * p) % 8]);
            const uint4 b = lds128<128 * (p / 4)>(unit_base[(2 * p + 1) % 8]);
            const uint32_t u0 = upper_halves_set(a.x, a.y), u1 = upper_halves_set(a.z, a.w);
            const uint32_t u2 = upper_halves_set(b.x, b.y), u3 = upper_halves_set(b.z, b.w);
            const uint32_t f_low = static_cast<uint32_t>(
                dp4a_ss(prmt(u2 - low2, u3 - low2, 0xFDB9u), w_second, dp4a_ss(prmt(u0 - low2, u1 - low2, 0xFDB9u), w_first, 0)));
            const uint32_t f_high = static_cast<uint32_t>(
                dp4a_ss(prmt(u2 - high2, u3 - high2, 0xFDB9u), w_second, dp4a_ss(prmt(u0 - high2, u1 - high2, 0xFDB9u), w_first, 0)));
            // piece p (in read order) is byte 3 - p % 4 of word p / 4
            constexpr uint32_t sel = p % 4 == 1 ? 0x3410u : (p % 4 == 2 ? 0x3240u : 0x3214u);
            ge_low[p / 4] = (p % 4 == 0) ? (f_low << 24) : prmt(ge_low[p / 4], f_low, sel);
            ge_high[p / 4] = (p % 4 == 0) ? (f_high << 24) : prmt(ge_high[p / 4], f_high, sel);
        });
        uint32_t mine = 0;
#pragma unroll
        for (int i = 0; i < kWords; ++i) {
            ge_low[i] = prmt(ge_low[i], 0u, fix_sel);
            ge_high[i] = prmt(ge_high[i], 0u, fix_sel);
            mine += (__popc(ge_low[i]) << 16) | __popc(ge_high[i]);
        }
        return mine;
    };
    auto counted_pass = [&](uint32_t low, uint32_t high, uint32_t& pass_no) -> uint32_t {
        const uint32_t mine = flag_pass(low, high);
        uint32_t before;
        const uint32_t total = cta_sum(s_cnt, pass_no & 1u, __reduce_add_sync(0xFFFFFFFFu, mine), before);
        ++pass_no;
        return total;
    };

    if (blockIdx.x < rows) request_row(blockIdx.x);
    uint32_t use = 0, pass_no = 0;
    uint32_t guess_low = 0;
    uint32_t window = kWideWindowF32;
    for (uint64_t row64 = blockIdx.x; row64 < rows; row64 += gridDim.x, ++use) {
        const uint32_t row = static_cast<uint32_t>(row64);
        if (!__syncthreads_and(mbar_wait_bounded(&s_bar, use & 1u, 1u << 24, &s_stop) ? 1 : 0)) {
            s_stop = 1;
            if (threadIdx.x == 0 && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_TIMEOUT));
            return;
        }
        const size_t out_base = static_cast<size_t>(row) * k;
        for (uint32_t b = threadIdx.x; b < Lay::kHistBytes / 4; b += W * 32u) hist[b] = 0;   // (a barrier follows in B)

        // ---- A: bounds around the bucket of tau_i ------------------------------------------------------------
        uint32_t low = guess_low;
        if (low == 0) {
            // the (k/d)-quantile of 128 samples of the first warp's columns, taken a little low, found bit by bit
            if (warp == 0) {
                uint32_t sample[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) sample[c] = *reinterpret_cast<const uint16_t*>(own + c * 16 + 2) & 0x7FFFu;
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

        // ---- B: the window ---------------------------------------------------------------------------------
        uint32_t n_low = 0, n_high = 0;
        bool pinned = false, moved = false, bucket_zero = false;
#pragma unroll 1
        for (int attempt = 0; attempt < kWideRetriesF32; ++attempt) {
            const uint32_t total = counted_pass(low, low + window, pass_no);
            n_low = total >> 16;
            n_high = total & 0xFFFFu;
            if (n_high < k && k <= n_low) {
                pinned = true;
                break;
            }
            const uint32_t per_key_x16 = max(((n_low - n_high) << 4) / window, 4u);
            moved = true;
            if (n_low < k) {
                if (low == 1) {                                    // fewer than k elements outside bucket 0
                    bucket_zero = true;
                    break;
                }
                const uint32_t below = max(((k - n_low) << 4) / per_key_x16 + window / 2u, window / 2u);
                low = low > below ? low - below : 1u;
            } else {
                const uint32_t above = ((n_high - k + 1u) << 4) / per_key_x16 + window / 2u;
                low = low + above < 0x7F80u ? low + above : 0x7F80u;
            }
        }

        // ---- C: the bucket of tau_i, then tau_i inside it ----------------------------------------------------------
        // A radix select over the window elements: their bucket (64 bins), then the lower 16 key bits of the members of
        // the chosen bucket in digits of 6, 6 and 4 bits.  rank_in(h, r): the bin of h that holds the r-th largest
        // element, how many of that bin belong to the top r, and how many the bin holds.
        auto rank_in = [&](const uint32_t* h64, uint32_t r, uint32_t& bin_take, uint32_t& bin_count) -> uint32_t {
            const uint2 h = reinterpret_cast<const uint2*>(h64)[31u - lane];   // lane owns bins 63 - 2 lane (h.y), 62 - 2 lane
            const uint32_t own_cnt = h.x + h.y;
            const uint32_t before = warp_inclusive_sum(own_cnt) - own_cnt;      // elements in higher bins
            uint32_t my_bin = 0, my_take = 0, my_count = 0;
            bool mine = false;
            if (before < r && r <= before + h.y) {
                mine = true;
                my_bin = 63u - 2u * lane;
                my_take = r - before;
                my_count = h.y;
            } else if (before + h.y < r && r <= before + own_cnt) {
                mine = true;
                my_bin = 62u - 2u * lane;
                my_take = r - before - h.y;
                my_count = h.x;
            }
            const uint32_t who = __ballot_sync(0xFFFFFFFFu, mine);
            const int src = who ? __ffs(who) - 1 : 0;
            bin_take = __shfl_sync(0xFFFFFFFFu, my_take, src);
            bin_count = __shfl_sync(0xFFFFFFFFu, my_count, src);
            return __shfl_sync(0xFFFFFFFFu, my_bin, src);
        };
        uint32_t bucket = 0, take = 0;                             // `take` members of the bucket belong to the top k
        uint32_t members[kWords];
        if (pinned) {
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t m = ge_low[i] & ~ge_high[i];
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    uint32_t v;
                    asm volatile("ld.shared.u16 %0, [%1+2];" : "=r"(v) : "r"(row_addr + 4u * (col0 + 32u * i + 31u - q)));
                    atomicAdd(&hist[(v & 0x7FFFu) - low], 1u);
                }
            }
            __syncthreads();
            uint32_t bucket_count;
            bucket = low + rank_in(hist, k - n_high, take, bucket_count);
            if (moved) {
                window = window < kWideWindowF32 ? window * 2u : kWideWindowF32;
            } else if (n_low - n_high > 128u * W && window > 8u) {
                window >>= 1;                                      // many window elements per lane: a narrower one next time
            }
            guess_low = bucket > window / 2u ? bucket - window / 2u : 1u;
            // window elements above the bucket join the kept columns, those inside it are its members
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t m = ge_low[i] & ~ge_high[i];
                members[i] = 0;
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    uint32_t v;
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(row_addr + 4u * (col0 + 32u * i + 31u - q)));
                    const uint32_t b = (v >> 16) & 0x7FFFu;
                    if (b > bucket) ge_high[i] |= 1u << q;
                    if (b == bucket) {
                        members[i] |= 1u << q;
                        atomicAdd(&hist[64u + ((v >> 10) & 63u)], 1u);
                    }
                }
            }
        } else {
            // the largest bucket v with #{bucket >= v} >= k, bit by bit (known to be 0 if the window ended there)
            uint32_t v = 0;
            if (!bucket_zero) {
#pragma unroll 1
                for (int bit = 14; bit >= 0; --bit) {
                    const uint32_t trial = v | (1u << bit);
                    if ((counted_pass(trial, trial, pass_no) >> 16) >= k) v = trial;
                }
            }
            bucket = v;
            guess_low = 0;
            // the members of the bucket (bucket 0: every zero, the padding behind the row included)
            take = k - (counted_pass(bucket, bucket + 1u, pass_no) & 0xFFFFu);
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t m = members[i] = ge_low[i] & ~ge_high[i];
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    uint32_t lo16;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(lo16) : "r"(row_addr + 4u * (col0 + 32u * i + 31u - q)));
                    atomicAdd(&hist[64u + (lo16 >> 10)], 1u);
                }
            }
        }
        __syncthreads();
        // t = the take-th largest of the members' lower 16 key bits: up to three digits, fewer if a bin of one is met
        uint32_t t = 0;
        {
            uint32_t count;
            uint32_t prefix = rank_in(hist + 64, take, take, count);        // bits 15..10
            int known = 6;                                                  // upper bits of t in `prefix`
#pragma unroll 1
            for (int round = 0; round < 2 && count > 1u; ++round) {
                const int digit_bits = round == 0 ? 6 : 4;
                uint32_t* h = hist + 128 + 64 * round;
#pragma unroll
                for (int i = 0; i < kWords; ++i) {
                    uint32_t m = members[i];
                    while (m) {
                        const uint32_t q = bfind(m);
                        m ^= 1u << q;
                        uint32_t lo16;
                        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(lo16) : "r"(row_addr + 4u * (col0 + 32u * i + 31u - q)));
                        if ((lo16 >> (16 - known)) == prefix)
                            atomicAdd(&h[(lo16 >> (16 - known - digit_bits)) & ((1u << digit_bits) - 1u)], 1u);
                    }
                }
                __syncthreads();
                prefix = (prefix << digit_bits) | rank_in(h, take, take, count);
                known += digit_bits;
            }
            if (known == 16) {
                t = prefix;
            } else {
                // one member left under the prefix: its owner announces it
#pragma unroll
                for (int i = 0; i < kWords; ++i) {
                    uint32_t m = members[i];
                    while (m) {
                        const uint32_t q = bfind(m);
                        m ^= 1u << q;
                        uint32_t lo16;
                        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(lo16) : "r"(row_addr + 4u * (col0 + 32u * i + 31u - q)));
                        if ((lo16 >> (16 - known)) == prefix) s_guess = lo16;
                    }
                }
                __syncthreads();
                t = s_guess;
            }
        }
        if (threadIdx.x == 0 && tau_out) tau_out[row] = (bucket << 16) | t;

        // ---- D: every lane stages its kept entries at its offset of the row's output ----------------------------
        // kept: the columns above the bucket, the members above t, and the first ties at t in column order.  One scan
        // of (#certain << 16 | #ties) over the CTA gives every lane both its offset and its share of the ties.
        const uint32_t shift = static_cast<uint32_t>(out_base) & 1u;
        if (emit) {
            uint32_t keep[kWords], eq[kWords], packed = 0;
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                keep[i] = ge_high[i];
                eq[i] = 0;
                uint32_t m = members[i];
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    uint32_t lo16;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(lo16) : "r"(row_addr + 4u * (col0 + 32u * i + 31u - q)));
                    keep[i] |= lo16 > t ? 1u << q : 0u;
                    eq[i] |= lo16 == t ? 1u << q : 0u;
                }
                packed += (__popc(keep[i]) << 16) | __popc(eq[i]);
            }
            const uint32_t incl = warp_inclusive_sum(packed);
            uint32_t warps_before;
            const uint32_t total = cta_sum(s_sum, use & 1u, __shfl_sync(0xFFFFFFFFu, incl, 31), warps_before);
            const uint32_t ties_to_take = k - (total >> 16);
            const uint32_t mine_before = warps_before + incl - packed;
            const uint32_t ties_before = mine_before & 0xFFFFu;
            uint32_t room = ties_before < ties_to_take ? ties_to_take - ties_before : 0u;
            uint32_t at = (mine_before >> 16) + (ties_before < ties_to_take ? ties_before : ties_to_take);
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t z = eq[i];
                const uint32_t n = __popc(z);
                if (n > room) {
                    for (uint32_t extra = n - room; extra; --extra) z &= z - 1u;   // the highest columns go (lowest bits)
                    room = 0;
                } else {
                    room -= n;
                }
                keep[i] |= z;
            }
            const uint32_t vals_addr = smem_addr(stage_vals), cols_addr = smem_addr(stage_cols) + 2u * shift;
#pragma unroll
            for (int i = 0; i < kWords; ++i) {
                uint32_t m = keep[i];
                const uint32_t colb = col0 + 32u * i + 31u;
                while (m) {
                    const uint32_t q = bfind(m);
                    m ^= 1u << q;
                    const uint32_t col = colb - q;
                    uint32_t v;
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(row_addr + 4u * col));
                    asm volatile("st.shared.u32 [%0], %1;" ::"r"(vals_addr + 4u * at), "r"(v) : "memory");
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(cols_addr + 2u * at), "h"(static_cast<uint16_t>(col)) : "memory");
                    ++at;
                }
            }
        }
        fence_proxy_async_smem();                              // this thread's reads of the row come before the next bulk copy into it
        __syncthreads();                                       // the stage is complete, the row buffer free
        if (row64 + gridDim.x < rows) request_row(row64 + gridDim.x);

        // ---- E: the staged entries leave: values one by one, columns in pairs --------------------------------------
        if (emit) {
            for (uint32_t p = threadIdx.x; p < k; p += W * 32u) vals_out[out_base + p] = stage_vals[p];
            const size_t pair_base = out_base - shift;
            const uint32_t last = shift + k;
            for (uint32_t p = 2u * threadIdx.x; p < last; p += 2u * W * 32u) {
                const uint32_t e = *reinterpret_cast<const uint32_t*>(stage_cols + p);
                const bool first = p >= shift, second = p + 1u < last;
                if (first && second) {
                    *reinterpret_cast<uint32_t*>(cols_out + pair_base + p) = e;
                } else if (first) {
                    cols_out[pair_base + p] = static_cast<int16_t>(e & 0xFFFFu);
                } else if (second) {
                    cols_out[pair_base + p + 1u] = static_cast<int16_t>(e >> 16);
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
dct_status_t launch_wide_f32(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, int16_t* cols_out,
                             void* vals_out, int32_t* rows_out, void* tau_out, dct_result_t* result,
                             cudaStream_t stream) {
    using Lay = WideLayoutF32<W, KW>;
    auto kernel = mp_topk_fwd_f32_wide_kernel<W, KW>;
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
                                     static_cast<const float*>(x_act), rows, d, ld, k, cols_out,
                                     static_cast<uint32_t*>(vals_out), rows_out, static_cast<uint32_t*>(tau_out), result));
    return DCT_OK;
}

}  // namespace

// The per-row thresholds alone (tau_out[row], nothing packed): for the threshold diagnostics.
dct_status_t launch_tau_f32_wide(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k, void* tau_out,
                                 cudaStream_t stream, bool* handled) {
    bool dummy = false;
    *handled = false;
    if (d <= 512 || d > 32768 || d % 4 != 0 || k > kWideMaxKF32 || 8ull * k > 3ull * d || !aligned_to(x_act, 16) ||
        (static_cast<size_t>(ld) * 4) % 16 != 0)
        return DCT_OK;
    const dct_status_t st = launch_fwd_f32_wide(x_act, rows, d, ld, k, nullptr, nullptr, nullptr, tau_out, nullptr, stream,
                                                &dummy);
    *handled = dummy;
    return st;
}

// *handled = false: the shape is not one of this path's; the caller runs the general kernel.
dct_status_t launch_fwd_f32_wide(const void* x_act, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                                 int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
                                 dct_result_t* result, cudaStream_t stream, bool* handled) {
    *handled = false;
    // (beyond 3/8 of the row a post-ReLU row's threshold is next to zero, where buckets are sparse and the window
    // rarely settles: the general kernel serves those)
    if (d <= 512 || d > 32768 || d % 4 != 0 || k > kWideMaxKF32 || 8ull * k > 3ull * d) return DCT_OK;
    if (!aligned_to(x_act, 16) || (static_cast<size_t>(ld) * 4) % 16 != 0 || !aligned_to(cols_out, 4)) return DCT_OK;
    *handled = true;
    // As many warps as the row has segments of 1024 or 2048 columns (the last one zero-padded): 64 columns per lane,
    // but 32 for rows of up to 4096 columns, which would otherwise be left with two warps (measured: 8 to 10 %
    // faster there, 2 to 10 % slower on wider rows, where the CTA-wide steps weigh more than the lanes' own).
    const bool narrow_spans = d <= 4096;
    if (narrow_spans) {
#define DCT_WIDE_F32_WARPS(W) \
    if (d <= 1024u * W) return launch_wide_f32<W, 1>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream)
        DCT_WIDE_F32_WARPS(1);
        DCT_WIDE_F32_WARPS(2);
        DCT_WIDE_F32_WARPS(3);
        DCT_WIDE_F32_WARPS(4);
#undef DCT_WIDE_F32_WARPS
    } else {
#define DCT_WIDE_F32_WARPS(W) \
    if (d <= 2048u * W) return launch_wide_f32<W, 2>(x_act, rows, d, ld, k, cols_out, vals_out, rows_out, tau_out, result, stream)
        DCT_WIDE_F32_WARPS(3);
        DCT_WIDE_F32_WARPS(4);
        DCT_WIDE_F32_WARPS(6);
        DCT_WIDE_F32_WARPS(8);
        DCT_WIDE_F32_WARPS(12);
        DCT_WIDE_F32_WARPS(16);
#undef DCT_WIDE_F32_WARPS
    }
    *handled = false;
    return DCT_OK;
}

}  // namespace dct
