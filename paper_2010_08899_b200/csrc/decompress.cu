// Receiver side of the two "send" steps: turning the packed messages back into dense tensors.
//
//   dct_dp_decompress : Algorithm 1, what the parameter server does with the sparse W_hat it receives:
//                       dense[idx[j]] = val[j] on a zero vector, or dense[idx[j]] += val[j] when the
//                       messages of several trainers are accumulated.
//   dct_mp_unpack     : Algorithm 2, what the next worker does with X_act .* M (and the previous worker
//                       with X_grad .* M): rebuild the [rows, d] matrix that is zero outside the mask.
//
// The paper counts decompression in the overhead of the scheme (Sec. 2) but gives no procedure; both
// are plain scatters.  Indices inside one message are distinct (ascending), so no atomics are needed.
#include "common.cuh"

namespace dct {
namespace {

// dense[0..n) = 0 with 128-bit stores, then the scatter, in one kernel: a grid-wide ordering between
// the two is not needed because every CTA first clears, and then scatters into, ITS OWN range of
// the dense vector: entries are routed to the CTA that owns idx via a binary search on the ascending idx.
__global__ void __launch_bounds__(256)
dp_decompress_kernel(const int32_t* __restrict__ idx, const float* __restrict__ val,
                     const dct_result_t* __restrict__ packed, uint64_t capacity, float* __restrict__ dense,
                     uint32_t n, int accumulate, dct_result_t* __restrict__ result) {
    const uint64_t have = packed->count < capacity ? packed->count : capacity;
    const uint32_t count = static_cast<uint32_t>(have);
    // this CTA owns dense[lo, hi): a multiple of 4 elements so that the clearing stores stay aligned
    const uint32_t per = ((n + gridDim.x - 1) / gridDim.x + 3u) & ~3u;
    const uint64_t lo64 = static_cast<uint64_t>(blockIdx.x) * per;
    bool bad = false;
    if (lo64 < n) {               // (CTAs past the end of the vector only help to check the list)
    const uint32_t lo = static_cast<uint32_t>(lo64);
    const uint32_t hi = (n - lo > per) ? lo + per : n;
    if (!accumulate) {
        const bool vec = (reinterpret_cast<uintptr_t>(dense) & 15u) == 0;
        if (vec) {
            const uint32_t hi4 = lo + ((hi - lo) & ~3u);
            for (uint32_t i = lo + threadIdx.x * 4; i < hi4; i += blockDim.x * 4)
                st_stream_f4(dense + i, make_float4(0.f, 0.f, 0.f, 0.f));
            for (uint32_t i = hi4 + threadIdx.x; i < hi; i += blockDim.x) dense[i] = 0.0f;
        } else {
            for (uint32_t i = lo + threadIdx.x; i < hi; i += blockDim.x) dense[i] = 0.0f;
        }
        __syncthreads();          // this CTA's range is clear before this CTA writes into it
    }
    // first entry with idx >= lo (idx ascending; malformed input only costs misplaced work, never a fault)
    uint32_t a = 0, b = count;
    while (a < b) {
        const uint32_t mid = (a + b) >> 1;
        if (static_cast<uint32_t>(idx[mid]) < lo) a = mid + 1; else b = mid;
    }
    for (uint32_t j = a + threadIdx.x; j < count; j += blockDim.x) {
        const uint32_t i = static_cast<uint32_t>(idx[j]);
        if (i >= hi) break;       // the rest belongs to later CTAs (or is out of range)
        if (i < lo) { bad = true; continue; }   // not ascending
        if (accumulate) dense[i] += val[j]; else dense[i] = val[j];
    }
    }
    // The list itself is checked once, by all CTAs together: every index inside [0, n), every index above the one
    // before it.  (An index that fails is never written outside the vector -- the loop above only writes inside this
    // CTA's range -- but the dense vector is then not what the sender meant: DCT_ERR_BAD_MASK.)
    for (uint64_t j = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < count;
         j += static_cast<uint64_t>(gridDim.x) * blockDim.x) {
        const int32_t i = idx[j];
        if (static_cast<uint32_t>(i) >= n || (j > 0 && i <= idx[j - 1])) bad = true;
    }
    if (bad) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_BAD_MASK));
}

// The same for a 16-byte aligned dense vector, with every tile of 4096 elements built in shared memory (cleared or,
// when accumulating, loaded; the tile's entries scattered into it) and written out with full 128-bit streaming
// stores: HBM sees 4 B per element (8 B when accumulating) plus the 8 B per entry, whatever the density, instead of
// one 32-byte sector per entry on top of the clearing stores.  A CTA walks through the tiles of its range; the
// entries of a tile follow those of the tile before it in the list, so one binary search per CTA is enough.
constexpr uint32_t kDecompTile = 4096;
// First entry of idx[0, count) that is >= bound, found by the whole CTA (256 threads): every round the threads probe
// 256 evenly spaced entries of the range that is left, so a list of 2^28 entries takes four rounds of one load each
// instead of 28 loads one after the other.  (A list that is not ascending gives some position inside it.)
__device__ __forceinline__ uint32_t cta_lower_bound(const int32_t* __restrict__ idx, uint32_t count, uint32_t bound) {
    uint32_t a = 0, b = count;                     // the answer lies in [a, b]
    while (b > a) {
        const uint32_t step = (b - a + 255u) / 256u;
        const uint64_t pos = static_cast<uint64_t>(a) + static_cast<uint64_t>(threadIdx.x) * step;
        const bool below = pos < b && static_cast<uint32_t>(idx[pos]) < bound;
        const uint32_t c = static_cast<uint32_t>(__syncthreads_count(below));   // probes 0 .. c-1 lie below the bound
        const uint32_t probes = (b - a + step - 1u) / step;
        const uint32_t new_a = c ? a + (c - 1u) * step + 1u : a;
        const uint32_t new_b = c < probes ? a + c * step : b;
        a = new_a;
        b = new_b;
        if (step == 1u) break;                     // every entry of the range was probed: a is the answer
    }
    return a;
}
template <bool kShifted>
__global__ void __launch_bounds__(256)
dp_decompress_tiled_kernel(const int32_t* __restrict__ idx, const float* __restrict__ val,
                           const dct_result_t* __restrict__ packed, uint64_t capacity, float* __restrict__ dense,
                           uint32_t n, int accumulate, dct_result_t* __restrict__ result, uint32_t lead_arg) {
    const uint32_t lead = kShifted ? lead_arg : 0u;          // (the aligned instance carries no checks for it)
    // lead != 0: the dense vector starts 4, 8 or 12 bytes past a 16-byte boundary; `dense` points to that boundary, n
    // counts from there and an index i of the list means position i + lead.  The `lead` elements before the vector share
    // its first 16 bytes: they are read when accumulating, never written.
    __shared__ __align__(16) float tile[kDecompTile];
    __shared__ uint32_t s_taken[2];     // entries the tile took, and
    __shared__ uint32_t s_first[2];     // the index of the first entry after them (two rounds in turn)
    const uint64_t have = packed->count < capacity ? packed->count : capacity;
    const uint32_t count = static_cast<uint32_t>(have);
    const uint32_t per = ((n + gridDim.x - 1) / gridDim.x + 3u) & ~3u;     // this CTA owns dense[lo, hi)
    const uint64_t lo64 = static_cast<uint64_t>(blockIdx.x) * per;
    bool bad = false;
    if (lo64 < n) {               // (CTAs past the end of the vector only help to check the list)
        const uint32_t lo = static_cast<uint32_t>(lo64);
        const uint32_t hi = (n - lo > per) ? lo + per : n;
        // the entries of this CTA's range: idx[a, end) (idx ascending; malformed input only costs misplaced work,
        // never a fault)
        const uint32_t n_own = n - lead;
        auto place_of = [&](uint32_t i) -> uint32_t { return i < n_own ? i + lead : 0xFFFFFFFFu; };   // (past the end: nowhere)
        uint32_t a = cta_lower_bound(idx, count, lo > lead ? lo - lead : 0u);
        const uint32_t end = hi < n ? cta_lower_bound(idx, count, hi - lead) : count;
        auto before_vector = [&](uint32_t at) -> bool {     // a position that is not the vector's
            if constexpr (kShifted) return at < lead; else return false;
        };
        auto store4 = [&](uint32_t at, float4 v) {     // 16 bytes at position `at`, but never the elements before the vector
            if (!before_vector(at)) {
                st_stream_f4(dense + at, v);
            } else {
                if (lead <= 1) dense[1] = v.y;
                if (lead <= 2) dense[2] = v.z;
                dense[3] = v.w;
            }
        };
        if (threadIdx.x < 2) {
            s_taken[threadIdx.x] = 0;
            s_first[threadIdx.x] = 0xFFFFFFFFu;
        }
        // index of the first entry that is not placed yet (none: past every tile); after a tile it is what the thread
        // that ran into it saw, so only this one is a load of its own
        uint32_t first = a < end ? place_of(static_cast<uint32_t>(idx[a])) : 0xFFFFFFFFu;
        uint32_t round = 0;
        for (uint32_t t_lo = lo; t_lo < hi; t_lo += kDecompTile) {
            const uint32_t t_hi = hi - t_lo > kDecompTile ? t_lo + kDecompTile : hi;
            const uint32_t len = t_hi - t_lo, len4 = len & ~3u;
            // A tile without an entry (most tiles of a sparse message) needs no shared memory: it is cleared straight
            // from registers or, when accumulating, left as it is.
            if (first >= t_hi) {
                if (!accumulate) {
                    for (uint32_t i = threadIdx.x * 4; i < len4; i += blockDim.x * 4)
                        store4(t_lo + i, make_float4(0.f, 0.f, 0.f, 0.f));
                    for (uint32_t i = len4 + threadIdx.x; i < len; i += blockDim.x)
                        if (!before_vector(t_lo + i)) dense[t_lo + i] = 0.0f;
                }
                continue;
            }
            for (uint32_t i = threadIdx.x * 4; i < len4; i += blockDim.x * 4)
                *reinterpret_cast<float4*>(tile + i) = accumulate ? ld_stream_f4(dense + t_lo + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            for (uint32_t i = len4 + threadIdx.x; i < len; i += blockDim.x) tile[i] = accumulate ? dense[t_lo + i] : 0.0f;
            __syncthreads();      // the tile is set up (and the counter of the round before last is free)
            if (threadIdx.x == 0) {
                s_taken[(round + 1) & 1u] = 0;
                s_first[(round + 1) & 1u] = 0xFFFFFFFFu;
            }
            uint32_t mine = 0, seen = 0xFFFFFFFFu;
            bool more = true;
            for (uint32_t j0 = a + threadIdx.x; more && j0 < end; j0 += 4u * blockDim.x) {
                uint32_t i4[4];
                float v4[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {     // four entries in flight (the values on the chance that they are needed)
                    const uint32_t j = j0 + u * blockDim.x;
                    i4[u] = j < end ? place_of(static_cast<uint32_t>(idx[j])) : 0xFFFFFFFFu;
                    v4[u] = j < end ? val[j] : 0.0f;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (!more || i4[u] >= t_hi) {  // the rest belongs to later tiles (or is out of range)
                        if (more) seen = i4[u];
                        more = false;
                        continue;
                    }
                    ++mine;
                    if (i4[u] < t_lo) { bad = true; continue; }   // not ascending
                    if (accumulate) tile[i4[u] - t_lo] += v4[u]; else tile[i4[u] - t_lo] = v4[u];
                }
            }
            if (mine) atomicAdd(&s_taken[round & 1u], mine);
            if (seen != 0xFFFFFFFFu) atomicMin(&s_first[round & 1u], seen);
            __syncthreads();      // every entry of the tile is in place
            for (uint32_t i = threadIdx.x * 4; i < len4; i += blockDim.x * 4)
                store4(t_lo + i, *reinterpret_cast<const float4*>(tile + i));
            for (uint32_t i = len4 + threadIdx.x; i < len; i += blockDim.x)
                if (!before_vector(t_lo + i)) dense[t_lo + i] = tile[i];
            a += s_taken[round & 1u];
            first = s_first[round & 1u];
            ++round;
            __syncthreads();      // the tile has been read out before the next one is set up
        }
    }
    // the list itself is checked once, by all CTAs together (see dp_decompress_kernel)
    for (uint64_t j = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < count;
         j += static_cast<uint64_t>(gridDim.x) * blockDim.x) {
        const int32_t i = idx[j];
        if (static_cast<uint32_t>(i) >= n - lead || (j > 0 && i <= idx[j - 1])) bad = true;
    }
    if (bad) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_BAD_MASK));
}

template <typename T>
__global__ void __launch_bounds__(256)
mp_unpack_kernel(const int16_t* __restrict__ cols, const T* __restrict__ vals, uint32_t rows, uint32_t d, uint32_t ld,
                 uint32_t k, T* __restrict__ dense, dct_result_t* __restrict__ result) {
    const uint32_t lane = lane_id();
    const uint32_t warps_per_cta = blockDim.x >> 5;
    bool bad = false;
    for (uint64_t row = static_cast<uint64_t>(blockIdx.x) * warps_per_cta + (threadIdx.x >> 5); row < rows;
         row += static_cast<uint64_t>(gridDim.x) * warps_per_cta) {
        T* out = dense + row * ld;
        // clear the d columns of the row: 16-byte stores where the row allows it
        const uintptr_t addr = reinterpret_cast<uintptr_t>(out);
        constexpr uint32_t per16 = 16 / sizeof(T);
        uint32_t head = static_cast<uint32_t>(((16 - (addr & 15u)) & 15u) / sizeof(T));
        if (head > d) head = d;
        for (uint32_t j = lane; j < head; j += 32) out[j] = T(0);
        const uint32_t nvec = (d - head) / per16;
        uint4* out16 = reinterpret_cast<uint4*>(out + head);
        for (uint32_t v = lane; v < nvec; v += 32) out16[v] = make_uint4(0, 0, 0, 0);
        for (uint32_t j = head + nvec * per16 + lane; j < d; j += 32) out[j] = T(0);
        __syncwarp();             // the row is clear before any of its kept entries is written
        const int16_t* cr = cols + row * k;
        const T* vr = vals + row * k;
        for (uint32_t s = lane; s < k; s += 32) {
            const uint32_t c = static_cast<uint16_t>(__ldg(cr + s));
            if (c < d) out[c] = __ldg(vr + s); else bad = true;
        }
    }
    if (bad && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_BAD_MASK));
}

// Fast path for rows that start on 16-byte boundaries and are at most 16 KiB long: every warp builds its
// row in shared memory (clear, scatter the k kept values) and writes it out with 128-bit streaming stores, so HBM only
// sees full, sequential 16-byte-aligned writes.
constexpr int kUnpackWarps = 8;
// kSlots > 0: the row's entries (k <= 32 kSlots) in registers, fetched one row ahead; kSlots == 0: any k, the entries
// read as they are scattered; kSlots == -1: the same for the denser k, where zeroing the whole row buffer again (one
// 128-bit store per 16 bytes) is cheaper than clearing the k positions one by one.
template <typename T, int kSlots>
__global__ void __launch_bounds__(kUnpackWarps * 32)
mp_unpack_staged_kernel(const int16_t* __restrict__ cols, const T* __restrict__ vals, uint32_t rows, uint32_t d,
                        uint32_t ld, uint32_t k, T* __restrict__ dense, dct_result_t* __restrict__ result) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lane = lane_id(), warp = threadIdx.x >> 5;
    const uint32_t row_bytes = d * static_cast<uint32_t>(sizeof(T));          // a multiple of 16
    T* buf = reinterpret_cast<T*>(smem_raw + static_cast<size_t>(warp) * row_bytes);
    bool bad = false;
    const uint64_t first_row = static_cast<uint64_t>(blockIdx.x) * kUnpackWarps + warp;
    const uint64_t row_step = static_cast<uint64_t>(gridDim.x) * kUnpackWarps;
    uint4* b16 = reinterpret_cast<uint4*>(buf);
    // The warp's row buffer is zeroed once; a row is scattered into it, leaves as 128-bit streaming stores (measured:
    // 29.9 us for 16384x4096 bf16 against 34.3 us with a bulk store per row and 36.5 us when the whole buffer was
    // zeroed again for every row), and only the positions it had written are cleared again.
    for (uint32_t v = lane; v < row_bytes / 16; v += 32) b16[v] = make_uint4(0, 0, 0, 0);
    auto write_out = [&](uint64_t row) {
        uint4* dst = reinterpret_cast<uint4*>(dense + row * ld);
        for (uint32_t v = lane; v < row_bytes / 16; v += 32) __stcs(dst + v, b16[v]);
    };
    if (kSlots > 0) {
        // k <= 32 kSlots: the row's packed entries live in registers, and the next row's are fetched while the
        // current row is written out
        constexpr int kS = kSlots > 0 ? kSlots : 1;
        // (two rows ahead was tried: 34.2 us, the registers cost more warps than the longer reach gains)
        uint32_t c_cur[kS], c_old[kS];
        T v_cur[kS];
        auto fetch = [&](uint64_t row) {
#pragma unroll
            for (int j = 0; j < kS; ++j) {
                const uint32_t sidx = lane + 32u * j;
                c_cur[j] = sidx < k ? static_cast<uint16_t>(__ldg(cols + row * k + sidx)) : 0xFFFFFFFFu;
                if (sidx < k) v_cur[j] = __ldg(vals + row * k + sidx);
            }
        };
#pragma unroll
        for (int j = 0; j < kS; ++j) c_old[j] = 0xFFFFFFFFu;
        if (first_row < rows) fetch(first_row);
        for (uint64_t row = first_row; row < rows; row += row_step) {
            __syncwarp();                          // the previous row has been read out of the buffer
#pragma unroll
            for (int j = 0; j < kS; ++j)
                if (c_old[j] < d) buf[c_old[j]] = T(0);
            __syncwarp();                          // (a column of the old row may be one of the new row's)
#pragma unroll
            for (int j = 0; j < kS; ++j) {
                if (c_cur[j] < d) buf[c_cur[j]] = v_cur[j];
                else if (c_cur[j] != 0xFFFFFFFFu) bad = true;
                c_old[j] = c_cur[j];
            }
            __syncwarp();
            if (row + row_step < rows) fetch(row + row_step);
            write_out(row);
        }
    } else {
        for (uint64_t row = first_row; row < rows; row += row_step) {
            const int16_t* cr = cols + row * k;
            const T* vr = vals + row * k;
            __syncwarp();
            for (uint32_t s0 = lane; s0 < k; s0 += 128) {          // four entries of a lane in flight
                uint32_t c[4];
                T v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t s = s0 + 32u * u;
                    c[u] = s < k ? static_cast<uint16_t>(__ldg(cr + s)) : 0xFFFFFFFFu;
                    if (s < k) v[u] = __ldg(vr + s);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (c[u] < d) buf[c[u]] = v[u];
                    else if (c[u] != 0xFFFFFFFFu) bad = true;
                }
            }
            __syncwarp();
            write_out(row);
            __syncwarp();
            if (kSlots < 0) {
                for (uint32_t v = lane; v < row_bytes / 16; v += 32) b16[v] = make_uint4(0, 0, 0, 0);
            } else {
                for (uint32_t s = lane; s < k; s += 32) {          // (L1 still holds the columns)
                    const uint32_t c = static_cast<uint16_t>(__ldg(cr + s));
                    if (c < d) buf[c] = T(0);
                }
            }
        }
    }
    if (bad && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_BAD_MASK));
}

// (a thread walks all k columns of its row, so the work per row is units * k: beyond ~250 the warp-per-row kernel with
// its shared-memory row wins again -- 393216 rows of 256 bf16 columns, k = 12: 0.231 against 0.094 ms)
constexpr uint32_t kUnpackFlatMaxWork = 256;
// Short rows with few kept columns (the paper's layer widths): one THREAD per 16-byte unit of the dense matrix.  The
// thread reads the k columns of its row (the threads of a row sit in the same warp or the next: the loads are
// broadcasts or L1 hits), puts the values that fall into its unit into four registers and stores the unit; nothing
// goes through shared memory, every lane works, HBM sees full sequential 16-byte writes.  (With a warp per row a row
// of 128 bytes uses 8 of 32 lanes per store: 1572864 rows of 64 bf16 columns, k = 3: 0.354 ms.)  Row and unit advance
// by fixed steps from one of a thread's units to the next, so only the first costs a division.
template <typename T>
__global__ void __launch_bounds__(256)
mp_unpack_flat_kernel(const int16_t* __restrict__ cols, const T* __restrict__ vals, uint32_t rows, uint32_t d,
                      uint32_t ld, uint32_t k, T* __restrict__ dense, dct_result_t* __restrict__ result) {
    constexpr uint32_t per16 = 16 / sizeof(T);
    const uint32_t units = d / per16;                  // 16-byte units of a row
    const uint64_t total = static_cast<uint64_t>(rows) * units;
    const uint64_t round = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    const uint64_t round_q = round / units;
    const uint32_t round_r = static_cast<uint32_t>(round % units);
    uint64_t e = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    uint64_t row = e / units;
    uint32_t unit = static_cast<uint32_t>(e - row * units);
    bool bad = false;
    for (; e < total; e += round) {
        const int16_t* cr = cols + row * k;
        const T* vr = vals + row * k;
        uint32_t w0 = 0, w1 = 0, w2 = 0, w3 = 0;
        for (uint32_t s = 0; s < k; ++s) {
            const uint32_t c = static_cast<uint16_t>(__ldg(cr + s));
            if (c >= d) {
                bad = true;
                continue;
            }
            if (c / per16 != unit) continue;
            const uint32_t p = c % per16;
            if constexpr (sizeof(T) == 2) {
                const uint32_t sh = (p & 1u) * 16u, keep = ~(0xFFFFu << sh);
                const uint32_t v = static_cast<uint32_t>(__ldg(reinterpret_cast<const uint16_t*>(vr) + s)) << sh;
                const uint32_t word = p >> 1;
                w0 = word == 0 ? (w0 & keep) | v : w0;
                w1 = word == 1 ? (w1 & keep) | v : w1;
                w2 = word == 2 ? (w2 & keep) | v : w2;
                w3 = word == 3 ? (w3 & keep) | v : w3;
            } else {
                const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(vr) + s);
                w0 = p == 0 ? v : w0;
                w1 = p == 1 ? v : w1;
                w2 = p == 2 ? v : w2;
                w3 = p == 3 ? v : w3;
            }
        }
        __stcs(reinterpret_cast<uint4*>(dense + row * ld + static_cast<size_t>(unit) * per16), make_uint4(w0, w1, w2, w3));
        row += round_q;
        unit += round_r;
        if (unit >= units) {
            unit -= units;
            ++row;
        }
    }
    if (bad && result) atomicMax(&result->status, static_cast<uint32_t>(DCT_ERR_BAD_MASK));
}

template <typename T>
cudaError_t launch_unpack(const int16_t* cols, const void* vals, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
                          void* dense_out, dct_result_t* result, int sms, cudaStream_t stream) {
    const size_t row_bytes = static_cast<size_t>(d) * sizeof(T);
    const bool staged = aligned_to(dense_out, 16) && (static_cast<size_t>(ld) * sizeof(T)) % 16 == 0 &&
                        row_bytes % 16 == 0 && row_bytes <= 16 * 1024;
    if (staged && (row_bytes / 16) * k <= kUnpackFlatMaxWork) {
        const uint64_t total = static_cast<uint64_t>(rows) * (row_bytes / 16);
        const uint64_t need = (total + 255) / 256;
        const uint64_t cap = static_cast<uint64_t>(sms) * 32;
        mp_unpack_flat_kernel<T><<<static_cast<unsigned>(need < cap ? need : cap), 256, 0, stream>>>(
            cols, static_cast<const T*>(vals), rows, d, ld, k, static_cast<T*>(dense_out), result);
    } else if (staged) {
        const size_t smem = kUnpackWarps * row_bytes;
        // (the denser k, more than an eighth of the row: zero the whole buffer instead of the k positions)
        const bool zero_all = static_cast<size_t>(k) * (sizeof(T) == 2 ? 16 : 32) > row_bytes;     // k > d / 8
        auto kernel = zero_all ? mp_unpack_staged_kernel<T, -1>
                               : (k <= 256 ? mp_unpack_staged_kernel<T, 8>
                                           : (k <= 512 ? mp_unpack_staged_kernel<T, 16> : mp_unpack_staged_kernel<T, 0>));
        // (static shared memory counts against the 48 KiB a kernel gets without asking: ask well below that)
        if (smem > 32 * 1024) {
            const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                       static_cast<int>(kUnpackWarps * 16 * 1024));
            if (e != cudaSuccess) return e;
        }
        size_t per_sm = (200 * 1024) / (smem + 1024);
        if (per_sm < 1) per_sm = 1;
        if (per_sm > 8) per_sm = 8;
        const uint64_t ctas_needed = (static_cast<uint64_t>(rows) + kUnpackWarps - 1) / kUnpackWarps;
        const uint64_t max_grid = static_cast<uint64_t>(sms) * per_sm;
        const unsigned grid = static_cast<unsigned>(ctas_needed < max_grid ? ctas_needed : max_grid);
        kernel<<<grid, kUnpackWarps * 32, smem, stream>>>(cols, static_cast<const T*>(vals), rows, d, ld, k,
                                                          static_cast<T*>(dense_out), result);
    } else {
        const uint64_t ctas_needed = (static_cast<uint64_t>(rows) + 7) / 8;
        const uint64_t max_grid = static_cast<uint64_t>(sms) * 8;
        const unsigned grid = static_cast<unsigned>(ctas_needed < max_grid ? ctas_needed : max_grid);
        mp_unpack_kernel<T><<<grid, 256, 0, stream>>>(cols, static_cast<const T*>(vals), rows, d, ld, k,
                                                      static_cast<T*>(dense_out), result);
    }
    return cudaGetLastError();
}

}  // namespace
}  // namespace dct

using namespace dct;

extern "C" dct_status_t dct_dp_decompress(const int32_t* idx, const float* val, const dct_result_t* packed,
                                          uint64_t capacity, float* dense, uint64_t n, int accumulate,
                                          dct_result_t* result, dct_stream_t stream_) {
    if (!packed || !dense || !result || n == 0 || n > 0x7FFFFFFFull) return DCT_ERR_INVALID_ARG;
    if (capacity > 0 && (!idx || !val)) return DCT_ERR_INVALID_ARG;
    if (capacity > 0x7FFFFFFFull) capacity = 0x7FFFFFFFull;
    if (!aligned_to(idx, 4) || !aligned_to(val, 4) || !aligned_to(dense, 4) || !aligned_to(packed, 8) ||
        !aligned_to(result, 8) || packed == result)
        return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    DCT_CUDA_TRY(cudaMemsetAsync(result, 0, sizeof(dct_result_t), stream));
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    // enough CTAs to fill the machine, but at least 1024 elements of the dense vector each
    uint64_t grid = static_cast<uint64_t>(sms) * 8;
    const uint64_t by_size = (n + 1023) / 1024;
    if (grid > by_size) grid = by_size;
    // ... and at most 16384 elements (64 KB) each: the CTAs at work then write neighbouring ranges instead of 1184
    // streams spread over the whole vector (2^30 elements: 0.749 -> 0.620 ms; ranges of 8192 or 32768 are slower)
    const uint64_t by_range = (n + 16383) / 16384;
    if (grid < by_range) grid = by_range;
    // (a dense vector 4, 8 or 12 bytes past a 16-byte boundary is written from that boundary on, its neighbours before it
    // left alone)
    const uint32_t lead = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(dense) & 15u) / 4u);
    if (lead == 0)
        dp_decompress_tiled_kernel<false><<<static_cast<unsigned>(grid), 256, 0, stream>>>(
            idx, val, packed, capacity, dense, static_cast<uint32_t>(n), accumulate, result, 0u);
    else if (n + lead <= 0x7FFFFFFFull)
        dp_decompress_tiled_kernel<true><<<static_cast<unsigned>(grid), 256, 0, stream>>>(
            idx, val, packed, capacity, dense - lead, static_cast<uint32_t>(n) + lead, accumulate, result, lead);
    else
        dp_decompress_kernel<<<static_cast<unsigned>(grid), 256, 0, stream>>>(idx, val, packed, capacity, dense,
                                                                             static_cast<uint32_t>(n), accumulate, result);
    DCT_CUDA_TRY(cudaGetLastError());
    return DCT_OK;
}

extern "C" dct_status_t dct_mp_unpack(const int16_t* cols, const void* vals, dct_dtype_t dtype, uint32_t rows,
                                      uint32_t d, uint32_t ld, uint32_t k, void* dense_out, dct_result_t* result,
                                      dct_stream_t stream_) {
    if (!cols || !vals || !dense_out || rows == 0 || d == 0 || k == 0 || k > d || ld < d || d > 32768u)
        return DCT_ERR_INVALID_ARG;
    if (dtype != DCT_F32 && dtype != DCT_BF16) return DCT_ERR_UNSUPPORTED;
    const size_t es = dtype == DCT_F32 ? 4 : 2;
    if (!aligned_to(vals, es) || !aligned_to(dense_out, es) || !aligned_to(cols, 2) || (result && !aligned_to(result, 8)))
        return DCT_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (result) DCT_CUDA_TRY(cudaMemsetAsync(result, 0, sizeof(dct_result_t), stream));
    const int sms = sm_count();
    if (sms <= 0) return DCT_ERR_CUDA;
    if (dtype == DCT_F32)
        DCT_CUDA_TRY(launch_unpack<float>(cols, vals, rows, d, ld, k, dense_out, result, sms, stream));
    else
        DCT_CUDA_TRY(launch_unpack<uint16_t>(cols, vals, rows, d, ld, k, dense_out, result, sms, stream));
    return DCT_OK;
}
