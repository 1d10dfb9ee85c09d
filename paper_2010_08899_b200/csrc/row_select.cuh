// Exact k-th largest magnitude of one row held in shared memory, by a whole CTA: the row threshold
// tau_i of Algorithm 2 (DCT-MP).  Most-significant-digit-first radix select over key(x) with 8-bit
// digits: 4 passes for fp32's 31 key bits, 2 for bf16's 15.
#pragma once
#include "common.cuh"

namespace dct {

template <typename T> struct ElemTraits;
template <> struct ElemTraits<float> {
    static constexpr int kPasses = 4;
    __device__ static __forceinline__ uint32_t key(float x) { return key_f32(x); }
    __device__ static __forceinline__ float from_key(uint32_t k) { return __uint_as_float(k); }
    __device__ static __forceinline__ double to_double(float x) { return static_cast<double>(x); }
    __host__ __device__ static constexpr int shift(int p) { return p == 0 ? 23 : (p == 1 ? 15 : (p == 2 ? 7 : 0)); }
    __host__ __device__ static constexpr int bits(int p) { return p == 3 ? 7 : 8; }
};
template <> struct ElemTraits<uint16_t> {   // bf16 carried as its bit pattern
    static constexpr int kPasses = 2;
    __device__ static __forceinline__ uint32_t key(uint16_t x) { return key_bf16(x); }
    __device__ static __forceinline__ uint16_t from_key(uint32_t k) { return static_cast<uint16_t>(k); }
    __device__ static __forceinline__ double to_double(uint16_t x) {
        return static_cast<double>(__uint_as_float(static_cast<uint32_t>(x) << 16));
    }
    __host__ __device__ static constexpr int shift(int p) { return p == 0 ? 7 : 0; }
    __host__ __device__ static constexpr int bits(int p) { return p == 0 ? 8 : 7; }
};

// Called by every thread of the CTA with the same arguments; row_s[0..d) must have been written
// before the call (the first barrier inside orders those writes before the first read).
//   s_hist  256 words of shared memory;  s_sel  2 words of shared memory.
// On return every thread has tau_key = the k-th largest key of the row and take = how many of the
// elements whose key equals tau_key belong to the top k (ties: the caller keeps the lowest columns).
// The call ends with a barrier, so it may be repeated at once with another k.
template <typename T>
__device__ __forceinline__ void cta_row_select(const T* row_s, uint32_t d, uint32_t k, uint32_t* s_hist,
                                               uint32_t* s_sel, uint32_t& tau_key, uint32_t& take) {
    using Tr = ElemTraits<T>;
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    const uint32_t lane = tid & 31u, warp = tid >> 5;
    if (tid == 0) {
        s_sel[0] = 0;      // digits chosen so far
        s_sel[1] = k;      // rank still to be located inside the prefix bucket
    }
#pragma unroll
    for (int p = 0; p < Tr::kPasses; ++p) {
        const int shift = Tr::shift(p), bits = Tr::bits(p);
        const uint32_t nbins = 1u << bits;
        for (uint32_t b = tid; b < 256; b += nt) s_hist[b] = 0;
        __syncthreads();
        const uint32_t prefix = s_sel[0];
        // Exact zeros are the common value after a ReLU: in the first pass they are counted in a register
        // and added to bin 0 once per thread instead of colliding on one shared-memory word.
        uint32_t zeros = 0;
        for (uint32_t j = tid; j < d; j += nt) {
            const uint32_t key = Tr::key(row_s[j]);
            if (p == 0 && key == 0) {
                ++zeros;
            } else if (p == 0 || (key >> (shift + bits)) == prefix) {
                atomicAdd(&s_hist[(key >> shift) & (nbins - 1u)], 1u);
            }
        }
        if (zeros) atomicAdd(&s_hist[0], zeros);
        __syncthreads();
        if (warp == 0) {
            // lane owns 8 bins, top-down: bin(lane, q) = 255 - (8 lane + q); bins >= nbins are empty
            const uint32_t k_rem = s_sel[1];
            uint32_t c[8], own = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                c[q] = s_hist[255 - (8 * lane + q)];
                own += c[q];
            }
            uint32_t incl = own;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= static_cast<uint32_t>(o)) incl += t;
            }
            uint32_t above = incl - own;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                if (above < k_rem && k_rem <= above + c[q]) {
                    s_sel[0] = (prefix << bits) | (255u - (8u * lane + q));
                    s_sel[1] = k_rem - above;
                }
                above += c[q];
            }
        }
        __syncthreads();
    }
    tau_key = s_sel[0];
    take = s_sel[1];
    __syncthreads();
}

}  // namespace dct
