// ReLU and dropout operators with a packed 1-bit mask (the paper's appendix algorithms "Relu operator" and
// "Dropout operator": V = mask, H_out = V (.) H_in, V packed and cached; backward grad_in = V (.) grad_out;
// N^2/8 bytes per plane in the byte count of Theorem 3A's proof).
//
// Pure streaming work, bound by HBM: a thread takes 8 consecutive elements (32 bytes of fp32, one 16-byte load of
// bf16), so a warp reads 1 KB of contiguous x, writes the same of y and 32 contiguous mask bytes.
//   ReLU     V = [H > 0] (zeros of either sign and NaN give 0); masked outputs are +0.0
//   dropout  V = [field >= drop_threshold], field = the 16-bit DIVRNG-v1 number of (seed, sample 0, flat index i);
//            no rescaling (the paper's algorithm has none)
//   packing  bit (i mod 32) of little-endian 32-bit word i / 32; the mask buffer is addressed in bytes here
#pragma once

#include "common.cuh"

namespace divk {

template <typename T> struct Oct;
template <> struct Oct<float> {
    static __device__ __forceinline__ void load(const float* p, float (&v)[8]) {
        const float4 a = __ldcs(reinterpret_cast<const float4*>(p)), b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
    static __device__ __forceinline__ void store(float* p, const float (&v)[8]) {
        __stcs(reinterpret_cast<float4*>(p), make_float4(v[0], v[1], v[2], v[3]));
        __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(v[4], v[5], v[6], v[7]));
    }
};
template <> struct Oct<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
        const uint4 a = __ldcs(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    // the values are bfloat16 numbers already (kept inputs or +0.0): the upper half-words are exact
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = (__float_as_uint(v[2 * i]) >> 16) | (__float_as_uint(v[2 * i + 1]) & 0xFFFF0000u);
        __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
    }
};

// 64-bit group counter form of the random stream (see common.cuh): the groups of sample 0
__device__ __forceinline__ uint64_t rng_group64(uint64_t base, uint64_t g) {
    uint64_t z = base + K_GROUP * (g + 1ull);
    z ^= z >> 32;
    z *= K_MIX;
    z ^= z >> 32;
    z *= K_MIX;
    z ^= z >> 32;
    return z;
}

// keep bits of the 8 elements starting at i0 (a multiple of 8)
template <bool DROPOUT>
__device__ __forceinline__ uint32_t keep_bits(const float (&v)[8], uint64_t i0, uint64_t base, uint32_t thr) {
    uint32_t bits = 0;
    if (DROPOUT) {
        const uint64_t z0 = rng_group64(base, i0 >> 2), z1 = rng_group64(base, (i0 >> 2) + 1ull);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            bits |= (((uint32_t)(z0 >> (16 * j)) & 0xFFFFu) >= thr ? 1u : 0u) << j;
            bits |= (((uint32_t)(z1 >> (16 * j)) & 0xFFFFu) >= thr ? 1u : 0u) << (4 + j);
        }
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) bits |= (v[j] > 0.f ? 1u : 0u) << j;
    }
    return bits;
}

// x and y may be the same buffer (every thread reads its 8 elements before it writes them)
template <typename XT, bool DROPOUT>
__global__ void __launch_bounds__(256)
mask_forward_kernel(const XT* x, XT* y, uint8_t* mask, uint64_t total, uint64_t base, uint32_t thr) {
    const uint64_t oct = (uint64_t)blockIdx.x * 256u + threadIdx.x;
    const uint64_t i0 = oct * 8u;
    if (i0 >= total) return;
    float v[8];
    if (i0 + 8u <= total) {
        Oct<XT>::load(x + i0, v);
        const uint32_t bits = keep_bits<DROPOUT>(v, i0, base, thr);
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = ((bits >> j) & 1u) ? v[j] : 0.f;
        Oct<XT>::store(y + i0, v);
        mask[oct] = (uint8_t)bits;
    } else {
        const uint32_t cnt = (uint32_t)(total - i0);       // ragged end: 1..7 elements
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (uint32_t)j < cnt ? Elem<XT>::load(x + i0 + j) : 0.f;
        uint32_t bits = keep_bits<DROPOUT>(v, i0, base, thr) & ((1u << cnt) - 1u);
        for (uint32_t j = 0; j < cnt; ++j) Elem<XT>::store(y + i0 + j, ((bits >> j) & 1u) ? v[j] : 0.f);
        mask[oct] = (uint8_t)bits;
    }
}

template <typename XT>
__global__ void __launch_bounds__(256)
mask_backward_kernel(const uint8_t* __restrict__ mask, const XT* g, XT* gin, uint64_t total) {
    const uint64_t oct = (uint64_t)blockIdx.x * 256u + threadIdx.x;
    const uint64_t i0 = oct * 8u;
    if (i0 >= total) return;
    const uint32_t bits = __ldg(mask + oct);
    float v[8];
    if (i0 + 8u <= total) {
        Oct<XT>::load(g + i0, v);
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = ((bits >> j) & 1u) ? v[j] : 0.f;
        Oct<XT>::store(gin + i0, v);
    } else {
        const uint32_t cnt = (uint32_t)(total - i0);
        for (uint32_t j = 0; j < cnt; ++j) {
            const float val = Elem<XT>::load(g + i0 + j);
            Elem<XT>::store(gin + i0 + j, ((bits >> j) & 1u) ? val : 0.f);
        }
    }
}

}  // namespace divk
