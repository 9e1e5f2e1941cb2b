// Device-side building blocks shared by the compress and decompress kernels.
//
// Arithmetic contract (DIVISION Sec. 4.1, Eq. 9; Sec. 4.2, Eq. 10): IEEE fp32, one rounding per
// operation.  The _rn intrinsics below keep the compiler from contracting a multiply and an add
// into a fused multiply-add where two roundings are specified.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace divk {

// ---------------------------------------------------------------------------------------------
// workspace layout (device scratch owned by the caller)
//   word 0          : device status (0 = ok, 7 = a bounded wait ran out)
//   word 1          : detail of the first failure (sample index)
//   words 16 + 32n.. : per-sample slot of 128 bytes (one cache line each, so that the slots of
//                      neighbouring samples do not share an L2 line): { ~key(min), key(max), arrivals,
//                      unused, 64-bit parameter word (general fused kernel), unused ... }
// key() maps a float to an unsigned integer with the same ordering, so that integer atomicMax
// implements float max (and, on the complemented key, float min).  All-zero is the neutral state.
// ---------------------------------------------------------------------------------------------
constexpr int WS_HEADER_WORDS = 16;
constexpr int WS_SLOT_WORDS = 32;

__device__ __forceinline__ uint32_t float_key(float f) {
    uint32_t b = __float_as_uint(f);
    return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
    uint32_t b = (k & 0x80000000u) ? (k ^ 0x80000000u) : ~k;
    return __uint_as_float(b);
}

// ---------------------------------------------------------------------------------------------
// element types
// ---------------------------------------------------------------------------------------------
template <typename T> struct Elem;
template <> struct Elem<float> {
    static __device__ __forceinline__ float load(const float* p) { return *p; }
    static __device__ __forceinline__ float load_cg(const float* p) { return __ldcg(p); }
    static __device__ __forceinline__ void store(float* p, float v) { *p = v; }
    static __device__ __forceinline__ float round(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ float load_cg(const __nv_bfloat16* p) {
        return __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short*>(p)) << 16);
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
    static __device__ __forceinline__ float round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
};

// ---------------------------------------------------------------------------------------------
// DIVRNG-v1: counter-based uniforms, one 64-bit mix per group of 4 consecutive elements.
//   z = seed ^ (K_SAMPLE * (n+1));  z += K_GROUP * (g+1);  three xor-shifts by 32 around two
//   multiplications by K_MIX;  element e uses bits [16*(e&3), 16*(e&3)+16) of z as u * 2^16.
// ---------------------------------------------------------------------------------------------
constexpr uint64_t K_SAMPLE = 0x9E3779B97F4A7C15ull;
constexpr uint64_t K_GROUP = 0xD1B54A32D192ED03ull;
constexpr uint64_t K_MIX = 0xD6E8FEB86659FD93ull;

__host__ __device__ __forceinline__ uint64_t rng_sample_base(uint64_t seed, uint32_t n) {
    return seed ^ (K_SAMPLE * ((uint64_t)n + 1ull));
}
__device__ __forceinline__ uint64_t rng_group(uint64_t base, uint32_t g) {
    uint64_t z = base + K_GROUP * (uint64_t)(g + 1u);
    z ^= z >> 32;
    z *= K_MIX;
    z ^= z >> 32;
    z *= K_MIX;
    z ^= z >> 32;
    return z;
}

// ---------------------------------------------------------------------------------------------
// per-sample quantisation parameters from the residual extremes (Eq. 9)
// ---------------------------------------------------------------------------------------------
struct QParams {
    float delta;   // min residual
    float step;    // Delta = (max - min) / (2^Q - 1)
    float scale;   // (2^Q - 1) / (max - min); 0 when the residual is constant
};
__device__ __forceinline__ QParams make_qparams(float rmin, float rmax, int qbits) {
    QParams q;
    const float qmax = (float)((1 << qbits) - 1);
    const float range = __fsub_rn(rmax, rmin);
    q.delta = rmin;
    q.step = 0.f;
    q.scale = 0.f;
    if (range > 0.f) {
        const float s = __fdiv_rn(qmax, range);
        if (s <= 3.402823466e+38f) {          // finite
            q.scale = s;
            q.step = __fdiv_rn(range, qmax);
        }
    }
    return q;
}

// Magic constant 1.5 * 2^23: floats in [2^23, 2^24) are the integers, so adding it with rounding
// towards +inf leaves ceil(d) in the low mantissa bits for any d in (-1, 255].
constexpr float MAGIC_CEIL = 12582912.0f;
constexpr uint32_t MAGIC_CEIL_BITS = 0x4B400000u;

// Code of one element (Eq. 9 with stochastic rounding): floor(t) + [u < frac(t)], clamped.
// Computed as ceil(min(t, qmax) - u): u < frac(t)  <=>  ceil(frac(t) - u) = 1, and t - u is exact in
// fp32 whenever it is positive (its sign is kept otherwise), so both forms give the same integer.
// `field16` is the 16-bit random field; returns MAGIC_CEIL_BITS + code.
__device__ __forceinline__ uint32_t quant_bits(float r, float delta, float scale, float qmax, uint32_t field16) {
    float t = __fmul_rn(__fsub_rn(r, delta), scale);
    t = fminf(t, qmax);
    const float fieldf = __fsub_rn(__uint_as_float(0x4B000000u | field16), 8388608.0f);   // exact
    const float d = __fmaf_rn(fieldf, -1.52587890625e-05f, t);                             // fl(t - u)
    return __float_as_uint(__fadd_ru(d, MAGIC_CEIL));
}

// four elements sharing one 64-bit random word; returns their codes packed Q bits apart
template <int Q>
__device__ __forceinline__ uint32_t quant4(float r0, float r1, float r2, float r3, float delta, float scale,
                                           uint64_t z) {
    constexpr float qmax = (float)((1 << Q) - 1);
    const uint32_t lo = (uint32_t)z, hi = (uint32_t)(z >> 32);
    const uint32_t b0 = quant_bits(r0, delta, scale, qmax, lo & 0xFFFFu);
    const uint32_t b1 = quant_bits(r1, delta, scale, qmax, lo >> 16);
    const uint32_t b2 = quant_bits(r2, delta, scale, qmax, hi & 0xFFFFu);
    const uint32_t b3 = quant_bits(r3, delta, scale, qmax, hi >> 16);
    constexpr uint32_t BIAS = MAGIC_CEIL_BITS * (1u + (1u << Q) + (1u << (2 * Q)) + (1u << (3 * Q)));   // mod 2^32
    uint32_t acc = b0 + (b1 << Q) + (b2 << (2 * Q)) + (b3 << (3 * Q));
    return acc - BIAS;
}

// Dequantise one code (Sec. 4.2): fl(fl(Delta * code) + delta).
__device__ __forceinline__ float dequantise(uint32_t code, float step, float delta) {
    const float cf = __fsub_rn(__uint_as_float(0x4B000000u | code), 8388608.0f);   // (float)code, exact
    return __fadd_rn(__fmul_rn(step, cf), delta);
}

// Dequantise and reconstruct one element (Sec. 4.2): x_hat = lfc + (Delta * code + delta).
__device__ __forceinline__ float reconstruct(uint32_t code, float step, float delta, float lfc) {
    const float cf = __fsub_rn(__uint_as_float(0x4B000000u | code), 8388608.0f);   // (float)code, exact
    return __fadd_rn(lfc, __fadd_rn(__fmul_rn(step, cf), delta));
}

// division of a 31-bit number by a runtime constant: q = (n * mul) >> shift, exact for n < 2^31
struct FastDiv {
    uint32_t d, mul, shift;
};
__device__ __forceinline__ uint32_t fdiv(uint32_t n, const FastDiv& f) {
    return (uint32_t)(((uint64_t)n * f.mul) >> f.shift);
}

}  // namespace divk
