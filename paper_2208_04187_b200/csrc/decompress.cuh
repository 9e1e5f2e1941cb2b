// Decompress kernels (DIVISION Sec. 4.2, Eq. 10; Algorithm 1, backward loop):
//   x_hat = UpSampling(H^L) + (Delta * V^H + delta), rounded to the activation dtype.
// One fused pass: unpack, dequantise, add the nearest-upsampled low-frequency value, store.
#pragma once

#include "common.cuh"
#include "twopass.cuh"   // Shape

namespace divk {

// ---------------------------------------------------------------------------------------------
// general kernel: one thread per packed word, any shape
// ---------------------------------------------------------------------------------------------
template <typename XT, typename LT, int Q>
__global__ void __launch_bounds__(256)
decompress_general_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                          const float* __restrict__ stats, XT* __restrict__ xhat, Shape s, uint64_t nwords) {
    constexpr uint32_t PER = 32 / Q;
    constexpr uint32_t MASK = (Q == 32) ? 0xFFFFFFFFu : ((1u << Q) - 1u);
    const uint64_t word = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= nwords) return;
    uint64_t i = word * PER;
    uint32_t n = (uint32_t)(i / s.CHW);
    uint32_t e = (uint32_t)(i - (uint64_t)n * s.CHW);
    uint32_t plane = e / s.HW;
    uint32_t rem = e - plane * s.HW;
    uint32_t h = rem / s.W, w = rem - h * s.W;
    const uint32_t bits = packed[word];
    uint32_t cur_n = 0xFFFFFFFFu;
    float delta = 0.f, step = 0.f;
    for (uint32_t j = 0; j < PER && i < s.total; ++j, ++i) {
        if (n != cur_n) {
            delta = stats[2 * (size_t)n];
            step = stats[2 * (size_t)n + 1];
            cur_n = n;
        }
        const size_t lidx = ((size_t)n * s.C + plane) * s.TPP + (h / s.B) * s.Wb + (w / s.B);
        const float l = Elem<LT>::load(lfc + lidx);
        Elem<XT>::store(xhat + i, reconstruct((bits >> (j * Q)) & MASK, step, delta, l));
        if (++w == s.W) {
            w = 0;
            if (++h == s.H) {
                h = 0;
                if (++plane == s.C) {
                    plane = 0;
                    ++n;
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// vector kernel: W % 4 == 0, B a power of two >= 4 (so that 4 consecutive elements share a tile).
// One thread produces QPT quads (4 elements each, one 16-byte or 8-byte store); quads of a warp are
// consecutive, so every store instruction of a warp writes one contiguous 512-byte (fp32) span.
// grid = (ceil(quads_per_sample / (256*QPT)), N)
// ---------------------------------------------------------------------------------------------
struct DecFast {
    uint32_t qps;        // quads per sample = CHW / 4
    uint32_t C, TPP, Wb;
    uint32_t log2B;
    FastDiv by_hwq;      // / (HW/4)
    FastDiv by_wq;       // / (W/4)
    uint32_t hwq, wq;
};

template <typename XT> struct Quad;
template <> struct Quad<float> {
    static __device__ __forceinline__ void store(float* p, float a, float b, float c, float d) {
        __stcs(reinterpret_cast<float4*>(p), make_float4(a, b, c, d));
    }
};
template <> struct Quad<__nv_bfloat16> {
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float a, float b, float c, float d) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
        uint2 v;
        v.x = *reinterpret_cast<uint32_t*>(&lo);
        v.y = *reinterpret_cast<uint32_t*>(&hi);
        __stcs(reinterpret_cast<uint2*>(p), v);
    }
};

template <typename XT, typename LT, int Q, int QPT>
__global__ void __launch_bounds__(256)
decompress_quad_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                       const float* __restrict__ stats, XT* __restrict__ xhat, DecFast d) {
    constexpr uint32_t QMASK = (1u << Q) - 1u;
    constexpr uint32_t GMASK = (Q == 8) ? 0xFFFFFFFFu : ((1u << (4 * Q)) - 1u);
    const uint32_t n = blockIdx.y;
    const float delta = __ldg(stats + 2 * (size_t)n);
    const float step = __ldg(stats + 2 * (size_t)n + 1);
    const uint64_t sample_quad0 = (uint64_t)n * d.qps;
    const LT* lfc_n = lfc + (size_t)n * d.C * d.TPP;
    const uint32_t q0 = blockIdx.x * (256u * QPT) + threadIdx.x;

    uint32_t bits[QPT];
    float lf[QPT];
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < d.qps) {
            const uint64_t bitpos = (sample_quad0 + q) * (4u * Q);
            bits[k] = (__ldg(packed + (bitpos >> 5)) >> (uint32_t)(bitpos & 31u)) & GMASK;
            const uint32_t plane = fdiv(q, d.by_hwq);
            const uint32_t rem = q - plane * d.hwq;
            const uint32_t h = fdiv(rem, d.by_wq);
            const uint32_t wq = rem - h * d.wq;
            lf[k] = Elem<LT>::load(lfc_n + (size_t)plane * d.TPP + (h >> d.log2B) * d.Wb + ((wq * 4u) >> d.log2B));
        }
    }
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < d.qps) {
            const uint32_t b = bits[k];
            Quad<XT>::store(xhat + (sample_quad0 + q) * 4u,
                            reconstruct(b & QMASK, step, delta, lf[k]),
                            reconstruct((b >> Q) & QMASK, step, delta, lf[k]),
                            reconstruct((b >> (2 * Q)) & QMASK, step, delta, lf[k]),
                            reconstruct((b >> (3 * Q)) & QMASK, step, delta, lf[k]));
        }
    }
}

}  // namespace divk
