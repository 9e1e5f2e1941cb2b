// General two-pass compress kernels: any shape, any block size, any Q in {1,2,4,8}.
//
//   pass 1 (lfc_stats_kernel):  one thread per B x B tile: block mean -> stored low-frequency value
//                               (Sec. 4.1), residual extremes of the tile -> per-sample min / max.
//   pass 2 (quant_pack_kernel): one thread per packed 32-bit word: residual against the stored
//                               low-frequency value, Eq. 9 with stochastic rounding, bit packing.
//
// x is read twice, so this path is the fallback for descriptors the fused single-pass kernel does
// not cover (block sizes that are not a power of two or exceed 32, samples whose size is not a
// multiple of the packing unit, samples too large to keep on chip).
#pragma once

#include "common.cuh"

namespace divk {

struct Shape {
    uint32_t N, C, H, W, B, Hb, Wb, P2;   // P2 = smallest power of two >= B
    uint32_t HW, CHW, TPP;                // TPP = Hb * Wb tiles per plane
    uint64_t total;                       // N * CHW
    uint64_t tiles;                       // N * C * TPP
};

// Balanced pairwise sum of P2 (a power of two) values produced by `fetch(i)`, neighbours first.
template <typename F>
__device__ __forceinline__ float tree_sum(uint32_t p2, F fetch) {
    float level[33];
    for (uint32_t i = 0; i < p2; ++i) {
        float v = fetch(i);
        int k = 0;
        while (i & (1u << k)) {
            v = __fadd_rn(level[k], v);
            ++k;
        }
        level[k] = v;
    }
    return level[31 - __clz(p2)];
}

// mean of one tile in the fixed summation order; also min / max of its in-bounds elements
template <typename XT>
__device__ __forceinline__ float tile_mean(const XT* __restrict__ plane, const Shape& s, uint32_t bh, uint32_t bw,
                                           float& xmin, float& xmax) {
    const uint32_t h0 = bh * s.B, w0 = bw * s.B;
    const uint32_t rows = min(s.B, s.H - h0), cols = min(s.B, s.W - w0);
    const XT* base = plane + (size_t)h0 * s.W + w0;
    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
    const float total = tree_sum(s.P2, [&](uint32_t c) -> float {
        if (c >= cols) return 0.f;
        return tree_sum(s.P2, [&](uint32_t r) -> float {
            if (r >= rows) return 0.f;
            const float v = Elem<XT>::load(base + (size_t)r * s.W + c);
            lo = fminf(lo, v);
            hi = fmaxf(hi, v);
            return v;
        });
    });
    xmin = lo;
    xmax = hi;
    return __fdiv_rn(total, (float)(rows * cols));
}

template <typename XT, typename LT>
__global__ void __launch_bounds__(256)
lfc_stats_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, Shape s) {
    const uint64_t gt = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = gt < s.tiles;
    uint32_t n = 0xFFFFFFFFu;
    float rmin = 0.f, rmax = 0.f;
    if (active) {
        const uint64_t plane_id = gt / s.TPP;
        const uint32_t idx = (uint32_t)(gt - plane_id * s.TPP);
        n = (uint32_t)(plane_id / s.C);
        float xmin, xmax;
        const float mean = tile_mean(x + plane_id * s.HW, s, idx / s.Wb, idx % s.Wb, xmin, xmax);
        Elem<LT>::store(lfc + gt, mean);
        const float stored = Elem<LT>::round(mean);
        // x -> fl(x - stored) is monotone, so the residual extremes are those of the extreme x
        rmin = __fsub_rn(xmin, stored);
        rmax = __fsub_rn(xmax, stored);
    }
    // one atomic pair per warp when the whole warp sits in one sample, else one per thread
    const uint32_t n0 = __shfl_sync(0xFFFFFFFFu, n, 0);
    if (__all_sync(0xFFFFFFFFu, n == n0)) {
        if (n0 == 0xFFFFFFFFu) return;
        uint32_t kmin = ~float_key(rmin), kmax = float_key(rmax);
        kmin = __reduce_max_sync(0xFFFFFFFFu, kmin);
        kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
        if ((threadIdx.x & 31) == 0) {
            uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n0 * WS_SLOT_WORDS;
            atomicMax(slot + 0, kmin);
            atomicMax(slot + 1, kmax);
        }
    } else if (active) {
        uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
        atomicMax(slot + 0, ~float_key(rmin));
        atomicMax(slot + 1, float_key(rmax));
    }
}

template <typename XT, typename LT, int Q>
__global__ void __launch_bounds__(256)
quant_pack_kernel(const XT* __restrict__ x, const LT* __restrict__ lfc, const uint32_t* __restrict__ ws,
                  uint32_t* __restrict__ packed, float* __restrict__ stats, Shape s, uint64_t seed,
                  uint64_t nwords) {
    constexpr uint32_t PER = 32 / Q;
    constexpr float qmax = (float)((1 << Q) - 1);
    const uint64_t word = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= nwords) return;
    uint64_t i = word * PER;
    uint32_t n = (uint32_t)(i / s.CHW);
    uint32_t e = (uint32_t)(i - (uint64_t)n * s.CHW);
    uint32_t plane = e / s.HW;
    uint32_t rem = e - plane * s.HW;
    uint32_t h = rem / s.W, w = rem - h * s.W;

    uint32_t cur_n = 0xFFFFFFFFu;
    uint32_t cur_g = 0xFFFFFFFFu;
    uint64_t base = 0, z = 0;
    QParams qp = {0.f, 0.f, 0.f};
    uint32_t acc = 0;
    for (uint32_t j = 0; j < PER && i < s.total; ++j, ++i) {
        if (n != cur_n) {
            const uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
            qp = make_qparams(key_float(~slot[0]), key_float(slot[1]), Q);
            base = rng_sample_base(seed, n);
            cur_n = n;
            cur_g = 0xFFFFFFFFu;
        }
        if (e == 0) {               // the thread holding a sample's first element publishes its stats
            stats[2 * (size_t)n + 0] = qp.delta;
            stats[2 * (size_t)n + 1] = qp.step;
        }
        const uint32_t g = e >> 2;
        if (g != cur_g) {
            z = rng_group(base, g);
            cur_g = g;
        }
        const size_t lidx = ((size_t)n * s.C + plane) * s.TPP + (h / s.B) * s.Wb + (w / s.B);
        const float l = Elem<LT>::load(lfc + lidx);
        const float r = __fsub_rn(Elem<XT>::load(x + i), l);
        const uint32_t field = (uint32_t)(z >> (16 * (e & 3))) & 0xFFFFu;
        const uint32_t code = quant_bits(r, qp.delta, qp.scale, qmax, field) - MAGIC_CEIL_BITS;
        acc |= code << (j * Q);
        // advance (n, e, plane, h, w)
        ++e;
        if (++w == s.W) {
            w = 0;
            if (++h == s.H) {
                h = 0;
                if (++plane == s.C) {
                    plane = 0;
                    e = 0;
                    ++n;
                }
            }
        }
    }
    packed[word] = acc;
}

}  // namespace divk
