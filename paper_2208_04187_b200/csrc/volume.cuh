// 3-D activation maps (the paper's appendix "Compression of 1D and 3D Activation Maps": Minibatch x Channel x
// N x N x N, average pooling and nearest up-sampling over B x B x B blocks; Eq. 9 and its inverse unchanged).
// General kernels for any shape, any block size and any Q in {1,2,4,8}, in the manner of the 2-D two-pass path:
//   lfc_stats3d_kernel   one thread per block: mean in the fixed order (balanced pairwise tree along the depth
//                        axis, then down the rows, then across the columns), stored low-frequency value,
//                        residual extremes -> per-sample min / max keys in the scratch slots
//   quant_pack3d_kernel  one thread per packed 32-bit word
//   decompress3d_kernel  one thread per packed 32-bit word
// x is read twice by compress (the second time from L2 when the tensor fits).
#pragma once

#include "common.cuh"
#include "twopass.cuh"   // tree_sum

namespace divk {

struct Shape3 {
    uint32_t N, C, D, H, W, B, Db, Hb, Wb, P2;
    uint32_t HW, DHW, CDHW;     // per plane, per volume, per sample (< 2^32)
    uint32_t TPV;               // blocks per volume = Db * Hb * Wb
    uint64_t total;             // N * CDHW
    uint64_t tiles;             // N * C * TPV
};

template <typename XT, typename LT>
__global__ void __launch_bounds__(128)
lfc_stats3d_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, Shape3 s) {
    const uint64_t gt = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gt >= s.tiles) return;
    const uint64_t vol = gt / s.TPV;                       // n * C + c
    uint32_t idx = (uint32_t)(gt - vol * s.TPV);
    const uint32_t bd = idx / (s.Hb * s.Wb);
    idx -= bd * s.Hb * s.Wb;
    const uint32_t bh = idx / s.Wb, bw = idx - bh * s.Wb;
    const uint32_t n = (uint32_t)(vol / s.C);
    const uint32_t d0 = bd * s.B, h0 = bh * s.B, w0 = bw * s.B;
    const uint32_t nd = min(s.B, s.D - d0), nh = min(s.B, s.H - h0), nw = min(s.B, s.W - w0);
    const XT* base = x + vol * s.DHW + ((size_t)d0 * s.H + h0) * s.W + w0;
    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
    const float total = tree_sum(s.P2, [&](uint32_t c) -> float {
        if (c >= nw) return 0.f;
        return tree_sum(s.P2, [&](uint32_t r) -> float {
            if (r >= nh) return 0.f;
            return tree_sum(s.P2, [&](uint32_t k) -> float {
                if (k >= nd) return 0.f;
                const float v = Elem<XT>::load(base + ((size_t)k * s.H + r) * s.W + c);
                lo = fminf(lo, v);
                hi = fmaxf(hi, v);
                return v;
            });
        });
    });
    const float mean = __fdiv_rn(total, (float)(nd * nh * nw));
    Elem<LT>::store(lfc + gt, mean);
    const float stored = Elem<LT>::round(mean);
    // x -> fl(x - stored) is monotone, so the residual extremes are those of the extreme x
    uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
    atomicMax(slot + 0, ~float_key(__fsub_rn(lo, stored)));
    atomicMax(slot + 1, float_key(__fsub_rn(hi, stored)));
}

// position of a flat in-sample index
struct Pos3 {
    uint32_t vol, d, h, w;
};
__device__ __forceinline__ Pos3 pos3(const Shape3& s, uint32_t e) {
    Pos3 p;
    p.vol = e / s.DHW;
    uint32_t rem = e - p.vol * s.DHW;
    p.d = rem / s.HW;
    rem -= p.d * s.HW;
    p.h = rem / s.W;
    p.w = rem - p.h * s.W;
    return p;
}
__device__ __forceinline__ void advance3(const Shape3& s, uint32_t& n, uint32_t& e, Pos3& p) {
    ++e;
    if (++p.w == s.W) {
        p.w = 0;
        if (++p.h == s.H) {
            p.h = 0;
            if (++p.d == s.D) {
                p.d = 0;
                if (++p.vol == s.C) {
                    p.vol = 0;
                    e = 0;
                    ++n;
                }
            }
        }
    }
}
__device__ __forceinline__ size_t lfc_index3(const Shape3& s, uint32_t n, const Pos3& p) {
    return (((size_t)n * s.C + p.vol) * s.Db + p.d / s.B) * s.Hb * s.Wb + (p.h / s.B) * s.Wb + p.w / s.B;
}

template <typename XT, typename LT, int Q>
__global__ void __launch_bounds__(256)
quant_pack3d_kernel(const XT* __restrict__ x, const LT* __restrict__ lfc, const uint32_t* __restrict__ ws,
                    uint32_t* __restrict__ packed, float* __restrict__ stats, Shape3 s, uint64_t seed, uint64_t nwords) {
    constexpr uint32_t PER = 32 / Q;
    constexpr float qmax = (float)((1 << Q) - 1);
    const uint64_t word = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= nwords) return;
    uint64_t i = word * PER;
    uint32_t n = (uint32_t)(i / s.CDHW);
    uint32_t e = (uint32_t)(i - (uint64_t)n * s.CDHW);
    Pos3 p = pos3(s, e);
    uint32_t cur_n = 0xFFFFFFFFu, cur_g = 0xFFFFFFFFu;
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
        if ((e >> 2) != cur_g) {
            cur_g = e >> 2;
            z = rng_group(base, cur_g);
        }
        const float r = __fsub_rn(Elem<XT>::load(x + i), Elem<LT>::load(lfc + lfc_index3(s, n, p)));
        const uint32_t field = (uint32_t)(z >> (16 * (e & 3))) & 0xFFFFu;
        acc |= (quant_bits(r, qp.delta, qp.scale, qmax, field) - MAGIC_CEIL_BITS) << (j * Q);
        advance3(s, n, e, p);
    }
    packed[word] = acc;
}

template <typename XT, typename LT, int Q>
__global__ void __launch_bounds__(256)
decompress3d_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed, const float* __restrict__ stats,
                    XT* __restrict__ xhat, Shape3 s, uint64_t nwords) {
    constexpr uint32_t PER = 32 / Q;
    constexpr uint32_t MASK = (1u << Q) - 1u;
    const uint64_t word = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= nwords) return;
    uint64_t i = word * PER;
    uint32_t n = (uint32_t)(i / s.CDHW);
    uint32_t e = (uint32_t)(i - (uint64_t)n * s.CDHW);
    Pos3 p = pos3(s, e);
    const uint32_t bits = packed[word];
    uint32_t cur_n = 0xFFFFFFFFu;
    float delta = 0.f, step = 0.f;
    for (uint32_t j = 0; j < PER && i < s.total; ++j, ++i) {
        if (n != cur_n) {
            delta = stats[2 * (size_t)n];
            step = stats[2 * (size_t)n + 1];
            cur_n = n;
        }
        Elem<XT>::store(xhat + i, reconstruct((bits >> (j * Q)) & MASK, step, delta, Elem<LT>::load(lfc + lfc_index3(s, n, p))));
        advance3(s, n, e, p);
    }
}

}  // namespace divk
