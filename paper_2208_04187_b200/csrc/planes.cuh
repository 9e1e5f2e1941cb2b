// Compress kernels for maps with small planes whose width is not a multiple of 4 (the 14 x 14 and
// 7 x 7 maps of the ImageNet networks): DIVISION Sec. 4.1; Algorithm 1, forward loop.
//
// Two launches, no dependency inside a kernel:
//   plane_stats_kernel   block means in the fixed summation order, stored low-frequency values,
//                        residual extremes -> per-sample min / max keys in the scratch slots;
//   plane_quant_kernel   Eq. 9 with stochastic rounding and packing, 4 consecutive elements per step.
// The second kernel reads x again; these maps are a few tens of MB, so the second read comes from the
// 126 MB L2 (larger tensors are still handled correctly, at the price of reading x twice from HBM).
//
// plane_stats_kernel: a lane owns one tile column of one plane (P2 lanes per tile, tiles_per_row * P2
// lanes per plane, several planes per warp): per band it loads its column's rows, sums them with the
// balanced tree, meets the other columns of the tile with xor shuffles (the same tree across columns),
// and keeps the extremes of its column.
// plane_quant_kernel: one thread per 4 consecutive elements of the flat sample (they may lie in
// different tiles, rows or planes): the tile of every position of a plane comes from a table in shared
// memory, the arithmetic of Eq. 9 runs on packed pairs.
#pragma once

#include "decompress.cuh"   // flat_table_words, flat_planes_per_cta, flat_smem_bytes
#include "fused_v.cuh"

namespace divk {

struct PlaneGeom {
    uint32_t C, H, W, B, Hb, Wb, HW, CHW, TPP;
    uint32_t lanes_per_plane;     // Wb * P2
    uint32_t planes_per_warp;     // 32 / lanes_per_plane
    uint32_t groups;              // ceil(C / planes_per_warp): warp passes per sample
    uint32_t qps;                 // quads per sample = CHW / 4
    uint32_t table_words;         // 32-bit words the tile table takes in shared memory
    uint32_t planes_per_cta;      // upper bound of the planes one CTA of the quantise kernel touches
    FastDiv by_hw, by_w, by_b;
};

template <typename XT, typename LT, int P2>
__global__ void __launch_bounds__(256)
plane_stats_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, PlaneGeom g) {
    const uint32_t n = blockIdx.y;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t pl_local = lane / g.lanes_per_plane;
    const uint32_t lw = lane - pl_local * g.lanes_per_plane;
    const uint32_t bw = lw / P2, cw = lw % P2;
    const uint32_t cols = (bw < g.Wb) ? min(g.B, g.W - bw * g.B) : 0u;
    const bool lane_ok = pl_local < g.planes_per_warp && cw < cols;
    const uint32_t col = bw * g.B + cw;
    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
    for (uint32_t pg = blockIdx.x * 8u + warp; pg < g.groups; pg += gridDim.x * 8u) {
        const uint32_t plane = pg * g.planes_per_warp + pl_local;
        const bool ok = lane_ok && plane < g.C;
        const XT* xp = x + ((size_t)n * g.C + (ok ? plane : 0u)) * g.HW + (ok ? col : 0u);
        LT* lp = lfc + ((size_t)n * g.C + (ok ? plane : 0u)) * g.TPP + (ok ? bw : 0u);
        for (uint32_t bh = 0; bh < g.Hb; ++bh) {
            const uint32_t rows = min(g.B, g.H - bh * g.B);
            float v[P2];
#pragma unroll
            for (int r = 0; r < P2; ++r) v[r] = (ok && (uint32_t)r < rows) ? Elem<XT>::load(xp + (size_t)(bh * g.B + r) * g.W) : 0.f;
            float sum = tree8<P2>(v);
#pragma unroll
            for (int m = 1; m < P2; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
            // one lane per tile divides, the others take its result
            float mean = 0.f;
            if (cw == 0) mean = __fdiv_rn(sum, (float)(rows * max(cols, 1u)));
            mean = __shfl_sync(0xFFFFFFFFu, mean, (int)(lane - cw));
            const float stored = Elem<LT>::round(mean);
            if (ok) {
                if (cw == 0) Elem<LT>::store(lp + (size_t)bh * g.Wb, mean);
                float blo = 3.402823466e+38f, bhi = -3.402823466e+38f;
#pragma unroll
                for (int r = 0; r < P2; ++r) {
                    if ((uint32_t)r < rows) {
                        blo = fminf(blo, v[r]);
                        bhi = fmaxf(bhi, v[r]);
                    }
                }
                // x -> fl(x - stored) is monotone: the residual extremes are those of the extreme x
                lo = fminf(lo, __fsub_rn(blo, stored));
                hi = fmaxf(hi, __fsub_rn(bhi, stored));
            }
        }
    }
    const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
    const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
    if (lane == 0 && blockIdx.x * 8u + warp < g.groups) {
        uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
        atomicMax(slot + 0, kmin);
        atomicMax(slot + 1, kmax);
    }
}

template <typename XT, typename LT, int Q, int QPT>
__global__ void __launch_bounds__(256)
plane_quant_kernel(const XT* __restrict__ x, const LT* __restrict__ lfc, const uint32_t* __restrict__ ws,
                   void* __restrict__ packed_v, float* __restrict__ stats, PlaneGeom g, uint64_t seed) {
    typedef typename PackedUnit<Q>::type OutT;
    extern __shared__ uint32_t plane_smem[];
    uint16_t* tile_of = reinterpret_cast<uint16_t*>(plane_smem);          // position inside a plane -> tile inside the plane
    float* lfc_s = reinterpret_cast<float*>(plane_smem + g.table_words);  // stored low-frequency values of this CTA's planes
    const uint32_t n = blockIdx.y;
    for (uint32_t idx = threadIdx.x; idx < g.HW; idx += 256u) {
        const uint32_t h = fdiv(idx, g.by_w), w = idx - h * g.W;
        tile_of[idx] = (uint16_t)(fdiv(h, g.by_b) * g.Wb + fdiv(w, g.by_b));
    }
    const uint32_t plane0 = fdiv(blockIdx.x * (1024u * QPT), g.by_hw);
    const uint32_t nplanes = min(g.planes_per_cta, g.C - plane0);
    {
        const LT* src = lfc + ((size_t)n * g.C + plane0) * g.TPP;
        for (uint32_t idx = threadIdx.x; idx < nplanes * g.TPP; idx += 256u) lfc_s[idx] = Elem<LT>::load(src + idx);
    }
    __syncthreads();
    const uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
    const QParams qp = make_qparams(key_float(~__ldg(slot + 0)), key_float(__ldg(slot + 1)), Q);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        stats[2 * (size_t)n + 0] = qp.delta;
        stats[2 * (size_t)n + 1] = qp.step;
    }
    const uint64_t delta2 = pk2(qp.delta, qp.delta), scale2 = pk2(qp.scale, qp.scale);
    const uint64_t base = rng_sample_base(seed, n);
    const uint64_t sample_quad0 = (uint64_t)n * g.qps;
    const XT* x_n = x + (size_t)n * g.CHW;
    OutT* packed = reinterpret_cast<OutT*>(packed_v);
    const uint32_t q0 = blockIdx.x * (256u * QPT) + threadIdx.x;
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < g.qps) {
            uint64_t xy, zw;
            StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(x_n + (size_t)q * 4u), xy, zw);
            const uint32_t plane = fdiv(q * 4u, g.by_hw);
            uint32_t rem = q * 4u - plane * g.HW;
            const float* lfc_p = lfc_s + (plane - plane0) * g.TPP;
            float lf[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                lf[i] = lfc_p[tile_of[rem]];
                if (++rem == g.HW) {
                    rem = 0;
                    lfc_p += g.TPP;
                }
            }
            constexpr float qmax = (float)((1 << Q) - 1);
            const uint64_t z = rng_group(base, q);
            uint32_t b0, b1, b2, b3;
            quant2(xy, pk2(lf[0], lf[1]), delta2, scale2, qmax, (uint32_t)z, b0, b1);
            quant2(zw, pk2(lf[2], lf[3]), delta2, scale2, qmax, (uint32_t)(z >> 32), b2, b3);
            constexpr uint32_t BIAS = QUANT2_BITS * (1u + (1u << Q) + (1u << (2 * Q)) + (1u << (3 * Q)));   // mod 2^32
            packed[sample_quad0 + q] = (OutT)(b0 + (b1 << Q) + (b2 << (2 * Q)) + (b3 << (3 * Q)) - BIAS);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
constexpr uint32_t PLANE_MAX_HW = 8192;
constexpr int PLANE_QPT = 4;

inline bool plan_planes(const div_desc* d, const Shape& s, PlaneGeom* out) {
    if (!(d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return false;
    if (!(s.P2 == 4 || s.P2 == 8 || s.P2 == 16)) return false;
    if (s.Wb * s.P2 > 32u) return false;
    if (s.CHW % 4 != 0 || s.CHW >= (1u << 31)) return false;
    if (s.HW > PLANE_MAX_HW || s.TPP > 65535u || s.N > 65535u) return false;
    PlaneGeom g;
    g.C = s.C; g.H = s.H; g.W = s.W; g.B = s.B; g.Hb = s.Hb; g.Wb = s.Wb; g.HW = s.HW; g.CHW = s.CHW; g.TPP = s.TPP;
    g.lanes_per_plane = s.Wb * s.P2;
    g.planes_per_warp = 32u / g.lanes_per_plane;
    g.groups = (s.C + g.planes_per_warp - 1) / g.planes_per_warp;
    g.qps = s.CHW / 4;
    g.table_words = flat_table_words(s.HW);
    g.planes_per_cta = flat_planes_per_cta(4u * 256u * PLANE_QPT, s.HW);
    if (flat_smem_bytes(4u * 256u * PLANE_QPT, s.HW, s.TPP) > 44000) return false;
    g.by_hw = host_fastdiv(s.HW);
    g.by_w = host_fastdiv(s.W);
    g.by_b = host_fastdiv(s.B);
    *out = g;
    return true;
}

template <typename XT, typename LT>
inline div_status compress_planes_t(const div_desc* d, const Shape& s, const div_layout& lo, const PlaneGeom& g,
                                    const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st) {
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return DIV_ERR_CUDA;
    // pass 1: enough CTAs per sample to fill the GPU a few times over, never more than there are warp passes
    uint32_t bx = (uint32_t)((8ull * di.sms + s.N - 1) / s.N);
    const uint32_t bx_max = (g.groups + 7u) / 8u;
    if (bx > bx_max) bx = bx_max;
    if (bx < 1) bx = 1;
    const dim3 grid1(bx, s.N);
    const XT* xt = (const XT*)x;
    LT* lfc = (LT*)(blob + lo.lfc_off);
    switch (s.P2) {
        case 4: plane_stats_kernel<XT, LT, 4><<<grid1, 256, 0, st>>>(xt, lfc, ws, g); break;
        case 8: plane_stats_kernel<XT, LT, 8><<<grid1, 256, 0, st>>>(xt, lfc, ws, g); break;
        case 16: plane_stats_kernel<XT, LT, 16><<<grid1, 256, 0, st>>>(xt, lfc, ws, g); break;
        default: return DIV_ERR_PARAM;
    }
    if (cudaGetLastError() != cudaSuccess) return DIV_ERR_CUDA;
    const uint32_t per_block = 256u * PLANE_QPT;
    const dim3 grid2((g.qps + per_block - 1) / per_block, s.N);
    const size_t smem = flat_smem_bytes(4u * per_block, s.HW, s.TPP);
    void* packed = blob + lo.packed_off;
    float* stats = (float*)(blob + lo.stats_off);
    switch (d->qbits) {
        case 2: plane_quant_kernel<XT, LT, 2, PLANE_QPT><<<grid2, 256, smem, st>>>(xt, lfc, ws, packed, stats, g, seed); break;
        case 4: plane_quant_kernel<XT, LT, 4, PLANE_QPT><<<grid2, 256, smem, st>>>(xt, lfc, ws, packed, stats, g, seed); break;
        case 8: plane_quant_kernel<XT, LT, 8, PLANE_QPT><<<grid2, 256, smem, st>>>(xt, lfc, ws, packed, stats, g, seed); break;
        default: return DIV_ERR_PARAM;
    }
    return cudaGetLastError() == cudaSuccess ? DIV_OK : DIV_ERR_CUDA;
}

inline div_status compress_planes(const div_desc* d, const Shape& s, const div_layout& lo, const PlaneGeom& g,
                                  const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st) {
    typedef __nv_bfloat16 bf16;
    if (d->x_dtype == DIV_F32) {
        if (d->lfc_dtype == DIV_F32) return compress_planes_t<float, float>(d, s, lo, g, x, blob, ws, seed, st);
        return compress_planes_t<float, bf16>(d, s, lo, g, x, blob, ws, seed, st);
    }
    if (d->lfc_dtype == DIV_F32) return compress_planes_t<bf16, float>(d, s, lo, g, x, blob, ws, seed, st);
    return compress_planes_t<bf16, bf16>(d, s, lo, g, x, blob, ws, seed, st);
}

}  // namespace divk
