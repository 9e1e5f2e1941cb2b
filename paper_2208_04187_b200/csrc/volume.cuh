// 3-D activation maps (the paper's appendix "Compression of 1D and 3D Activation Maps": Minibatch x Channel x
// N x N x N, average pooling and nearest up-sampling over B x B x B blocks; Eq. 9 and its inverse unchanged).
// General kernels for any shape, any block size and any Q in {1,2,4,8}, in the manner of the 2-D two-pass path:
//   lfc_stats3d_kernel   one thread per block: mean in the fixed order (balanced pairwise tree along the depth
//                        axis, then down the rows, then across the columns), stored low-frequency value,
//                        residual extremes -> per-sample min / max keys in the scratch slots
//   lfc_stats3d_warp_kernel  the same with a lane per block column (blocks of padded side <= 32): coalesced loads
//   lfc_stats3d_strip_kernel, quant3d_strip_kernel, decompress3d_strip_kernel
//                        W % 4 == 0 and B = 4 or 8: a lane per strip of 4 adjacent columns of one block (16-byte
//                        accesses), the default for such shapes
//   quant_pack3d_kernel  one thread per packed 32-bit word
//   decompress3d_kernel  one thread per packed 32-bit word
// x is read twice by compress (the second time from L2 when the tensor fits).
#pragma once

#include "decompress.cuh"   // DeqTable, quad_bits, Quad
#include "fused_v.cuh"     // packed arithmetic, quant_row
#include "twopass.cuh"     // tree_sum

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

// The same for blocks whose padded side fits a warp (P2 <= 32): a lane owns one column of one block, the P2 lanes
// of a block sit side by side and a warp takes 32 / P2 blocks that are neighbours along w, so every load
// instruction of a warp reads one contiguous row segment.  A lane sums its column along the depth and down the
// rows (the same trees), the columns of a block meet through xor shuffles.  One warp per group of 32 / P2 blocks.
template <typename XT, typename LT, int P2>
__global__ void __launch_bounds__(256)
lfc_stats3d_warp_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, Shape3 s,
                        uint32_t groups_per_row, uint64_t groups) {
    constexpr uint32_t BPW = 32 / P2;                         // blocks per warp
    const uint64_t grp = (uint64_t)blockIdx.x * 8u + (threadIdx.x >> 5);
    if (grp >= groups) return;                                // whole warps leave together
    const uint32_t lane = threadIdx.x & 31;
    // group -> (volume, bd, bh, first bw)
    const uint64_t rowid = grp / groups_per_row;              // (vol * Db + bd) * Hb + bh
    const uint32_t bw = (uint32_t)(grp - rowid * groups_per_row) * BPW + lane / P2;
    const uint32_t cw = lane % P2;
    const uint64_t vd = rowid / s.Hb;
    const uint32_t bh = (uint32_t)(rowid - vd * s.Hb);
    const uint64_t vol = vd / s.Db;
    const uint32_t bd = (uint32_t)(vd - vol * s.Db);
    const uint32_t n = (uint32_t)(vol / s.C);
    const uint32_t d0 = bd * s.B, h0 = bh * s.B, w0 = bw * s.B;
    const uint32_t nd = min(s.B, s.D - d0), nh = min(s.B, s.H - h0);
    const uint32_t nw = bw < s.Wb ? min(s.B, s.W - w0) : 0u;
    const bool ok = cw < nw;
    const XT* base = x + vol * s.DHW + ((size_t)d0 * s.H + h0) * s.W + (ok ? w0 + cw : 0u);
    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
    float sum = tree_sum((uint32_t)P2, [&](uint32_t r) -> float {
        if (!ok || r >= nh) return 0.f;
        return tree_sum((uint32_t)P2, [&](uint32_t k) -> float {
            if (k >= nd) return 0.f;
            const float v = Elem<XT>::load(base + ((size_t)k * s.H + r) * s.W);
            lo = fminf(lo, v);
            hi = fmaxf(hi, v);
            return v;
        });
    });
#pragma unroll
    for (int m = 1; m < P2; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
    uint32_t kmin = 0u, kmax = 0u;                            // neutral keys
    if (bw < s.Wb) {
        const float mean = __fdiv_rn(sum, (float)(nd * nh * nw));
        const float stored = Elem<LT>::round(mean);
        if (cw == 0) Elem<LT>::store(lfc + ((vol * s.Db + bd) * s.Hb + bh) * s.Wb + bw, mean);
        if (ok) {
            kmin = ~float_key(__fsub_rn(lo, stored));         // x -> fl(x - stored) is monotone
            kmax = float_key(__fsub_rn(hi, stored));
        }
    }
    kmin = __reduce_max_sync(0xFFFFFFFFu, kmin);
    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
    if (lane == 0) {
        uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
        atomicMax(slot + 0, kmin);
        atomicMax(slot + 1, kmax);
    }
}

// The same for W % 4 == 0 and B = 4 or 8 (the shapes of video and volumetric networks): a lane owns a strip of 4
// adjacent columns of one block over all its rows and depths (16-byte loads, packed adds), B / 4 lanes per block
// side by side.  Per row of the block the lane sums its B depth values with the tree, then the B row sums with the
// same tree, then its 4 columns and, for B = 8, meets the block's other strip by one xor shuffle: the order of
// lfc_stats3d_kernel.  For more loads in flight the rows of a strip are split between two neighbouring lanes (upper
// and lower half); their partial sums meet at the top level of the row tree.  Slots are numbered
// ((vol * Db + bd) * Hb + bh) * (Wb * B / 4 * 2) + 2 * strip in the block row + half; a warp takes 32 consecutive
// slots (it may straddle block rows, volumes and samples).
template <typename XT, typename LT, int P2>
__global__ void __launch_bounds__(128)
lfc_stats3d_strip_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, Shape3 s, uint64_t slots) {
    constexpr uint32_t LPB = P2 / 4;                                   // lanes per block
    const uint32_t lane = threadIdx.x & 31;
    constexpr uint32_t HR = P2 / 2;                                    // rows per lane
    const uint64_t slot = (uint64_t)blockIdx.x * 128u + threadIdx.x;          // 4 warps of 32 consecutive slots
    const uint32_t spr = s.Wb * LPB * 2u;                              // slots per row of blocks
    const bool live = slot < slots;
    const uint64_t rowid = (live ? slot : 0ull) / spr;                 // (vol * Db + bd) * Hb + bh
    const uint32_t sq = (uint32_t)((live ? slot : 0ull) - rowid * spr);
    const uint32_t half = sq & 1u, strip = sq >> 1;
    const uint32_t bw = strip / LPB, cw = (strip % LPB) * 4u;
    const uint64_t vd = rowid / s.Hb;
    const uint32_t bh = (uint32_t)(rowid - vd * s.Hb);
    const uint64_t vol = vd / s.Db;
    const uint32_t bd = (uint32_t)(vd - vol * s.Db);
    const uint32_t n = (uint32_t)(vol / s.C);
    const uint32_t d0 = bd * s.B, h0 = bh * s.B, w0 = bw * s.B;
    const uint32_t nd = min(s.B, s.D - d0), nh = min(s.B, s.H - h0), nw = min(s.B, s.W - w0);
    const bool ok = live && cw < nw;                                   // W % 4 == 0: a strip is whole or absent
    const uint32_t r0 = half * HR;                                     // first own row inside the block
    const XT* base = x + vol * s.DHW + ((size_t)d0 * s.H + h0 + r0) * s.W + (ok ? w0 + cw : 0u);
    const bool full = __all_sync(0xFFFFFFFFu, !ok || (nd == (uint32_t)P2 && nh == (uint32_t)P2));
    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
    uint64_t txy[4], tzw[4];                                           // partial sums over the rows, one per tree level
#pragma unroll
    for (int r = 0; r < (int)HR; ++r) {
        uint64_t vxy[P2], vzw[P2];
        // all loads of the row first (they are independent), then the extremes
        const XT* row = base + (size_t)r * s.W;
        const size_t plane = (size_t)s.HW;
        if (full) {
            if (ok) {
#pragma unroll
                for (int k = 0; k < P2; ++k) StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(row + k * plane), vxy[k], vzw[k]);
            } else {
#pragma unroll
                for (int k = 0; k < P2; ++k) {
                    vxy[k] = 0ull;
                    vzw[k] = 0ull;
                }
            }
        } else {
#pragma unroll
            for (int k = 0; k < P2; ++k) {
                vxy[k] = 0ull;
                vzw[k] = 0ull;
                if (ok && r0 + (uint32_t)r < nh && (uint32_t)k < nd)
                    StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(row + k * plane), vxy[k], vzw[k]);
            }
        }
#pragma unroll
        for (int k = 0; k < P2; ++k) {
            if (ok && (full || (r0 + (uint32_t)r < nh && (uint32_t)k < nd))) {
                float a, b, c, d;
                upk2(vxy[k], a, b);
                upk2(vzw[k], c, d);
                lo = fmin3(lo, a, b);
                lo = fmin3(lo, c, d);
                hi = fmax3(hi, a, b);
                hi = fmax3(hi, c, d);
            }
        }
#pragma unroll
        for (int w = P2; w > 1; w >>= 1) {
#pragma unroll
            for (int i = 0; i < w / 2; ++i) {
                vxy[i] = add2_rn(vxy[2 * i], vxy[2 * i + 1]);
                vzw[i] = add2_rn(vzw[2 * i], vzw[2 * i + 1]);
            }
        }
        // the tree over the rows, neighbours first, kept as one partial sum per level (r is a compile-time
        // constant here): rows 0+1, 2+3, ... are added as soon as both are there
        uint64_t cxy = vxy[0], czw = vzw[0];
        int lv = 0;
#pragma unroll
        for (int bit = 1; bit < (int)HR; bit <<= 1) {
            if (r & bit) {
                cxy = add2_rn(txy[lv], cxy);
                czw = add2_rn(tzw[lv], czw);
                ++lv;
            } else {
                break;
            }
        }
        txy[lv] = cxy;
        tzw[lv] = czw;
    }
    constexpr int TOP = P2 == 8 ? 2 : 1;                                // log2(HR): where the sum over the own rows ends up
    // top level of the row tree: upper half + lower half (the neighbouring lane)
    const uint64_t sxy = add2_rn(txy[TOP], __shfl_xor_sync(0xFFFFFFFFu, txy[TOP], 1));
    const uint64_t szw = add2_rn(tzw[TOP], __shfl_xor_sync(0xFFFFFFFFu, tzw[TOP], 1));
    float c0, c1, c2, c3;
    upk2(sxy, c0, c1);
    upk2(szw, c2, c3);
    float sum = __fadd_rn(__fadd_rn(c0, c1), __fadd_rn(c2, c3));
    if (LPB == 2u) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, 2));      // an absent strip brings 0
    uint32_t kmin = 0u, kmax = 0u;                                      // neutral keys
    if (ok) {
        const float mean = __fdiv_rn(sum, (float)(nd * nh * nw));
        const float stored = Elem<LT>::round(mean);
        if (cw == 0 && half == 0) Elem<LT>::store(lfc + ((vol * s.Db + bd) * s.Hb + bh) * s.Wb + bw, mean);
        kmin = ~float_key(__fsub_rn(lo, stored));                       // x -> fl(x - stored) is monotone
        kmax = float_key(__fsub_rn(hi, stored));
    }
    // one pair of atomics per warp where the whole warp sits in one sample, else one per lane
    const uint32_t n0 = __shfl_sync(0xFFFFFFFFu, n, 0);
    if (__all_sync(0xFFFFFFFFu, !ok || n == n0)) {
        kmin = __reduce_max_sync(0xFFFFFFFFu, kmin);
        kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
        if (lane == 0 && (kmin | kmax)) {
            uint32_t* slot_n = ws + WS_HEADER_WORDS + (size_t)n0 * WS_SLOT_WORDS;
            atomicMax(slot_n + 0, kmin);
            atomicMax(slot_n + 1, kmax);
        }
    } else if (ok) {
        uint32_t* slot_n = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
        atomicMax(slot_n + 0, kmin);
        atomicMax(slot_n + 1, kmax);
    }
}

// Quantise half with the same lane-per-strip layout (W % 4 == 0, B = 4 or 8): the lane reads its sample's extremes
// and its block's stored low-frequency value once, then walks the rows and depths of its strip: per row of 4 elements
// one 16-byte load, the random word of that group of 4 (the counter advances by a constant per row and per plane),
// Eq. 9 on packed pairs, one byte / half-word / word of codes.  x is read a second time.
template <typename XT, typename LT, int Q, int P2>
__global__ void __launch_bounds__(128)
quant3d_strip_kernel(const XT* __restrict__ x, const LT* __restrict__ lfc, const uint32_t* __restrict__ ws,
                     void* __restrict__ packed_v, float* __restrict__ stats, Shape3 s, uint64_t seed, uint64_t slots) {
    typedef typename PackedUnit<Q>::type OutT;
    constexpr uint32_t LPB = P2 / 4;
    // slots are taken from the end of the tensor backwards: what the statistics kernel read last is still in the L2
    const uint64_t back = (uint64_t)blockIdx.x * 128u + threadIdx.x;
    if (back >= slots) return;
    const uint64_t slot = slots - 1u - back;
    const uint32_t spr = s.Wb * LPB * 2u;                              // two lanes per strip: upper and lower rows
    const uint64_t rowid = slot / spr;
    const uint32_t sq = (uint32_t)(slot - rowid * spr);
    const uint32_t half = sq & 1u, strip = sq >> 1;
    const uint32_t bw = strip / LPB, cw = (strip % LPB) * 4u;
    const uint64_t vd = rowid / s.Hb;
    const uint32_t bh = (uint32_t)(rowid - vd * s.Hb);
    const uint64_t vol = vd / s.Db;
    const uint32_t bd = (uint32_t)(vd - vol * s.Db);
    const uint32_t n = (uint32_t)(vol / s.C);
    const uint32_t c = (uint32_t)(vol - (uint64_t)n * s.C);
    const uint32_t d0 = bd * s.B, h0 = bh * s.B, w0 = bw * s.B;
    const uint32_t nd = min(s.B, s.D - d0), nh = min(s.B, s.H - h0), nw = min(s.B, s.W - w0);
    const uint32_t* slot_n = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
    const QParams qp = make_qparams(key_float(~__ldg(slot_n + 0)), key_float(__ldg(slot_n + 1)), Q);
    if (c == 0 && rowid == vol * s.Db * s.Hb && sq == 0) {             // the first slot of the sample
        stats[2 * (size_t)n + 0] = qp.delta;
        stats[2 * (size_t)n + 1] = qp.step;
    }
    if (cw >= nw) return;                                              // W % 4 == 0: a strip is whole or absent
    const float stored = Elem<LT>::load(lfc + ((vol * s.Db + bd) * s.Hb + bh) * s.Wb + bw);
    const uint64_t stored2 = pk2(stored, stored), delta2 = pk2(qp.delta, qp.delta), scale2 = pk2(qp.scale, qp.scale);
    const uint32_t e0 = c * s.DHW + (d0 * s.H + h0) * s.W + w0 + cw;   // in-sample index of the strip's first element
    const XT* base = x + (size_t)n * s.CDHW + e0;
    OutT* out = reinterpret_cast<OutT*>(packed_v) + (((uint64_t)n * s.CDHW + e0) >> 2);
    const uint32_t W4 = s.W >> 2, HW4 = s.HW >> 2;
    const uint64_t ctr0 = rng_sample_base(seed, n) + K_GROUP * (uint64_t)((e0 >> 2) + 1u);
    const uint64_t row_step = K_GROUP * (uint64_t)W4, plane_step = K_GROUP * (uint64_t)HW4;
    const bool full = nd == (uint32_t)P2;
    const uint32_t r_end = min(nh, (half + 1u) * (P2 / 2u));
    for (uint32_t r = half * (P2 / 2u); r < r_end; ++r) {
        const XT* row = base + (size_t)r * s.W;
        uint64_t vxy[P2], vzw[P2];
#pragma unroll
        for (int k = 0; k < P2; ++k) {
            vxy[k] = 0ull;
            vzw[k] = 0ull;
            if (full || (uint32_t)k < nd) StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(row + (size_t)k * s.HW), vxy[k], vzw[k]);
        }
        uint64_t ctr = ctr0 + row_step * r;
        OutT* o = out + (size_t)r * W4;
#pragma unroll
        for (int k = 0; k < P2; ++k) {
            if (full || (uint32_t)k < nd) *o = (OutT)quant_row<Q>(vxy[k], vzw[k], stored2, delta2, scale2, rng_mix(ctr));
            ctr += plane_step;
            o += HW4;
        }
    }
}

// Decompress with the lane-per-strip layout (W % 4 == 0, B = 4 or 8, Q in {2,4,8}): the lane reads its block's
// low-frequency value once, then per row of 4 elements one byte / half-word / word of codes, one look-up in the
// sample's dequantisation table and one 16-byte (fp32) store.  Two lanes per strip (upper and lower rows).
// grid = (ceil(slots per sample / 256), N)
template <typename XT, typename LT, int Q, int P2>
__global__ void __launch_bounds__(256)
decompress3d_strip_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed, const float* __restrict__ stats,
                          XT* __restrict__ xhat, Shape3 s, uint32_t slots_per_sample) {
    constexpr uint32_t LPB = P2 / 4;
    __shared__ DeqTable<Q> table;
    const uint32_t n = blockIdx.y;
    table.build(__ldg(stats + 2 * (size_t)n + 1), __ldg(stats + 2 * (size_t)n));
    __syncthreads();
    const uint32_t slot = blockIdx.x * 256u + threadIdx.x;
    if (slot >= slots_per_sample) return;
    const uint32_t spr = s.Wb * LPB * 2u;
    const uint32_t rowid = slot / spr;                                 // (c * Db + bd) * Hb + bh
    const uint32_t sq = slot - rowid * spr;
    const uint32_t half = sq & 1u, strip = sq >> 1;
    const uint32_t bw = strip / LPB, cw = (strip % LPB) * 4u;
    const uint32_t vd = rowid / s.Hb, bh = rowid - vd * s.Hb;
    const uint32_t c = vd / s.Db, bd = vd - c * s.Db;
    const uint32_t d0 = bd * s.B, h0 = bh * s.B, w0 = bw * s.B;
    const uint32_t nd = min(s.B, s.D - d0), nh = min(s.B, s.H - h0), nw = min(s.B, s.W - w0);
    if (cw >= nw) return;
    const float lf = Elem<LT>::load(lfc + (size_t)n * s.C * s.TPV + (size_t)rowid * s.Wb + bw);
    const uint32_t e0 = c * s.DHW + (d0 * s.H + h0) * s.W + w0 + cw;   // in-sample index of the strip's first element
    const uint64_t quad0 = ((uint64_t)n * s.CDHW + e0) >> 2;
    XT* out = xhat + (size_t)n * s.CDHW + e0;
    const uint32_t W4 = s.W >> 2, HW4 = s.HW >> 2;
    const bool full = nd == (uint32_t)P2;
    const uint32_t r_end = min(nh, (half + 1u) * (P2 / 2u));
    for (uint32_t r = half * (P2 / 2u); r < r_end; ++r) {
        uint32_t bits[P2];
#pragma unroll
        for (int k = 0; k < P2; ++k) {
            bits[k] = 0u;
            if (full || (uint32_t)k < nd) bits[k] = quad_bits<Q>(packed, quad0 + (uint64_t)r * W4 + (uint64_t)k * HW4);
        }
#pragma unroll
        for (int k = 0; k < P2; ++k) {
            if (full || (uint32_t)k < nd) {
                const float4 hq = table.quad(bits[k]);
                Quad<XT>::store(out + (size_t)r * s.W + (size_t)k * s.HW, __fadd_rn(lf, hq.x), __fadd_rn(lf, hq.y), __fadd_rn(lf, hq.z),
                                __fadd_rn(lf, hq.w));
            }
        }
    }
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

// ------------------------------------------------------------------------------------------------
// W % 4 == 0 and B % 4 == 0: 4 consecutive elements share a block.  One thread per QPT quads, 256 quads apart.
// grid = (ceil(quads_per_sample / (256*QPT)), N)
// ------------------------------------------------------------------------------------------------
struct Quad3 {
    uint32_t qps;                 // quads per sample
    uint32_t C, Db, Hb, Wb, B;
    uint32_t qpr, qpp, qpv;       // quads per row, per plane (H rows), per volume (D planes)
    FastDiv by_qpv, by_qpp, by_qpr, by_b;
};
// low-frequency value of quad q (inside sample n's map lfc_n)
template <typename LT>
__device__ __forceinline__ float quad3_lfc(const LT* __restrict__ lfc_n, const Quad3& g, uint32_t q) {
    const uint32_t vol = fdiv(q, g.by_qpv);
    uint32_t rem = q - vol * g.qpv;
    const uint32_t d = fdiv(rem, g.by_qpp);
    rem -= d * g.qpp;
    const uint32_t h = fdiv(rem, g.by_qpr);
    const uint32_t w = (rem - h * g.qpr) * 4u;
    return Elem<LT>::load(lfc_n + (((size_t)vol * g.Db + fdiv(d, g.by_b)) * g.Hb + fdiv(h, g.by_b)) * g.Wb + fdiv(w, g.by_b));
}

template <typename XT, typename LT, int Q, int QPT>
__global__ void __launch_bounds__(256)
quant3d_quad_kernel(const XT* __restrict__ x, const LT* __restrict__ lfc, const uint32_t* __restrict__ ws,
                    void* __restrict__ packed_v, float* __restrict__ stats, Quad3 g, uint64_t seed) {
    typedef typename PackedUnit<Q>::type OutT;
    const uint32_t n = blockIdx.y;
    const uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
    const QParams qp = make_qparams(key_float(~__ldg(slot + 0)), key_float(__ldg(slot + 1)), Q);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        stats[2 * (size_t)n + 0] = qp.delta;
        stats[2 * (size_t)n + 1] = qp.step;
    }
    const uint64_t delta2 = pk2(qp.delta, qp.delta), scale2 = pk2(qp.scale, qp.scale);
    const uint64_t base = rng_sample_base(seed, n);
    const XT* x_n = x + (size_t)n * g.qps * 4u;
    const LT* lfc_n = lfc + (size_t)n * g.C * g.Db * g.Hb * g.Wb;
    OutT* packed = reinterpret_cast<OutT*>(packed_v) + (uint64_t)n * g.qps;
    const uint32_t q0 = blockIdx.x * (256u * QPT) + threadIdx.x;
    uint64_t xy[QPT], zw[QPT];
    float lf[QPT];
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < g.qps) {
            StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(x_n + (size_t)q * 4u), xy[k], zw[k]);
            lf[k] = quad3_lfc(lfc_n, g, q);
        }
    }
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < g.qps)
            packed[q] = (OutT)quant_row<Q>(xy[k], zw[k], pk2(lf[k], lf[k]), delta2, scale2, rng_group(base, q));
    }
}

template <typename XT, typename LT, int Q, int QPT>
__global__ void __launch_bounds__(256)
decompress3d_quad_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                         const float* __restrict__ stats, XT* __restrict__ xhat, Quad3 g) {
    __shared__ DeqTable<Q> table;
    const uint32_t n = blockIdx.y;
    table.build(__ldg(stats + 2 * (size_t)n + 1), __ldg(stats + 2 * (size_t)n));
    __syncthreads();
    const uint64_t sample_quad0 = (uint64_t)n * g.qps;
    const LT* lfc_n = lfc + (size_t)n * g.C * g.Db * g.Hb * g.Wb;
    const uint32_t q0 = blockIdx.x * (256u * QPT) + threadIdx.x;
    uint32_t bits[QPT];
    float lf[QPT];
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < g.qps) {
            bits[k] = quad_bits<Q>(packed, sample_quad0 + q);
            lf[k] = quad3_lfc(lfc_n, g, q);
        }
    }
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < g.qps) {
            const float4 hq = table.quad(bits[k]);
            Quad<XT>::store(xhat + (sample_quad0 + q) * 4u, __fadd_rn(lf[k], hq.x), __fadd_rn(lf[k], hq.y),
                            __fadd_rn(lf[k], hq.z), __fadd_rn(lf[k], hq.w));
        }
    }
}

}  // namespace divk
