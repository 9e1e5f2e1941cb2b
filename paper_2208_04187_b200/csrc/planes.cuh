// Compress kernels for maps of small planes of any width (the 14 x 14 and 7 x 7 maps of the ImageNet networks;
// also the first choice for planes up to 32 wide below 56 MiB): DIVISION Sec. 4.1; Algorithm 1, forward loop.
//
// plane_fused_kernel does both halves in one launch (see there); where its CTAs cannot all be resident the pair
// below runs instead.  Two launches, no dependency inside a kernel:
//   plane_stats_kernel   block means in the fixed summation order, stored low-frequency values,
//                        residual extremes -> per-sample min / max keys in the scratch slots;
//   plane_quant_kernel   Eq. 9 with stochastic rounding and packing, 4 consecutive elements per step.
// The second kernel reads x again; these maps are a few tens of MB, so the second read comes from the
// 126 MB L2 (larger tensors are still handled correctly, at the price of reading x twice from HBM).
//
// First half (plane_half1, used by plane_stats_kernel and plane_fused_kernel): a lane owns two adjacent columns
// of one tile of one plane (P2 / 2 lanes per tile, several planes per warp): per band it loads its columns' rows
// (one 8-byte load per row where W and B are even, else two loads), sums each column with the balanced tree,
// meets the other columns of the tile with xor shuffles (the same tree across columns), and keeps the extremes
// of its columns.
// Second half (plane_quant_kernel, plane_fused_kernel): one thread per 4 consecutive elements of the flat sample
// (they may lie in different tiles, rows or planes): where their 4 low-frequency values sit comes from the quad
// table in shared memory (one 8-byte entry per quad of a period of lcm(HW, 4) elements), the arithmetic of Eq. 9
// runs on packed pairs.
#pragma once

#include "decompress.cuh"   // quad table, flat_planes_per_cta, flat_smem_bytes
#include "fused_v.cuh"

namespace divk {

struct PlaneGeom {
    uint32_t C, H, W, B, Hb, Wb, HW, CHW, TPP;
    uint32_t cpl;                 // first half, how a lane reads its 2 adjacent columns: 2 = one 8-byte load (W and B even), 3 = two loads
    uint32_t lanes_per_plane;     // Wb * P2 / 2
    uint32_t planes_per_warp;     // 32 / lanes_per_plane
    uint32_t groups;              // ceil(C / planes_per_warp): warp passes per sample
    uint32_t qps;                 // quads per sample = CHW / 4
    uint32_t table_words;         // 32-bit words the quad table takes in shared memory
    uint32_t planes_per_cta;      // upper bound of the planes one CTA of the quantise kernel touches
    uint32_t period;              // quads after which the quad table repeats
    uint32_t period_planes;       // planes one period covers (1, 2 or 4)
    FastDiv by_hw, by_w, by_b, by_period;
};

// One or two adjacent columns of one row, widened to fp32 and packed as a pair (the second half is 0 for one column)
template <typename XT, int CPL> struct ColLoad;
template <> struct ColLoad<float, 1> {
    static __device__ __forceinline__ uint64_t load(const float* p) { return pk2(*p, 0.f); }
};
template <> struct ColLoad<float, 2> {
    static __device__ __forceinline__ uint64_t load(const float* p) { return *reinterpret_cast<const uint64_t*>(p); }
};
template <> struct ColLoad<__nv_bfloat16, 1> {
    static __device__ __forceinline__ uint64_t load(const __nv_bfloat16* p) {
        return pk2u((uint32_t)*reinterpret_cast<const uint16_t*>(p) << 16, 0u);
    }
};
template <> struct ColLoad<__nv_bfloat16, 2> {
    static __device__ __forceinline__ uint64_t load(const __nv_bfloat16* p) {
        const uint32_t u = *reinterpret_cast<const uint32_t*>(p);
        return pk2u(u << 16, u & 0xFFFF0000u);
    }
};

// the lane's columns of one row: CPL 1 one column, 2 two columns by one aligned load, 3 two columns by two loads
// (the second only where it exists)
template <typename XT, int CPL>
__device__ __forceinline__ uint64_t load_cols(const XT* p, bool second) {
    if (CPL == 3) {
        float a, b, z;
        upk2(ColLoad<XT, 1>::load(p), a, z);
        b = 0.f;
        if (second) upk2(ColLoad<XT, 1>::load(p + 1), b, z);
        return pk2(a, b);
    }
    return ColLoad<XT, CPL == 3 ? 1 : CPL>::load(p);
}

// First half for a run of planes: a lane owns two adjacent columns of one tile of one plane (P2 / 2 lanes per
// tile, several planes per warp; CPL says how they are loaded, see load_cols).  Per band it loads its columns' rows, sums each column with the balanced tree
// down the rows, meets the tile's other columns (its own second column first, then xor shuffles: the same tree
// across columns) and keeps the extremes of its columns.  Planes first, first + stride, ... < count of the run at
// x_run / lfc_run; `keep` (may be null) receives the stored low-frequency values, TPP per plane of the run.
// Returns the residual extremes of this lane's elements in lo / hi.
template <typename XT, typename LT, int P2, int CPL>
__device__ __forceinline__ void plane_half1(const XT* __restrict__ x_run, LT* __restrict__ lfc_run, float* keep, uint32_t first,
                                            uint32_t stride, uint32_t count, const PlaneGeom& g, uint32_t lane, float& lo,
                                            float& hi) {
    constexpr uint32_t NC = CPL == 1 ? 1u : 2u;                   // columns per lane (CPL 2: one 8-byte load, 3: two loads)
    constexpr uint32_t LPT = P2 / NC;                             // lanes per tile
    const uint32_t pl_local = lane / g.lanes_per_plane;
    const uint32_t lw = lane - pl_local * g.lanes_per_plane;
    const uint32_t bw = lw / LPT, cw = (lw % LPT) * NC;           // tile column, first own column inside the tile
    const uint32_t cols = (bw < g.Wb) ? min(g.B, g.W - bw * g.B) : 0u;
    const bool lane_ok = pl_local < g.planes_per_warp && cw < cols;     // W and B even where CPL = 2: both columns or none
    const bool second = cw + 1u < cols;                                  // CPL = 3: the second column may lie past the tile's edge
    const uint32_t col = bw * g.B + cw;
    for (uint32_t pp = first; pp < count; pp += stride) {
        const uint32_t pl = pp + pl_local;
        const bool ok = lane_ok && pl < count;
        const XT* xp = x_run + (size_t)(ok ? pl : 0u) * g.HW + (ok ? col : 0u);
        LT* lp = lfc_run + (size_t)(ok ? pl : 0u) * g.TPP + (ok ? bw : 0u);
        for (uint32_t bh = 0; bh < g.Hb; ++bh) {
            const uint32_t rows = min(g.B, g.H - bh * g.B);       // the same in every lane
            uint64_t v[P2];
            if (rows == (uint32_t)P2) {
#pragma unroll
                for (int r = 0; r < P2; ++r) v[r] = ok ? load_cols<XT, CPL>(xp + (size_t)(bh * g.B + r) * g.W, second) : 0ull;
            } else {
#pragma unroll
                for (int r = 0; r < P2; ++r)
                    v[r] = (ok && (uint32_t)r < rows) ? load_cols<XT, CPL>(xp + (size_t)(bh * g.B + r) * g.W, second) : 0ull;
            }
            uint64_t t[P2];
#pragma unroll
            for (int i = 0; i < P2; ++i) t[i] = v[i];
#pragma unroll
            for (int w = P2; w > 1; w >>= 1) {
#pragma unroll
                for (int i = 0; i < w / 2; ++i) t[i] = add2_rn(t[2 * i], t[2 * i + 1]);
            }
            float c0, c1;
            upk2(t[0], c0, c1);
            float sum = NC == 2 ? __fadd_rn(c0, c1) : c0;              // an absent second column brings the zero it stands for
#pragma unroll
            for (int m = 1; m < (int)LPT; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
            // after the butterfly every lane of a tile holds the same sum: each divides for itself
            const float mean = __fdiv_rn(sum, (float)(rows * max(cols, 1u)));
            const float stored = Elem<LT>::round(mean);
            if (ok) {
                if (cw == 0) {
                    Elem<LT>::store(lp + (size_t)bh * g.Wb, mean);
                    if (keep) keep[pl * g.TPP + bh * g.Wb + bw] = stored;
                }
                float blo = 3.402823466e+38f, bhi = -3.402823466e+38f;
#pragma unroll
                for (int r = 0; r < P2; ++r) {
                    if ((uint32_t)r < rows) {
                        float a, b;
                        upk2(v[r], a, b);
                        if (CPL == 2 || (CPL == 3 && second)) {
                            blo = fmin3(blo, a, b);
                            bhi = fmax3(bhi, a, b);
                        } else {
                            blo = fminf(blo, a);
                            bhi = fmaxf(bhi, a);
                        }
                    }
                }
                // x -> fl(x - stored) is monotone: the residual extremes are those of the extreme x
                lo = fminf(lo, __fsub_rn(blo, stored));
                hi = fmaxf(hi, __fsub_rn(bhi, stored));
            }
        }
    }
}

template <typename XT, typename LT, int P2, int CPL>
__global__ void __launch_bounds__(256)
plane_stats_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, PlaneGeom g) {
    const uint32_t n = blockIdx.y;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
    plane_half1<XT, LT, P2, CPL>(x + (size_t)n * g.C * g.HW, lfc + (size_t)n * g.C * g.TPP, nullptr,
                                 (blockIdx.x * 8u + warp) * g.planes_per_warp, gridDim.x * 8u * g.planes_per_warp, g.C, g, lane,
                                 lo, hi);
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
    extern __shared__ __align__(16) uint32_t plane_smem[];
    uint2* quad_of = reinterpret_cast<uint2*>(plane_smem);                // quad inside a period -> where its 4 low-frequency values sit
    float* lfc_s = reinterpret_cast<float*>(plane_smem + g.table_words);  // stored low-frequency values of this CTA's planes
    const uint32_t n = blockIdx.y;
    for (uint32_t idx = threadIdx.x; idx < g.period; idx += 256u)
        quad_of[idx] = quad_table_entry(idx, g.HW, g.W, g.Wb, g.TPP, g.by_hw, g.by_w, g.by_b);
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
            const uint32_t grp = fdiv(q, g.by_period);
            const uint2 ent = quad_of[q - grp * g.period];
            // the period may start before the first plane staged here; the elements of this CTA do not
            const int lbase = ((int)(grp * g.period_planes) - (int)plane0) * (int)g.TPP;
            const float lf[4] = {lfc_s[lbase + (int)(ent.x & 0xFFFFu)], lfc_s[lbase + (int)(ent.x >> 16)],
                                 lfc_s[lbase + (int)(ent.y & 0xFFFFu)], lfc_s[lbase + (int)(ent.y >> 16)]};
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

// One launch for both halves.  CTA (b, n) owns the planes [b * ppc, (b + 1) * ppc) of sample n (ppc a multiple of 4
// and of the planes a warp takes at once, so that its elements are a whole number of quads):
//   1. block means, stored low-frequency values (also kept in shared memory) and residual extremes of its
//      planes, exactly as plane_stats_kernel; the CTA's extremes are folded into the sample's slot (two
//      reductions without an answer), then, behind a release fence, the CTA is counted as arrived;
//   2. thread 0 waits (bounded) until all CTAs of the sample have arrived and derives (delta, Delta, scale);
//   3. Eq. 9 and packing of the same planes as plane_quant_kernel, x read a second time (it is still in this
//      SM's L1 or in the L2), the low-frequency values from shared memory.
// The launch is cooperative so that the CTAs a wait depends on are resident; no grid-wide barrier is used.
struct PlaneFused {
    uint32_t ppc;                 // planes per CTA
    uint32_t ctas_per_sample;
    uint64_t timeout_ns;
    uint32_t expected;            // arrivals that complete a sample (a test may ask for an unreachable count)
};

template <typename XT, typename LT, int Q, int P2, int CPL>
__global__ void __launch_bounds__(256)
plane_fused_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, void* __restrict__ packed_v,
                   float* __restrict__ stats, PlaneGeom g, PlaneFused f, uint64_t seed) {
    typedef typename PackedUnit<Q>::type OutT;
    extern __shared__ __align__(16) uint32_t plane_smem[];
    uint2* quad_of = reinterpret_cast<uint2*>(plane_smem);                // quad inside a period -> where its 4 low-frequency values sit
    float* lfc_s = reinterpret_cast<float*>(plane_smem + g.table_words);  // stored low-frequency values of this CTA's planes
    __shared__ uint32_t s_kmin, s_kmax, s_delta, s_scale, s_ok;
    const uint32_t n = blockIdx.y;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t plane0 = blockIdx.x * f.ppc;
    const uint32_t nplanes = plane0 < g.C ? min(f.ppc, g.C - plane0) : 0u;
    for (uint32_t idx = threadIdx.x; idx < g.period; idx += 256u)
        quad_of[idx] = quad_table_entry(idx, g.HW, g.W, g.Wb, g.TPP, g.by_hw, g.by_w, g.by_b);
    if (threadIdx.x == 0) {
        s_kmin = 0;
        s_kmax = 0;
        s_ok = 0;
    }
    __syncthreads();

    // ---------------- half 1: a lane owns one or two tile columns of one plane ----------------
    {
        float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
        plane_half1<XT, LT, P2, CPL>(x + ((size_t)n * g.C + plane0) * g.HW, lfc + ((size_t)n * g.C + plane0) * g.TPP, lfc_s,
                                     warp * g.planes_per_warp, 8u * g.planes_per_warp, nplanes, g, lane, lo, hi);
        const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
        const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
        if (lane == 0) {
            atomicMax(&s_kmin, kmin);
            atomicMax(&s_kmax, kmax);
        }
    }
    __syncthreads();

    // ---------------- the sample's extremes: fold, count, wait for the other CTAs of the sample ----------------
    if (threadIdx.x == 0) {
        uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
        if (nplanes) {
            red_max_relaxed(slot + 0, s_kmin);
            red_max_relaxed(slot + 1, s_kmax);
        }
        fence_acq_rel_gpu();
        asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(slot + 2), "r"(1u) : "memory");
        uint32_t polls = 0;
        uint64_t t0 = 0;
        bool ok = true;
        while (ld_acquire_u32(slot + 2) != f.expected) {
            if ((++polls & 7u) == 0) {
                const uint64_t tn = now_ns();
                if (t0 == 0) t0 = tn;
                if (ld_relaxed_u32(ws) != 0u || tn - t0 > f.timeout_ns) {
                    atomicCAS(ws, 0u, (uint32_t)DIV_ERR_TIMEOUT);
                    atomicCAS(ws + 1, 0u, n + 1u);
                    ok = false;
                    break;
                }
            }
            __nanosleep(100);
        }
        if (ok) {
            const QParams qp = make_qparams(key_float(~ld_relaxed_u32(slot + 0)), key_float(ld_relaxed_u32(slot + 1)), Q);
            if (blockIdx.x == 0) {
                stats[2 * (size_t)n + 0] = qp.delta;
                stats[2 * (size_t)n + 1] = qp.step;
            }
            s_delta = __float_as_uint(qp.delta);
            s_scale = __float_as_uint(qp.scale);
            s_ok = 1;
        }
    }
    __syncthreads();
    if (!s_ok || nplanes == 0) return;

    // ---------------- half 2: a thread per 4 consecutive elements of the CTA's planes ----------------
    const float delta = __uint_as_float(s_delta), scale = __uint_as_float(s_scale);
    const uint64_t delta2 = pk2(delta, delta), scale2 = pk2(scale, scale);
    const uint64_t base = rng_sample_base(seed, n);
    const uint64_t sample_quad0 = (uint64_t)n * g.qps;
    const XT* x_n = x + (size_t)n * g.CHW;
    OutT* packed = reinterpret_cast<OutT*>(packed_v);
    const uint32_t qa = (plane0 * g.HW) >> 2, qb = ((plane0 + nplanes) * g.HW) >> 2;     // this CTA's quads [qa, qb)
    for (uint32_t q = qa + threadIdx.x; q < qb; q += 256u) {
        uint64_t xy, zw;
        StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(x_n + (size_t)q * 4u), xy, zw);
        const uint32_t grp = fdiv(q, g.by_period);
        const uint2 ent = quad_of[q - grp * g.period];
        // the period may start before this CTA's first plane; the elements of this CTA do not
        const int lbase = ((int)(grp * g.period_planes) - (int)plane0) * (int)g.TPP;
        const float lf[4] = {lfc_s[lbase + (int)(ent.x & 0xFFFFu)], lfc_s[lbase + (int)(ent.x >> 16)],
                             lfc_s[lbase + (int)(ent.y & 0xFFFFu)], lfc_s[lbase + (int)(ent.y >> 16)]};
        constexpr float qmax = (float)((1 << Q) - 1);
        const uint64_t z = rng_group(base, q);
        uint32_t b0, b1, b2, b3;
        quant2(xy, pk2(lf[0], lf[1]), delta2, scale2, qmax, (uint32_t)z, b0, b1);
        quant2(zw, pk2(lf[2], lf[3]), delta2, scale2, qmax, (uint32_t)(z >> 32), b2, b3);
        constexpr uint32_t BIAS = QUANT2_BITS * (1u + (1u << Q) + (1u << (2 * Q)) + (1u << (3 * Q)));   // mod 2^32
        packed[sample_quad0 + q] = (OutT)(b0 + (b1 << Q) + (b2 << (2 * Q)) + (b3 << (3 * Q)) - BIAS);
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
    g.cpl = (s.W % 2 == 0 && s.B % 2 == 0) ? 2u : 3u;
    g.lanes_per_plane = s.Wb * s.P2 / 2u;
    g.planes_per_warp = 32u / g.lanes_per_plane;
    g.groups = (s.C + g.planes_per_warp - 1) / g.planes_per_warp;
    g.qps = s.CHW / 4;
    g.table_words = quad_table_words(s.HW);
    g.period = quad_period(s.HW);
    g.period_planes = quad_period_planes(s.HW);
    g.by_period = host_fastdiv(g.period);
    g.planes_per_cta = flat_planes_per_cta(4u * 256u * PLANE_QPT, s.HW);
    if (flat_smem_bytes(4u * 256u * PLANE_QPT, s.HW, s.TPP) > 44000) return false;
    g.by_hw = host_fastdiv(s.HW);
    g.by_w = host_fastdiv(s.W);
    g.by_b = host_fastdiv(s.B);
    *out = g;
    return true;
}

// resident CTAs per SM of one instance of the fused kernel with `smem` bytes of dynamic shared memory (asked
// once per device and size)
template <typename XT, typename LT, int Q, int P2, int CPL>
inline int plane_fused_occupancy(int dev, size_t smem) {
    static SmemSeen cached[DEVICE_CACHE_SLOTS];          // .bytes holds (smem << 8) | count
    const void* kern = (const void*)plane_fused_kernel<XT, LT, Q, P2, CPL>;
    const bool slot = dev >= 0 && dev < DEVICE_CACHE_SLOTS && smem < (1u << 22);
    if (slot && cached[dev].fn.load(std::memory_order_acquire) == kern) {
        const int c = cached[dev].bytes.load(std::memory_order_acquire);
        if ((size_t)(c >> 8) == smem && (c & 255) > 0) return c & 255;
    }
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, plane_fused_kernel<XT, LT, Q, P2, CPL>, 256, smem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (slot && n > 0 && n < 256) {
        cached[dev].fn.store(nullptr, std::memory_order_release);
        cached[dev].bytes.store((int)((smem << 8) | (size_t)n), std::memory_order_release);
        cached[dev].fn.store(kern, std::memory_order_release);
    }
    return n;
}

// How the single-launch form would run a descriptor; false when it does not apply (its CTAs could not all be resident)
struct PlaneFusedPlan {
    uint32_t ppc, ctas_per_sample;
    size_t smem;
};
template <typename XT, typename LT, int Q, int P2, int CPL>
inline bool plan_plane_fused(const Shape& s, const PlaneGeom& g, const DeviceInfo& di, PlaneFusedPlan* out) {
    // planes per CTA: a multiple of 4 (whole quads) and of the planes a warp takes at once; about 8 CTAs per SM in all
    const uint32_t step = 4u / gcd_u32(4u, g.planes_per_warp) * g.planes_per_warp;
    uint32_t want = (uint32_t)((8ull * di.sms + s.N - 1) / s.N);
    if (want < 1) want = 1;
    uint32_t ppc = ((s.C + want - 1) / want + step - 1) / step * step;
    for (int attempt = 0; attempt < 2; ++attempt) {
        const uint32_t cps = (s.C + ppc - 1) / ppc;
        const size_t smem = 4ull * g.table_words + 4ull * ppc * s.TPP;
        if (smem > 40000) return false;
        const int occ = plane_fused_occupancy<XT, LT, Q, P2, CPL>(di.dev, smem);
        if (occ < 1) return false;
        if ((uint64_t)cps * s.N > (uint64_t)occ * di.sms) {
            if (attempt) return false;
            // fewer, larger CTAs so that all of them fit on the device at once
            const uint64_t fit = ((uint64_t)occ * di.sms) / s.N;
            if (fit < 1) return false;
            ppc = (uint32_t)(((s.C + fit - 1) / fit + step - 1) / step * step);
            continue;
        }
        out->ppc = ppc;
        out->ctas_per_sample = cps;
        out->smem = smem;
        return true;
    }
    return false;
}

// launch of the single-launch form; false when it does not apply or the launch was refused
template <typename XT, typename LT, int Q, int P2, int CPL>
inline bool launch_plane_fused(const Shape& s, const div_layout& lo, const PlaneGeom& g, const DeviceInfo& di, const void* x,
                               uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st, uint32_t expected, uint64_t timeout_ns) {
    PlaneFusedPlan pf;
    if (!plan_plane_fused<XT, LT, Q, P2, CPL>(s, g, di, &pf)) return false;
    PlaneFused f;
    f.ppc = pf.ppc;
    f.ctas_per_sample = pf.ctas_per_sample;
    f.timeout_ns = timeout_ns ? timeout_ns : 2000000000ull;
    f.expected = expected ? expected : pf.ctas_per_sample;
    const XT* xt = (const XT*)x;
    LT* lfc = (LT*)(blob + lo.lfc_off);
    void* packed = blob + lo.packed_off;
    float* stats = (float*)(blob + lo.stats_off);
    PlaneGeom gg = g;
    void* args[] = {(void*)&xt, (void*)&lfc, (void*)&ws, (void*)&packed, (void*)&stats, (void*)&gg, (void*)&f, (void*)&seed};
    if (cudaLaunchCooperativeKernel((const void*)plane_fused_kernel<XT, LT, Q, P2, CPL>, dim3(pf.ctas_per_sample, s.N), dim3(256), args,
                                    pf.smem, st) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return true;
}

template <typename XT, typename LT>
inline bool launch_plane_fused_q(int qbits, const Shape& s, const div_layout& lo, const PlaneGeom& g, const DeviceInfo& di,
                                 const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st, uint32_t expected,
                                 uint64_t timeout_ns) {
#define DIVK_PF(QQ, PP)                                                                                              \
    (g.cpl == 2 ? launch_plane_fused<XT, LT, QQ, PP, 2>(s, lo, g, di, x, blob, ws, seed, st, expected, timeout_ns) \
                : launch_plane_fused<XT, LT, QQ, PP, 3>(s, lo, g, di, x, blob, ws, seed, st, expected, timeout_ns))
    switch (s.P2) {
        case 4: return qbits == 2 ? DIVK_PF(2, 4) : qbits == 4 ? DIVK_PF(4, 4) : DIVK_PF(8, 4);
        case 8: return qbits == 2 ? DIVK_PF(2, 8) : qbits == 4 ? DIVK_PF(4, 8) : DIVK_PF(8, 8);
        case 16: return qbits == 2 ? DIVK_PF(2, 16) : qbits == 4 ? DIVK_PF(4, 16) : DIVK_PF(8, 16);
    }
#undef DIVK_PF
    return false;
}

// would the single-launch form run this descriptor?  (fills grid / shared memory for div_plan_query)
inline bool plane_fused_applies(const div_desc* d, const Shape& s, const PlaneGeom& g, PlaneFusedPlan* out) {
    typedef __nv_bfloat16 bf16;
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return false;
#define DIVK_PP(XT, LT, QQ, PP) \
    (g.cpl == 2 ? plan_plane_fused<XT, LT, QQ, PP, 2>(s, g, di, out) : plan_plane_fused<XT, LT, QQ, PP, 3>(s, g, di, out))
#define DIVK_PQ(XT, LT, PP) (d->qbits == 2 ? DIVK_PP(XT, LT, 2, PP) : d->qbits == 4 ? DIVK_PP(XT, LT, 4, PP) : DIVK_PP(XT, LT, 8, PP))
#define DIVK_PT(XT, LT) (s.P2 == 4 ? DIVK_PQ(XT, LT, 4) : s.P2 == 8 ? DIVK_PQ(XT, LT, 8) : s.P2 == 16 ? DIVK_PQ(XT, LT, 16) : false)
    if (d->x_dtype == DIV_F32) return d->lfc_dtype == DIV_F32 ? DIVK_PT(float, float) : DIVK_PT(float, bf16);
    return d->lfc_dtype == DIV_F32 ? DIVK_PT(bf16, float) : DIVK_PT(bf16, bf16);
#undef DIVK_PT
#undef DIVK_PQ
#undef DIVK_PP
}

template <typename XT, typename LT>
inline div_status compress_planes_t(const div_desc* d, const Shape& s, const div_layout& lo, const PlaneGeom& g,
                                    const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st,
                                    bool allow_fused, uint32_t expected, uint64_t timeout_ns) {
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return DIV_ERR_CUDA;
    if (allow_fused && launch_plane_fused_q<XT, LT>(d->qbits, s, lo, g, di, x, blob, ws, seed, st, expected, timeout_ns)) return DIV_OK;
    if (expected) return DIV_ERR_PARAM;              // the test hook is about the single-launch form only
    // pass 1: enough CTAs per sample to fill the GPU a few times over, never more than there are warp passes
    uint32_t bx = (uint32_t)((8ull * di.sms + s.N - 1) / s.N);
    const uint32_t bx_max = (g.groups + 7u) / 8u;
    if (bx > bx_max) bx = bx_max;
    if (bx < 1) bx = 1;
    const dim3 grid1(bx, s.N);
    const XT* xt = (const XT*)x;
    LT* lfc = (LT*)(blob + lo.lfc_off);
    switch (s.P2) {
        case 4:
            if (g.cpl == 2) plane_stats_kernel<XT, LT, 4, 2><<<grid1, 256, 0, st>>>(xt, lfc, ws, g);
            else plane_stats_kernel<XT, LT, 4, 3><<<grid1, 256, 0, st>>>(xt, lfc, ws, g);
            break;
        case 8:
            if (g.cpl == 2) plane_stats_kernel<XT, LT, 8, 2><<<grid1, 256, 0, st>>>(xt, lfc, ws, g);
            else plane_stats_kernel<XT, LT, 8, 3><<<grid1, 256, 0, st>>>(xt, lfc, ws, g);
            break;
        case 16:
            if (g.cpl == 2) plane_stats_kernel<XT, LT, 16, 2><<<grid1, 256, 0, st>>>(xt, lfc, ws, g);
            else plane_stats_kernel<XT, LT, 16, 3><<<grid1, 256, 0, st>>>(xt, lfc, ws, g);
            break;
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
                                  const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st,
                                  bool allow_fused = true, uint32_t expected = 0, uint64_t timeout_ns = 0) {
    typedef __nv_bfloat16 bf16;
    if (d->x_dtype == DIV_F32) {
        if (d->lfc_dtype == DIV_F32) return compress_planes_t<float, float>(d, s, lo, g, x, blob, ws, seed, st, allow_fused, expected, timeout_ns);
        return compress_planes_t<float, bf16>(d, s, lo, g, x, blob, ws, seed, st, allow_fused, expected, timeout_ns);
    }
    if (d->lfc_dtype == DIV_F32) return compress_planes_t<bf16, float>(d, s, lo, g, x, blob, ws, seed, st, allow_fused, expected, timeout_ns);
    return compress_planes_t<bf16, bf16>(d, s, lo, g, x, blob, ws, seed, st, allow_fused, expected, timeout_ns);
}

}  // namespace divk
