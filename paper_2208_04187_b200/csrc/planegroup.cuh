// Per-plane quantisation groups: one (delta, Delta) pair of two bfloat16 numbers per (sample, channel)
// plane -- the grouping behind the paper's byte count of N^2*Q/8 + 4 bytes per channel (Sec. 4.1, proof
// of Theorem 3A; "Delta and delta are cached in bfloat16").  Pooling, residual, stochastic rounding, the
// random stream and the packing order are those of the per-sample kernels.
//
// Rounding of the pair (the paper is silent): delta_b is the largest bfloat16 number <= min H^H and
// Delta_b the smallest bfloat16 number >= (max H^H - delta_b) / (2^Q - 1); encoder and decoder both use the
// stored pair: t = (h - delta_b) * (1 / Delta_b), h_hat = Delta_b * code + delta_b.  So t never turns
// negative and never passes 2^Q - 1 by more than a rounding error, which the clamp absorbs.
//
// A plane's extremes need no communication between CTAs here, so compress is a true single pass:
//   pg_strip_kernel    W % 4 == 0, B in {4, 8}, Q in {2, 4, 8}, planes of at most PG_CAP strip slots: a CTA
//                      takes a few whole planes; every thread keeps its strips (4 columns x B rows) in
//                      registers from the load, through the tile means and the CTA-wide extremes, to the
//                      quantiser.  x crosses HBM once and is never re-read from anywhere.
//   pg_general_kernel  any shape: one CTA per plane, second read of the plane from L1/L2.
#pragma once

#include "decompress.cuh"
#include "lagged.cuh"
#include "planes.cuh"     // ColLoad

namespace divk {

// Shape of the strip kernel: one strip slot per thread; a CTA of up to PG_MAX_THREADS threads takes one large
// plane, or a few whole small planes (CTAs of about DIVK_PG_SMALL_CTA threads, twice that for medium planes).
#ifndef DIVK_PG_SMALL_CTA
#define DIVK_PG_SMALL_CTA 128
#endif
constexpr uint32_t PG_MAX_THREADS = 512;
constexpr int PG_K = 1;                           // strip slots a thread keeps in registers
constexpr uint32_t PG_CAP = PG_MAX_THREADS;       // most strip slots of a plane

// ------------------------------------------------------------------------------------------------
// the bfloat16 pair of one plane
// ------------------------------------------------------------------------------------------------
struct PgQ {
    float delta;   // delta_b as fp32
    float step;    // Delta_b as fp32 (0: degenerate plane, every code 0)
    float scale;   // 1 / Delta_b (0 when degenerate)
};
__device__ __forceinline__ bool f32_finite(float v) { return (__float_as_uint(v) & 0x7F800000u) != 0x7F800000u; }
// largest bfloat16 number <= v / smallest bfloat16 number >= v, as fp32; a zero comes out as +0.0
__device__ __forceinline__ float bf16_floor(float v) {
    const uint32_t u = __float_as_uint(v);
    uint32_t hi = u >> 16;
    if ((u & 0xFFFFu) != 0u && v < 0.f) hi += 1u;     // cutting the low bits moves a negative number up
    if (v == 0.f) hi = 0u;
    return __uint_as_float(hi << 16);
}
__device__ __forceinline__ float bf16_ceil(float v) {
    const uint32_t u = __float_as_uint(v);
    uint32_t hi = u >> 16;
    if ((u & 0xFFFFu) != 0u && v > 0.f) hi += 1u;     // cutting the low bits moves a positive number down
    if (v == 0.f) hi = 0u;
    return __uint_as_float(hi << 16);
}
__device__ __forceinline__ PgQ pg_params(float rmin, float rmax, int qbits) {
    PgQ q = {0.f, 0.f, 0.f};
    const float d = bf16_floor(rmin);
    if (!f32_finite(d)) return q;                     // minimum below the most negative bfloat16 number
    q.delta = d;
    const float step = __fdiv_rn(__fsub_rn(rmax, d), (float)((1 << qbits) - 1));
    if (!f32_finite(step)) return q;
    const float sb = bf16_ceil(step);
    if (!f32_finite(sb) || !(sb > 0.f)) return q;
    const float sc = __fdiv_rn(1.0f, sb);
    if (!f32_finite(sc) || !(sc > 0.f)) return q;
    q.step = sb;
    q.scale = sc;
    return q;
}
// the stored pair: low half-word delta_b, high half-word Delta_b
__device__ __forceinline__ uint32_t pg_stats_word(const PgQ& q) {
    return (__float_as_uint(q.delta) >> 16) | (__float_as_uint(q.step) & 0xFFFF0000u);
}

// ------------------------------------------------------------------------------------------------
// strip kernel
// ------------------------------------------------------------------------------------------------
struct PgParams {
    Shape s;
    const void* x;
    void* lfc;
    void* packed;
    uint32_t* stats;
    uint64_t seed;
    uint64_t rng_row_step;   // K_GROUP * (W / 4)
    uint32_t planes;         // N * C
    uint32_t spb, spp;       // strip slots per band and per plane
    uint32_t G;              // planes per CTA
    uint32_t tail_rows;      // rows of the last band of a plane
    FastDiv by_spp, by_spb, by_c;
    float inv_cnt[4];        // as in the lagged kernel: [tail row band][tail column tile]
    float cnt[4];
};

template <typename XT, typename LT, int Q, int P2>
__global__ void __launch_bounds__(PG_MAX_THREADS, 2)
pg_strip_kernel(const PgParams p) {
    constexpr uint32_t LPT = P2 / 4;
    typedef typename PackedUnit<Q>::type OutT;
    __shared__ uint32_t s_key[2 * PG_MAX_THREADS];     // per plane of this CTA: ~key(min), key(max)
    __shared__ float s_par[2 * PG_MAX_THREADS];        // per plane: delta_b, 1 / Delta_b

    const Shape& s = p.s;
    const uint32_t tid = threadIdx.x;
    const uint32_t PG_THREADS = blockDim.x;               // a multiple of 32
    const uint32_t row_bytes = s.W * (uint32_t)sizeof(XT);
    const uint32_t W4 = s.W >> 2;
    const uint32_t plane0 = blockIdx.x * p.G;
    for (uint32_t i = tid; i < 2u * p.G; i += PG_THREADS) s_key[i] = 0u;

    // ---- where this thread's slots are, and their loads (everything a thread reads is requested at once)
    uint32_t rows[PG_K], pl[PG_K], first[PG_K], tile[PG_K], which[PG_K];
    uint64_t vxy[PG_K][P2], vzw[PG_K][P2];
#pragma unroll
    for (int k = 0; k < PG_K; ++k) {
        const uint32_t S = tid + (uint32_t)k * PG_THREADS;
        pl[k] = fdiv(S, p.by_spp);
        const uint32_t sl = S - pl[k] * p.spp;
        const uint32_t bh = fdiv(sl, p.by_spb);
        const uint32_t q = sl - bh * p.spb;
        const bool ok = pl[k] < p.G && plane0 + pl[k] < p.planes && 4u * q < s.W;
        rows[k] = ok ? ((bh + 1u == s.Hb) ? p.tail_rows : s.B) : 0u;
        first[k] = bh * s.B * s.W + 4u * q;                  // first element of the slot inside its plane
        tile[k] = bh * s.Wb + q / LPT;
        const uint32_t tail_col = (q / LPT == s.Wb - 1u && (s.W % s.B) != 0u) ? 1u : 0u;
        which[k] = ((rows[k] != s.B) ? 2u : 0u) + tail_col;
        const unsigned char* xs = reinterpret_cast<const unsigned char*>(
            reinterpret_cast<const XT*>(p.x) + ((size_t)(plane0 + (ok ? pl[k] : 0u)) * s.HW + first[k]));
#pragma unroll
        for (int r = 0; r < P2; ++r) {
            if ((uint32_t)r < rows[k]) {
                StripRow2<XT>::load(xs + (size_t)r * row_bytes, vxy[k][r], vzw[k][r]);
            } else {
                vxy[k][r] = 0ull;
                vzw[k][r] = 0ull;
            }
        }
    }
    __syncthreads();      // the key slots are cleared

    // ---- tile means (fixed summation order), stored low-frequency values, extremes of the residual
    float stored[PG_K];
#pragma unroll
    for (int k = 0; k < PG_K; ++k) {
        uint64_t cxy[P2], czw[P2];
#pragma unroll
        for (int r = 0; r < P2; ++r) {
            cxy[r] = vxy[k][r];
            czw[r] = vzw[k][r];
        }
#pragma unroll
        for (int w = P2; w > 1; w >>= 1) {
#pragma unroll
            for (int i = 0; i < w / 2; ++i) {
                cxy[i] = add2_rn(cxy[2 * i], cxy[2 * i + 1]);
                czw[i] = add2_rn(czw[2 * i], czw[2 * i + 1]);
            }
        }
        float c0, c1, c2, c3;
        upk2(cxy[0], c0, c1);
        upk2(czw[0], c2, c3);
        float sum = __fadd_rn(__fadd_rn(c0, c1), __fadd_rn(c2, c3));
#pragma unroll
        for (int m = 1; m < (int)LPT; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
        const float inv = p.inv_cnt[which[k]];
        const float mean = (inv != 0.f) ? __fmul_rn(sum, inv) : __fdiv_rn(sum, p.cnt[which[k]]);
        stored[k] = Elem<LT>::round(mean);
        if (rows[k] != 0u) {
            if ((tid % LPT) == 0u)
                Elem<LT>::store(reinterpret_cast<LT*>(p.lfc) + ((size_t)(plane0 + pl[k]) * s.TPP + tile[k]), mean);
            // extremes of x over the in-bounds rows; x -> fl(x - stored) is monotone
            float blo = 3.402823466e+38f, bhi = -3.402823466e+38f;
#pragma unroll
            for (int r = 0; r < P2; ++r) {
                if ((uint32_t)r < rows[k]) {
                    float a_, b_, c_, d_;
                    upk2(vxy[k][r], a_, b_);
                    upk2(vzw[k][r], c_, d_);
                    blo = fmin3(blo, a_, b_);
                    blo = fmin3(blo, c_, d_);
                    bhi = fmax3(bhi, a_, b_);
                    bhi = fmax3(bhi, c_, d_);
                }
            }
            atomicMax(&s_key[2u * pl[k]], ~float_key(__fsub_rn(blo, stored[k])));
            atomicMax(&s_key[2u * pl[k] + 1u], float_key(__fsub_rn(bhi, stored[k])));
        }
    }
    __syncthreads();      // every plane's extremes are complete

    for (uint32_t i = tid; i < p.G; i += PG_THREADS) {
        if (plane0 + i < p.planes) {
            const PgQ q = pg_params(key_float(~s_key[2u * i]), key_float(s_key[2u * i + 1u]), Q);
            s_par[2u * i] = q.delta;
            s_par[2u * i + 1u] = q.scale;
            p.stats[plane0 + i] = pg_stats_word(q);
        }
    }
    __syncthreads();

    // ---- Eq. 9 on the values still held in registers
#pragma unroll
    for (int k = 0; k < PG_K; ++k) {
        if (rows[k] != 0u) {
            const uint32_t plane = plane0 + pl[k];
            const uint32_t n = fdiv(plane, p.by_c);
            const uint32_t c = plane - n * s.C;
            const float delta = s_par[2u * pl[k]], scale = s_par[2u * pl[k] + 1u];
            const uint64_t delta2 = pk2(delta, delta), scale2 = pk2(scale, scale), stored2 = pk2(stored[k], stored[k]);
            const uint32_t e = c * s.HW + first[k];                         // in-sample index, a multiple of 4
            uint64_t ctr = rng_sample_base(p.seed, n) + K_GROUP * (uint64_t)((e >> 2) + 1u);
            OutT* out = reinterpret_cast<OutT*>(p.packed) + ((((uint64_t)plane * s.HW) + first[k]) >> 2);
#pragma unroll
            for (int r = 0; r < P2; ++r) {
                if ((uint32_t)r < rows[k]) *out = (OutT)quant_row<Q>(vxy[k][r], vzw[k][r], stored2, delta2, scale2, rng_mix(ctr));
                out += W4;
                ctr += p.rng_row_step;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// small-plane kernel: planes of any width whose padded tile row fits a warp (the 14 x 14 and 7 x 7 maps).
// A CTA takes G whole planes, contiguous in memory.  First half: a lane owns one tile column of one plane
// (as in plane_stats_kernel): block means in the fixed order, stored low-frequency values (also kept in
// shared memory), extremes per plane through shared-memory atomics.  Second half: one thread per 4
// consecutive elements of the CTA's range (they may lie in different tiles, rows or planes; the tile of a
// position comes from a table in shared memory); x is read a second time, from L1/L2.
// ------------------------------------------------------------------------------------------------
struct PgSmall {
    Shape s;
    const void* x;
    void* lfc;
    void* packed;
    uint32_t* stats;
    uint64_t seed;
    uint32_t planes;            // N * C
    uint32_t G;                 // planes per CTA; G * HW is a multiple of 4
    uint32_t cpl;               // first half, how a lane reads its 2 adjacent columns: 2 = one 8-byte load (W and B even), 3 = two loads
    uint32_t quads_same_plane;  // 1: HW % 4 == 0, the 4 elements of a quad lie in one plane (quad table instead of the tile table)
    uint32_t lanes_per_plane;   // Wb * P2 / 2
    uint32_t planes_per_warp;   // 32 / lanes_per_plane
    uint32_t table_words;       // 32-bit words of the tile table
    FastDiv by_hw, by_w, by_b, by_c;
};
inline size_t pg_small_smem_bytes(const PgSmall& g) {
    return 4ull * (g.table_words + (size_t)g.G * g.s.TPP + 4ull * g.G);
}

template <typename XT, typename LT, int Q, int P2, int CPL>
__global__ void __launch_bounds__(256)
pg_small_kernel(const PgSmall g) {
    typedef typename PackedUnit<Q>::type OutT;
    extern __shared__ __align__(16) uint32_t pg_smem[];
    const Shape& s = g.s;
    uint16_t* tile_of = reinterpret_cast<uint16_t*>(pg_smem);                 // position in a plane -> tile in the plane
    float* lfc_s = reinterpret_cast<float*>(pg_smem + g.table_words);         // stored low-frequency values, G * TPP
    uint32_t* s_key = pg_smem + g.table_words + g.G * s.TPP;                  // per plane: ~key(min), key(max)
    float* s_par = reinterpret_cast<float*>(s_key + 2u * g.G);                // per plane: delta_b, 1 / Delta_b
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31u;
    const uint32_t plane0 = blockIdx.x * g.G;
    const uint32_t nplanes = min(g.G, g.planes - plane0);
    const XT* x = reinterpret_cast<const XT*>(g.x);

    uint2* quad_of = reinterpret_cast<uint2*>(pg_smem);                       // HW % 4 == 0: quad in a plane -> its 4 tiles
    if (g.quads_same_plane) {
        for (uint32_t idx = tid; idx < (s.HW >> 2); idx += 256u)
            quad_of[idx] = quad_table_entry(idx, s.HW, s.W, s.Wb, s.TPP, g.by_hw, g.by_w, g.by_b);
    } else {
        for (uint32_t idx = tid; idx < s.HW; idx += 256u) {
            const uint32_t h = fdiv(idx, g.by_w), w = idx - h * s.W;
            tile_of[idx] = (uint16_t)(fdiv(h, g.by_b) * s.Wb + fdiv(w, g.by_b));
        }
    }
    for (uint32_t i = tid; i < 2u * g.G; i += 256u) s_key[i] = 0u;
    __syncthreads();

    // ---- first half: lane = two adjacent columns of one tile (packed adds; CPL says how they are loaded, see load_cols)
    {
        constexpr uint32_t NC = CPL == 1 ? 1u : 2u;
        constexpr uint32_t LPT = P2 / NC;                                   // lanes per tile
        const uint32_t pl_local = lane / g.lanes_per_plane;
        const uint32_t lw = lane - pl_local * g.lanes_per_plane;
        const uint32_t bw = lw / LPT, cw = (lw % LPT) * NC;
        const uint32_t cols = (bw < s.Wb) ? min(s.B, s.W - bw * s.B) : 0u;
        const bool lane_ok = pl_local < g.planes_per_warp && cw < cols;
        const bool second = cw + 1u < cols;
        const uint32_t col = bw * s.B + cw;
        for (uint32_t pp = warp; pp * g.planes_per_warp < nplanes; pp += 8u) {
            const uint32_t pc = pp * g.planes_per_warp + pl_local;          // plane inside the CTA
            const bool ok = lane_ok && pc < nplanes;
            const XT* xp = x + ((size_t)(plane0 + (ok ? pc : 0u)) * s.HW + (ok ? col : 0u));
            LT* lp = reinterpret_cast<LT*>(g.lfc) + ((size_t)(plane0 + (ok ? pc : 0u)) * s.TPP + (ok ? bw : 0u));
            float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
            for (uint32_t bh = 0; bh < s.Hb; ++bh) {
                const uint32_t rows = min(s.B, s.H - bh * s.B);
                uint64_t v[P2];
#pragma unroll
                for (int r = 0; r < P2; ++r)
                    v[r] = (ok && (uint32_t)r < rows) ? load_cols<XT, CPL>(xp + (size_t)(bh * s.B + r) * s.W, second) : 0ull;
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
                float sum = NC == 2 ? __fadd_rn(c0, c1) : c0;
#pragma unroll
                for (int m = 1; m < (int)LPT; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
                // after the butterfly every lane of a tile holds the same sum: each divides for itself
                const float mean = __fdiv_rn(sum, (float)(rows * max(cols, 1u)));
                const float stored = Elem<LT>::round(mean);
                if (ok) {
                    if (cw == 0) {
                        Elem<LT>::store(lp + (size_t)bh * s.Wb, mean);
                        lfc_s[pc * s.TPP + bh * s.Wb + bw] = stored;
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
            // the columns of one tile meet through shuffles, the tiles of one plane in shared memory
            uint32_t kmin = ~float_key(lo), kmax = float_key(hi);
#pragma unroll
            for (int m = 1; m < (int)LPT; m <<= 1) {
                kmin = max(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, m));
                kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, m));
            }
            if (pl_local < g.planes_per_warp && bw < s.Wb && cw == 0 && pc < nplanes) {
                atomicMax(&s_key[2u * pc], kmin);
                atomicMax(&s_key[2u * pc + 1u], kmax);
            }
        }
    }
    __syncthreads();
    for (uint32_t i = tid; i < nplanes; i += 256u) {
        const PgQ q = pg_params(key_float(~s_key[2u * i]), key_float(s_key[2u * i + 1u]), Q);
        s_par[2u * i] = q.delta;
        s_par[2u * i + 1u] = q.scale;
        g.stats[plane0 + i] = pg_stats_word(q);
    }
    __syncthreads();

    // ---- second half: Eq. 9 on 4 consecutive elements per step
    {
        constexpr float qmax = (float)((1 << Q) - 1);
        const uint64_t e0 = (uint64_t)plane0 * s.HW;                      // first element of the CTA, a multiple of 4
        const uint32_t nquads = (nplanes * s.HW) >> 2;
        const XT* xc = x + e0;
        OutT* out = reinterpret_cast<OutT*>(g.packed) + (e0 >> 2);
        for (uint32_t qi = tid; qi < nquads; qi += 256u) {
            uint64_t xy, zw;
            StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(xc + (size_t)qi * 4u), xy, zw);
            uint32_t pc = fdiv(qi * 4u, g.by_hw);
            uint32_t rem = qi * 4u - pc * s.HW;
            // the 4 elements lie in one sample (its size is a multiple of 4)
            const uint32_t plane = plane0 + pc;
            const uint32_t n = fdiv(plane, g.by_c);
            const uint32_t e = (plane - n * s.C) * s.HW + rem;             // in-sample index of the first element
            float lf[4], dl[4], sc[4];
            if (g.quads_same_plane) {
                // one 8-byte entry holds the 4 tiles; one pair of parameters for the quad
                const uint2 ent = quad_of[rem >> 2];
                const float* lp = lfc_s + pc * s.TPP;
                lf[0] = lp[ent.x & 0xFFFFu];
                lf[1] = lp[ent.x >> 16];
                lf[2] = lp[ent.y & 0xFFFFu];
                lf[3] = lp[ent.y >> 16];
                const float d0 = s_par[2u * pc], s0 = s_par[2u * pc + 1u];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    dl[i] = d0;
                    sc[i] = s0;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    lf[i] = lfc_s[pc * s.TPP + tile_of[rem]];
                    dl[i] = s_par[2u * pc];
                    sc[i] = s_par[2u * pc + 1u];
                    if (++rem == s.HW) {
                        rem = 0;
                        ++pc;
                    }
                }
            }
            const uint64_t z = rng_group(rng_sample_base(g.seed, n), e >> 2);
            uint32_t b0, b1, b2, b3;
            quant2(xy, pk2(lf[0], lf[1]), pk2(dl[0], dl[1]), pk2(sc[0], sc[1]), qmax, (uint32_t)z, b0, b1);
            quant2(zw, pk2(lf[2], lf[3]), pk2(dl[2], dl[3]), pk2(sc[2], sc[3]), qmax, (uint32_t)(z >> 32), b2, b3);
            constexpr uint32_t BIAS = QUANT2_BITS * (1u + (1u << Q) + (1u << (2 * Q)) + (1u << (3 * Q)));   // mod 2^32
            out[qi] = (OutT)(b0 + (b1 << Q) + (b2 << (2 * Q)) + (b3 << (3 * Q)) - BIAS);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// general kernel: one CTA per plane, any shape
// ------------------------------------------------------------------------------------------------
template <typename XT, typename LT, int Q>
__global__ void __launch_bounds__(256)
pg_general_kernel(const XT* __restrict__ x, LT* lfc, uint32_t* packed, uint32_t* __restrict__ stats, Shape s,
                  uint64_t seed) {
    constexpr uint32_t PER = 32 / Q;
    constexpr float qmax = (float)((1 << Q) - 1);
    __shared__ uint32_t s_kmin, s_kmax;
    __shared__ float s_delta, s_scale;
    const uint32_t tid = threadIdx.x;
    const uint32_t plane = blockIdx.x;
    const uint32_t n = plane / s.C, c = plane - n * s.C;
    const XT* xp = x + (size_t)plane * s.HW;
    LT* lp = lfc + (size_t)plane * s.TPP;
    if (tid == 0) {
        s_kmin = 0u;
        s_kmax = 0u;
    }
    __syncthreads();
    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
    for (uint32_t t = tid; t < s.TPP; t += 256u) {
        float xmin, xmax;
        const float mean = tile_mean(xp, s, t / s.Wb, t % s.Wb, xmin, xmax);
        Elem<LT>::store(lp + t, mean);
        const float stored = Elem<LT>::round(mean);
        lo = fminf(lo, __fsub_rn(xmin, stored));
        hi = fmaxf(hi, __fsub_rn(xmax, stored));
    }
    const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
    const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
    if ((tid & 31u) == 0u) {
        atomicMax(&s_kmin, kmin);
        atomicMax(&s_kmax, kmax);
    }
    __syncthreads();
    if (tid == 0) {
        const PgQ q = pg_params(key_float(~s_kmin), key_float(s_kmax), Q);
        s_delta = q.delta;
        s_scale = q.scale;
        stats[plane] = pg_stats_word(q);
    }
    __syncthreads();      // also makes this CTA's low-frequency values visible to all its threads
    const float delta = s_delta, scale = s_scale;
    const uint64_t base = rng_sample_base(seed, n);
    const uint64_t i0 = (uint64_t)plane * s.HW, i1 = i0 + s.HW;       // the plane's global element range
    const uint64_t w0 = i0 / PER, w1 = (i1 + PER - 1) / PER;
    for (uint64_t word = w0 + tid; word < w1; word += 256u) {
        const uint64_t a = max(word * PER, i0), b = min((word + 1) * PER, i1);
        uint32_t acc = 0;
        uint32_t cur_g = 0xFFFFFFFFu;
        uint64_t z = 0;
        for (uint64_t i = a; i < b; ++i) {
            const uint32_t ep = (uint32_t)(i - i0);
            const uint32_t h = ep / s.W, w = ep - h * s.W;
            const uint32_t e = c * s.HW + ep;
            if ((e >> 2) != cur_g) {
                cur_g = e >> 2;
                z = rng_group(base, cur_g);
            }
            const float l = Elem<LT>::load(lp + (h / s.B) * s.Wb + (w / s.B));
            const float r = __fsub_rn(Elem<XT>::load(xp + ep), l);
            const uint32_t field = (uint32_t)(z >> (16 * (e & 3))) & 0xFFFFu;
            const uint32_t code = quant_bits(r, delta, scale, qmax, field) - MAGIC_CEIL_BITS;
            acc |= code << ((uint32_t)(i - word * PER) * Q);
        }
        // a word shared with a neighbouring plane (or the zero-padded end of the stream) is merged into the
        // pre-cleared buffer; every other word is written whole
        if (b - a == PER) packed[word] = acc;
        else atomicOr(packed + word, acc);
    }
}

// ------------------------------------------------------------------------------------------------
// decompress: x_hat = UpSampling(H^L) + (Delta_b * V^H + delta_b)   (Sec. 4.2, Eq. 10)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void pg_unpack_stats(uint32_t w, float& delta, float& step) {
    delta = __uint_as_float(w << 16);
    step = __uint_as_float(w & 0xFFFF0000u);
}

// W % 4 == 0 and B a power of two >= 4: same tiling of the work as decompress_quad_kernel (a thread produces
// the same 4 columns of 4 consecutive rows: one low-frequency value, one plane pair, one set of index arithmetic)
// SPREAD: as in decompress_quad_kernel (rows that are not whole 32-byte sectors: the 4 rows of an item lie
// hq_count rows apart, each with its own tile's low-frequency value)
template <typename XT, typename LT, int Q, int QPT, bool SPREAD>
__global__ void __launch_bounds__(256)
pg_decompress_quad_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                          const uint32_t* __restrict__ stats, XT* __restrict__ xhat, DecFast d) {
    static_assert(QPT == 4, "a work item is 4 rows high");
    constexpr uint32_t MASK = (1u << Q) - 1u;
    const uint32_t n = blockIdx.y;
    const uint32_t item = blockIdx.x * 256u + threadIdx.x;
    if (item >= d.items) return;
    const uint32_t plane = fdiv(item, d.by_ipp);
    const uint32_t rem = item - plane * d.ipp;
    const uint32_t hq = fdiv(rem, d.by_wq);
    const uint32_t wq = rem - hq * d.wq;
    const uint32_t h0 = SPREAD ? hq : hq * 4u;
    const uint32_t hstep = SPREAD ? d.hq_count : 1u;
    const size_t gp = (size_t)n * d.C + plane;
    const LT* lfc_p = lfc + gp * d.TPP + ((wq * 4u) >> d.log2B);
    float delta, step;
    pg_unpack_stats(__ldg(stats + gp), delta, step);
    const uint64_t quad0 = (uint64_t)n * d.qps + plane * d.hwq + h0 * d.wq + wq;
    const uint32_t qstep = hstep * d.wq;
    uint32_t bits[4];
    float lf[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const uint32_t h = h0 + (uint32_t)r * hstep;
        bits[r] = 0u;
        lf[r] = 0.f;
        if (h < d.H) {
            bits[r] = quad_bits<Q>(packed, quad0 + (uint32_t)r * qstep);
            if (SPREAD || r == 0) lf[r] = Elem<LT>::load(lfc_p + (h >> d.log2B) * d.Wb);
        }
        if (!SPREAD && r > 0) lf[r] = lf[0];
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        if (h0 + (uint32_t)r * hstep < d.H) {
            Quad<XT>::store(xhat + (quad0 + (uint32_t)r * qstep) * 4u, reconstruct(bits[r] & MASK, step, delta, lf[r]),
                            reconstruct((bits[r] >> Q) & MASK, step, delta, lf[r]),
                            reconstruct((bits[r] >> (2 * Q)) & MASK, step, delta, lf[r]),
                            reconstruct((bits[r] >> (3 * Q)) & MASK, step, delta, lf[r]));
        }
    }
}

// any shape: one thread per packed word
template <typename XT, typename LT, int Q>
__global__ void __launch_bounds__(256)
pg_decompress_general_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                             const uint32_t* __restrict__ stats, XT* __restrict__ xhat, Shape s, uint64_t nwords) {
    constexpr uint32_t PER = 32 / Q;
    constexpr uint32_t MASK = (1u << Q) - 1u;
    const uint64_t word = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= nwords) return;
    uint64_t i = word * PER;
    uint64_t plane = i / s.HW;                       // global plane index n * C + c
    uint32_t rem = (uint32_t)(i - plane * s.HW);
    uint32_t h = rem / s.W, w = rem - h * s.W;
    const uint32_t bits = packed[word];
    uint64_t cur = ~0ull;
    float delta = 0.f, step = 0.f;
    for (uint32_t j = 0; j < PER && i < s.total; ++j, ++i) {
        if (plane != cur) {
            pg_unpack_stats(stats[plane], delta, step);
            cur = plane;
        }
        const float l = Elem<LT>::load(lfc + plane * s.TPP + (h / s.B) * s.Wb + (w / s.B));
        Elem<XT>::store(xhat + i, reconstruct((bits >> (j * Q)) & MASK, step, delta, l));
        if (++w == s.W) {
            w = 0;
            if (++h == s.H) {
                h = 0;
                ++plane;
            }
        }
    }
}

// total size a multiple of 4, planes of at most FLAT_MAX_HW elements, any W and B: one thread per 4 consecutive
// elements of the flat stream; the tile of a position comes from a table in shared memory, the plane's pair
// and low-frequency values from global memory (a few bytes per plane, served by L1)
struct PgDecFlat {
    uint64_t quads;          // N*C*H*W / 4
    uint32_t HW, W, Wb, TPP;
    uint32_t table_words;
    uint32_t quads_same_plane;   // 1: HW % 4 == 0, a quad lies in one plane (quad table, one pair of parameters per quad)
    FastDiv by_hw, by_w, by_b;
};
template <typename XT, typename LT, int Q, int QPT>
__global__ void __launch_bounds__(256)
pg_decompress_flat_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                          const uint32_t* __restrict__ stats, XT* __restrict__ xhat, PgDecFlat d) {
    constexpr uint32_t MASK = (1u << Q) - 1u;
    extern __shared__ __align__(16) uint32_t pg_smem[];
    uint16_t* tile_of = reinterpret_cast<uint16_t*>(pg_smem);
    uint2* quad_of = reinterpret_cast<uint2*>(pg_smem);
    if (d.quads_same_plane) {
        for (uint32_t idx = threadIdx.x; idx < (d.HW >> 2); idx += 256u)
            quad_of[idx] = quad_table_entry(idx, d.HW, d.W, d.Wb, d.TPP, d.by_hw, d.by_w, d.by_b);
    } else {
        for (uint32_t idx = threadIdx.x; idx < d.HW; idx += 256u) {
            const uint32_t h = fdiv(idx, d.by_w), w = idx - h * d.W;
            tile_of[idx] = (uint16_t)(fdiv(h, d.by_b) * d.Wb + fdiv(w, d.by_b));
        }
    }
    __syncthreads();
    const uint64_t cta_e0 = (uint64_t)blockIdx.x * (1024u * QPT);           // first element of this CTA
    const uint64_t cta_plane0 = cta_e0 / d.HW;
    const uint32_t cta_rem0 = (uint32_t)(cta_e0 - cta_plane0 * d.HW);
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t lq = threadIdx.x + (uint32_t)k * 256u;               // quad inside the CTA
        const uint64_t gq = (uint64_t)blockIdx.x * (256u * QPT) + lq;
        if (gq < d.quads) {
            const uint32_t bits = quad_bits<Q>(packed, gq);
            const uint32_t loc = cta_rem0 + 4u * lq;                         // < HW + 4096 * QPT
            const uint32_t dp = fdiv(loc, d.by_hw);
            uint32_t rem = loc - dp * d.HW;
            uint64_t plane = cta_plane0 + dp;
            float v[4];
            if (d.quads_same_plane) {
                float delta, step;
                pg_unpack_stats(__ldg(stats + plane), delta, step);
                const uint2 ent = quad_of[rem >> 2];
                const LT* lp = lfc + plane * d.TPP;
                v[0] = reconstruct(bits & MASK, step, delta, Elem<LT>::load(lp + (ent.x & 0xFFFFu)));
                v[1] = reconstruct((bits >> Q) & MASK, step, delta, Elem<LT>::load(lp + (ent.x >> 16)));
                v[2] = reconstruct((bits >> (2 * Q)) & MASK, step, delta, Elem<LT>::load(lp + (ent.y & 0xFFFFu)));
                v[3] = reconstruct((bits >> (3 * Q)) & MASK, step, delta, Elem<LT>::load(lp + (ent.y >> 16)));
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float delta, step;
                    pg_unpack_stats(__ldg(stats + plane), delta, step);
                    const float l = Elem<LT>::load(lfc + plane * d.TPP + tile_of[rem]);
                    v[i] = reconstruct((bits >> (i * Q)) & MASK, step, delta, l);
                    if (++rem == d.HW) {
                        rem = 0;
                        ++plane;
                    }
                }
            }
            Quad<XT>::store(xhat + gq * 4u, v[0], v[1], v[2], v[3]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct PgPlan {
    uint32_t spb, spp, G;
    uint32_t threads;
    int32_t grid;
};

inline bool plan_pg_strip(const div_desc* d, const Shape& s, PgPlan* out) {
    if (s.W % 4 != 0) return false;
    if (!(s.B == 4 || s.B == 8) || s.P2 != s.B) return false;
    if (!(d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return false;
    const uint64_t planes = (uint64_t)s.N * s.C;
    if (planes >= (1ull << 31)) return false;
    PgPlan pl = PgPlan();
    pl.spb = s.Wb * (s.P2 / 4);
    const uint64_t spp = (uint64_t)s.Hb * pl.spb;
    if (spp > PG_CAP) return false;
    pl.spp = (uint32_t)spp;
    // CTAs of about DIVK_PG_SMALL_CTA threads (twice that for medium planes), so that several CTAs share an SM
    // and their load and compute phases interleave (measured on the 64-sample ResNet-50 maps: 56 x 56 planes
    // 64 -> 56 us, 28 x 28 planes 41 -> 33 us).  A larger plane takes one CTA of its own; splitting it over a
    // thread-block cluster of 2 or 4 smaller CTAs that exchange their extremes through distributed shared
    // memory was measured slower (70 and 78 us against 66 us on the 112 x 112 planes).
    uint32_t cap = PG_MAX_THREADS;
    if (pl.spp <= DIVK_PG_SMALL_CTA / 2u) cap = DIVK_PG_SMALL_CTA;
    else if (pl.spp <= 2u * DIVK_PG_SMALL_CTA) cap = 2u * DIVK_PG_SMALL_CTA;
    uint64_t G = cap / pl.spp;
    if (G > planes) G = planes;
    pl.G = (uint32_t)G;
    pl.threads = ((pl.G * pl.spp + 31u) / 32u) * 32u;
    pl.grid = (int32_t)((planes + G - 1) / G);
    *out = pl;
    return true;
}

template <typename XT, typename LT>
inline div_status launch_pg_strip(int qbits, uint32_t p2, const PgParams& prm, const PgPlan& pl, cudaStream_t st) {
#define DIVK_PG_CASE(QQ, PP) \
    if (qbits == QQ && p2 == PP) { pg_strip_kernel<XT, LT, QQ, PP><<<pl.grid, pl.threads, 0, st>>>(prm); return DIV_OK; }
    DIVK_PG_CASE(2, 8)
    DIVK_PG_CASE(4, 8)
    DIVK_PG_CASE(8, 8)
    DIVK_PG_CASE(2, 4)
    DIVK_PG_CASE(4, 4)
    DIVK_PG_CASE(8, 4)
#undef DIVK_PG_CASE
    return DIV_ERR_PARAM;
}

inline div_status compress_pg_strip(const div_desc* d, const Shape& s, const div_layout& lo, const PgPlan& pl,
                                    const void* x, uint8_t* blob, uint64_t seed, cudaStream_t st) {
    PgParams prm;
    prm.s = s;
    prm.x = x;
    prm.lfc = blob + lo.lfc_off;
    prm.packed = blob + lo.packed_off;
    prm.stats = reinterpret_cast<uint32_t*>(blob + lo.stats_off);
    prm.seed = seed;
    prm.rng_row_step = K_GROUP * (uint64_t)(s.W / 4u);
    prm.planes = s.N * s.C;
    prm.spb = pl.spb;
    prm.spp = pl.spp;
    prm.G = pl.G;
    prm.tail_rows = s.H - (s.Hb - 1u) * s.B;
    prm.by_spp = host_fastdiv(pl.spp);
    prm.by_spb = host_fastdiv(pl.spb);
    prm.by_c = host_fastdiv(s.C);
    const uint32_t tail_cols = s.W - (s.Wb - 1u) * s.B;
    for (int i = 0; i < 4; ++i) {
        const uint32_t rows = (i & 2) ? prm.tail_rows : s.B, cols = (i & 1) ? tail_cols : s.B;
        const uint32_t cnt = rows * cols;
        prm.cnt[i] = (float)cnt;
        prm.inv_cnt[i] = (cnt & (cnt - 1)) == 0 ? 1.0f / (float)cnt : 0.f;      // exact for a power of two
    }
    typedef __nv_bfloat16 bf16;
    div_status r;
    if (d->x_dtype == DIV_F32)
        r = d->lfc_dtype == DIV_F32 ? launch_pg_strip<float, float>(d->qbits, s.P2, prm, pl, st)
                                    : launch_pg_strip<float, bf16>(d->qbits, s.P2, prm, pl, st);
    else
        r = d->lfc_dtype == DIV_F32 ? launch_pg_strip<bf16, float>(d->qbits, s.P2, prm, pl, st)
                                    : launch_pg_strip<bf16, bf16>(d->qbits, s.P2, prm, pl, st);
    if (r != DIV_OK) return r;
    return cudaGetLastError() == cudaSuccess ? DIV_OK : DIV_ERR_CUDA;
}

inline bool plan_pg_small(const div_desc* d, const Shape& s, PgSmall* out) {
    if (!(d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return false;
    if (!(s.P2 == 4 || s.P2 == 8 || s.P2 == 16)) return false;
    if (s.Wb * s.P2 > 32u) return false;
    if (s.CHW % 4 != 0 || s.HW > FLAT_MAX_HW) return false;
    const uint64_t planes = (uint64_t)s.N * s.C;
    if (planes >= (1ull << 31)) return false;
    PgSmall g;
    g.s = s;
    g.planes = (uint32_t)planes;
    g.cpl = (s.W % 2 == 0 && s.B % 2 == 0) ? 2u : 3u;
    g.quads_same_plane = (s.HW % 4 == 0) ? 1u : 0u;
    g.lanes_per_plane = s.Wb * s.P2 / 2u;
    g.planes_per_warp = 32u / g.lanes_per_plane;
    // planes per CTA: whole passes of the 8 warps (a multiple of 8, so G * HW is a multiple of 4), about 8192
    // elements, bounded so that the per-plane arrays stay small
    const uint32_t unit = 8u * g.planes_per_warp;
    uint32_t m = 8192u / (unit * s.HW);
    if (m < 1u) m = 1u;
    while (m > 1u && (unit * m > 1024u || unit * m * s.TPP > 2048u)) --m;
    g.G = unit * m;
    if (g.G > 1024u || g.G * s.TPP > 4096u) return false;
    g.table_words = flat_table_words(s.HW);
    g.by_hw = host_fastdiv(s.HW);
    g.by_w = host_fastdiv(s.W);
    g.by_b = host_fastdiv(s.B);
    g.by_c = host_fastdiv(s.C);
    if (pg_small_smem_bytes(g) > 46000) return false;
    *out = g;
    return true;
}

template <typename XT, typename LT>
inline div_status launch_pg_small(int qbits, uint32_t p2, const PgSmall& g, cudaStream_t st) {
    const uint32_t grid = (g.planes + g.G - 1) / g.G;
    const size_t smem = pg_small_smem_bytes(g);
#define DIVK_PGS_CASE(QQ, PP) \
    if (qbits == QQ && p2 == PP) {                                                      \
        if (g.cpl == 2) pg_small_kernel<XT, LT, QQ, PP, 2><<<grid, 256, smem, st>>>(g); \
        else pg_small_kernel<XT, LT, QQ, PP, 3><<<grid, 256, smem, st>>>(g);            \
        return DIV_OK;                                                                  \
    }
    DIVK_PGS_CASE(2, 4)
    DIVK_PGS_CASE(4, 4)
    DIVK_PGS_CASE(8, 4)
    DIVK_PGS_CASE(2, 8)
    DIVK_PGS_CASE(4, 8)
    DIVK_PGS_CASE(8, 8)
    DIVK_PGS_CASE(2, 16)
    DIVK_PGS_CASE(4, 16)
    DIVK_PGS_CASE(8, 16)
#undef DIVK_PGS_CASE
    return DIV_ERR_PARAM;
}

inline div_status compress_pg_small(const div_desc* d, const Shape& s, const div_layout& lo, PgSmall g,
                                    const void* x, uint8_t* blob, uint64_t seed, cudaStream_t st) {
    g.x = x;
    g.lfc = blob + lo.lfc_off;
    g.packed = blob + lo.packed_off;
    g.stats = reinterpret_cast<uint32_t*>(blob + lo.stats_off);
    g.seed = seed;
    typedef __nv_bfloat16 bf16;
    div_status r;
    if (d->x_dtype == DIV_F32)
        r = d->lfc_dtype == DIV_F32 ? launch_pg_small<float, float>(d->qbits, s.P2, g, st)
                                    : launch_pg_small<float, bf16>(d->qbits, s.P2, g, st);
    else
        r = d->lfc_dtype == DIV_F32 ? launch_pg_small<bf16, float>(d->qbits, s.P2, g, st)
                                    : launch_pg_small<bf16, bf16>(d->qbits, s.P2, g, st);
    if (r != DIV_OK) return r;
    return cudaGetLastError() == cudaSuccess ? DIV_OK : DIV_ERR_CUDA;
}

}  // namespace divk
