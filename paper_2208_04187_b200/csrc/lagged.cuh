// Lagged single-launch compress kernel (DIVISION Sec. 4.1; Algorithm 1, forward loop) for the common
// CNN shapes: W % 4 == 0, B in {4, 8}, Q in {2, 4, 8}.
//
// The per-sample (delta, scale) of Eq. 9 depend on every residual of the sample, so each element is
// needed twice: once for the block means and the residual extremes ("reduce"), once for the codes
// ("quantise").  This kernel reads x from HBM once and takes the second read from L2: the warps of the
// grid sweep the tensor together in units, and a warp that has reduced unit j goes on to quantise unit
// j - D.  The span of D units (a few tens of MB, kept in L2 by a residency hint on the first read) is
// still in the 126 MB L2 when it is read again, and by then its sample has been completed by the other
// warps, so that in the steady state nothing waits on the grid-wide dependency.
//
//   * a STRIP is 4 adjacent columns of one tile row band (4 x B elements).  A lane owns the strips at
//     one column position in J consecutive bands: per band B 16-byte global loads, column sums in
//     registers, one shuffle to meet the other half of a B = 8 tile.  A UNIT is 32 such lanes; the
//     set-up arithmetic of a lane is paid once per J bands, and from one band to the next every index
//     advances by a constant.
//   * warps are independent: each claims the next unit from a counter in global scratch (one atomic
//     per unit), reduces it at once, folds its residual extremes into the sample's slot
//     in global scratch and counts the unit as arrived; the arrival that completes a sample derives
//     (delta, Delta, scale), writes the first two to the blob and publishes all of it in the slot.
//   * the quantise half reads the slot (bounded wait; normally the first look succeeds), re-reads the
//     stored low-frequency values and x, and emits the 4 codes of each strip row as one byte (Q = 2),
//     half-word (Q = 4) or word (Q = 8): lanes of a warp write consecutive bytes.  Its fp32 arithmetic
//     runs on packed pairs (.f32x2: two IEEE results per instruction, same roundings as scalar code).
//
// The launch is cooperative so that all CTAs are resident (a warp that waits for a sample needs the
// warps that hold the sample's other units to be running); no grid-wide barrier is used.  Every wait is
// bounded: when a limit runs out the kernel records DIV_ERR_TIMEOUT in the workspace status word, stops
// waiting everywhere and finishes without the quantise halves that could not start.
#pragma once

#include "fused_v.cuh"

namespace divk {

#ifndef DIVK_L_WARPS
#define DIVK_L_WARPS 8
#endif
#ifndef DIVK_L_MIN_CTAS
#define DIVK_L_MIN_CTAS 2
#endif
#ifndef DIVK_L_LAG_BYTES
#define DIVK_L_LAG_BYTES (16u << 20)
#endif
#ifndef DIVK_L_BANDS
#define DIVK_L_BANDS 4
#endif
constexpr int L_WARPS = DIVK_L_WARPS;
constexpr int L_THREADS = 32 * L_WARPS;

// workspace words used by this kernel (see common.cuh): header word 2 = unit claim counter; per-sample
// slot: 0 ~key(min), 1 key(max), 2 units arrived, 3 ready flag, 4 delta bits, 5 scale bits
constexpr int WS_CLAIM_WORD = 2;

struct LPlan {
    int32_t grid, threads, ctas_per_sm;
    uint32_t spb;                 // strip slots per band
    uint32_t bands;               // C * Hb bands per sample
    uint32_t bands_per_lane;      // J
    uint32_t slots_per_sample;    // ceil(bands / J) * spb
    uint32_t units_per_sample;    // ceil(slots_per_sample / 32)
    uint32_t lag_units;           // D
    uint64_t total_units;
};

struct LParams {
    Shape s;
    LPlan pl;
    FastDiv by_US, by_spb, by_hb;
    const void* x;
    void* lfc;
    void* packed;
    float* stats;
    uint32_t* ws;
    uint64_t seed;
    uint64_t rng_row_step;        // K_GROUP * (W / 4): counter step of the random stream between rows
    uint64_t timeout_ns;
    uint32_t expected_units;      // units per sample (a test may ask for an unreachable count)
    uint32_t tail_rows;           // rows of the last band of a plane
    float inv_cnt[4];             // 1 / (rows * cols) for [tail row band][tail column tile] when it is a power of two, else 0
    float cnt[4];                 // rows * cols for the same four cases
};

// L2 residency hints: the first read of x asks L2 to keep the line (it comes back soon), the second read
// releases it
__device__ __forceinline__ uint64_t l2_policy_keep() {
    uint64_t pol;
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_release() {
    uint64_t pol;
    asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint32_t atom_add_release(uint32_t* p, uint32_t v) {
    uint32_t old;
    asm volatile("atom.release.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
// a strip row from global memory as two packed pairs (x, y) and (z, w), widened to fp32
template <typename XT> struct GlobalRow2;
template <> struct GlobalRow2<float> {
    static __device__ __forceinline__ void load(const unsigned char* ptr, uint64_t pol, uint64_t& xy, uint64_t& zw) {
        asm("ld.global.L2::cache_hint.v2.u64 {%0, %1}, [%2], %3;" : "=l"(xy), "=l"(zw) : "l"(ptr), "l"(pol));
    }
};
template <> struct GlobalRow2<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const unsigned char* ptr, uint64_t pol, uint64_t& xy, uint64_t& zw) {
        uint32_t a, b;
        asm("ld.global.L2::cache_hint.v2.u32 {%0, %1}, [%2], %3;" : "=r"(a), "=r"(b) : "l"(ptr), "l"(pol));
        xy = pk2u(a << 16, a & 0xFFFF0000u);
        zw = pk2u(b << 16, b & 0xFFFF0000u);
    }
};

// where lane `lane` of unit `uu` starts inside its sample
struct LStart {
    uint32_t e;        // in-sample index of the first element of its first strip
    uint32_t ts;       // tile index (inside the sample) of its first strip
    uint32_t bh;       // band row of its first band inside the plane
    uint32_t nb;       // bands it owns (0: the slot is padding)
    uint32_t q;        // slot inside the band
};
template <int P2>
__device__ __forceinline__ LStart l_start(const LParams& p, uint32_t uu, uint32_t lane) {
    constexpr uint32_t LPT = P2 / 4;
    const Shape& s = p.s;
    LStart t;
    const uint32_t sl = uu * 32u + lane;
    const bool valid = sl < p.pl.slots_per_sample;
    const uint32_t slc = valid ? sl : 0u;
    const uint32_t grp = fdiv(slc, p.by_spb);
    t.q = slc - grp * p.pl.spb;
    const uint32_t band0 = grp * p.pl.bands_per_lane;
    const uint32_t plane = fdiv(band0, p.by_hb);
    t.bh = band0 - plane * s.Hb;
    const uint32_t col0 = 4u * t.q;
    const bool ok = valid && col0 < s.W;
    t.nb = ok ? min(p.pl.bands_per_lane, p.pl.bands - band0) : 0u;
    t.e = plane * s.HW + t.bh * s.B * s.W + (ok ? col0 : 0u);
    t.ts = plane * s.TPP + t.bh * s.Wb + t.q / LPT;
    return t;
}

// the B rows of one full band of a strip
template <typename XT, int P2>
__device__ __forceinline__ void l_load_band(const unsigned char* xs, uint32_t row_bytes, uint64_t pol,
                                            uint64_t (&vxy)[P2], uint64_t (&vzw)[P2]) {
#pragma unroll
    for (int r = 0; r < P2; ++r) GlobalRow2<XT>::load(xs + r * row_bytes, pol, vxy[r], vzw[r]);
}

// reduce half of one full band (all B rows in bounds): tile mean in the fixed order, stored low-frequency
// value, extremes of the residual folded into (lo, hi)
template <typename LT, int P2>
__device__ __forceinline__ void l_reduce_full_band(const uint64_t (&vxy)[P2], const uint64_t (&vzw)[P2], float inv,
                                                   float cnt, bool writer, bool live, LT* lfc_n, float& lo, float& hi) {
    constexpr uint32_t LPT = P2 / 4;
    uint64_t cxy[P2], czw[P2];
#pragma unroll
    for (int r = 0; r < P2; ++r) {
        cxy[r] = vxy[r];
        czw[r] = vzw[r];
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
    const float mean = (inv != 0.f) ? __fmul_rn(sum, inv) : __fdiv_rn(sum, cnt);
    const float stored = Elem<LT>::round(mean);
    if (live) {
        if (writer) Elem<LT>::store(lfc_n, mean);
        float blo = 3.402823466e+38f, bhi = -3.402823466e+38f;
#pragma unroll
        for (int r = 0; r < P2; ++r) {
            float a_, b_, c_, d_;
            upk2(vxy[r], a_, b_);
            upk2(vzw[r], c_, d_);
            blo = fmin3(blo, a_, b_);
            blo = fmin3(blo, c_, d_);
            bhi = fmax3(bhi, a_, b_);
            bhi = fmax3(bhi, c_, d_);
        }
        lo = fminf(lo, __fsub_rn(blo, stored));
        hi = fmaxf(hi, __fsub_rn(bhi, stored));
    }
}

// quantise half of one full band: B rows of 4 codes each
template <typename OutT, int Q, int P2>
__device__ __forceinline__ void l_quant_full_band(const uint64_t (&vxy)[P2], const uint64_t (&vzw)[P2], float stored,
                                                  uint64_t delta2, uint64_t scale2, uint64_t& ctr, uint64_t row_step,
                                                  OutT*& out, uint32_t W4) {
    const uint64_t stored2 = pk2(stored, stored);
#pragma unroll
    for (int r = 0; r < P2; ++r) {
        *out = (OutT)quant_row<Q>(vxy[r], vzw[r], stored2, delta2, scale2, rng_mix(ctr));
        out += W4;
        ctr += row_step;
    }
}

template <typename XT, typename LT, int Q, int P2>
__global__ void __launch_bounds__(L_THREADS, DIVK_L_MIN_CTAS)
lagged_kernel(const LParams p) {
    constexpr uint32_t LPT = P2 / 4;
    typedef typename PackedUnit<Q>::type OutT;

    const Shape& s = p.s;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t US = p.pl.units_per_sample;
    const uint32_t TU = (uint32_t)p.pl.total_units;        // < 2^30 (checked by the planner)
    const uint32_t D = p.pl.lag_units;
    const uint32_t J = p.pl.bands_per_lane;
    const uint32_t row_bytes = s.W * (uint32_t)sizeof(XT);
    const uint32_t W4 = s.W >> 2;
    const uint64_t pol_keep = l2_policy_keep(), pol_release = l2_policy_release();
    const XT* x = reinterpret_cast<const XT*>(p.x);
    LT* lfc_out = reinterpret_cast<LT*>(p.lfc);
    OutT* packed = reinterpret_cast<OutT*>(p.packed);
    uint32_t* claim_word = p.ws + WS_CLAIM_WORD;

    bool gave_up = false;
    uint32_t next = 0;
    if (lane == 0) next = atomicAdd(claim_word, 1u);

    while (true) {
        const uint32_t j = __shfl_sync(0xFFFFFFFFu, next, 0);
        if (j >= TU + D) break;

        // ================= reduce half: unit j =================
        if (j < TU) {
            const uint32_t n = fdiv(j, p.by_US);
            const LStart t = l_start<P2>(p, j - n * US, lane);
            const unsigned char* xs = reinterpret_cast<const unsigned char*>(x + ((size_t)n * s.CHW + t.e));
            LT* lfc_n = lfc_out + (size_t)n * s.C * s.TPP + t.ts;
            const uint32_t tail_col = (t.q / LPT == s.Wb - 1u && (s.W % s.B) != 0u) ? 1u : 0u;
            const bool writer = (t.q % LPT) == 0;
            const bool all_full = __all_sync(0xFFFFFFFFu, t.nb == J) && (p.tail_rows == s.B);
            uint32_t bh = t.bh;
            float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
            if (all_full && J == 4u) {
                // four full bands for every lane: two register buffers, the loads of a band are issued
                // before the band in the other buffer is worked on
                const uint32_t band_bytes = s.B * row_bytes;
                const float inv = p.inv_cnt[tail_col], cnt = p.cnt[tail_col];
                uint64_t axy[P2], azw[P2], bxy[P2], bzw[P2];
                l_load_band<XT, P2>(xs, row_bytes, pol_keep, axy, azw);
                l_load_band<XT, P2>(xs + band_bytes, row_bytes, pol_keep, bxy, bzw);
                l_reduce_full_band<LT, P2>(axy, azw, inv, cnt, writer, true, lfc_n, lo, hi);
                l_load_band<XT, P2>(xs + 2u * band_bytes, row_bytes, pol_keep, axy, azw);
                l_reduce_full_band<LT, P2>(bxy, bzw, inv, cnt, writer, true, lfc_n + s.Wb, lo, hi);
                l_load_band<XT, P2>(xs + 3u * band_bytes, row_bytes, pol_keep, bxy, bzw);
                l_reduce_full_band<LT, P2>(axy, azw, inv, cnt, writer, true, lfc_n + 2u * s.Wb, lo, hi);
                l_reduce_full_band<LT, P2>(bxy, bzw, inv, cnt, writer, true, lfc_n + 3u * s.Wb, lo, hi);
            } else
            for (uint32_t jb = 0; jb < J; ++jb) {
                const uint32_t rows = (jb < t.nb) ? ((bh + 1u == s.Hb) ? p.tail_rows : s.B) : 0u;
                uint64_t vxy[P2], vzw[P2];
                if (all_full) {
#pragma unroll
                    for (int r = 0; r < P2; ++r) GlobalRow2<XT>::load(xs + r * row_bytes, pol_keep, vxy[r], vzw[r]);
                } else {
#pragma unroll
                    for (int r = 0; r < P2; ++r) {
                        if ((uint32_t)r < rows) {
                            GlobalRow2<XT>::load(xs + r * row_bytes, pol_keep, vxy[r], vzw[r]);
                        } else {
                            vxy[r] = 0ull;
                            vzw[r] = 0ull;
                        }
                    }
                }
                // column sums: balanced tree down the rows of each of the 4 columns
                uint64_t cxy[P2], czw[P2];
#pragma unroll
                for (int r = 0; r < P2; ++r) {
                    cxy[r] = vxy[r];
                    czw[r] = vzw[r];
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
                const uint32_t which = ((rows != s.B) ? 2u : 0u) + tail_col;
                const float inv = p.inv_cnt[which];
                const float mean = (inv != 0.f) ? __fmul_rn(sum, inv) : __fdiv_rn(sum, p.cnt[which]);
                const float stored = Elem<LT>::round(mean);
                if (rows != 0u) {
                    if (writer) Elem<LT>::store(lfc_n, mean);
                    // extremes of x over the strip's in-bounds rows; x -> fl(x - stored) is monotone
                    float blo = 3.402823466e+38f, bhi = -3.402823466e+38f;
#pragma unroll
                    for (int r = 0; r < P2; ++r) {
                        if (all_full || (uint32_t)r < rows) {
                            float a_, b_, c_, d_;
                            upk2(vxy[r], a_, b_);
                            upk2(vzw[r], c_, d_);
                            blo = fmin3(blo, a_, b_);
                            blo = fmin3(blo, c_, d_);
                            bhi = fmax3(bhi, a_, b_);
                            bhi = fmax3(bhi, c_, d_);
                        }
                    }
                    lo = fminf(lo, __fsub_rn(blo, stored));
                    hi = fmaxf(hi, __fsub_rn(bhi, stored));
                }
                xs += rows * row_bytes;
                lfc_n += s.Wb;
                bh = (bh + 1u == s.Hb) ? 0u : bh + 1u;
            }
            const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
            const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
            // bar.warp.sync orders the other lanes' stores of low-frequency values before lane 0's release below
            __syncwarp();
            if (lane == 0) {
                uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
                red_max_relaxed(slot + 0, kmin);
                red_max_relaxed(slot + 1, kmax);
                const uint32_t before = atom_add_release(slot + 2, 1u);
                if (before + 1u == p.expected_units) {
                    // this arrival completes the sample
                    fence_acq_rel_gpu();
                    const QParams qp = make_qparams(key_float(~ld_relaxed_u32(slot + 0)), key_float(ld_relaxed_u32(slot + 1)), Q);
                    p.stats[2 * (size_t)n + 0] = qp.delta;
                    p.stats[2 * (size_t)n + 1] = qp.step;
                    slot[4] = __float_as_uint(qp.delta);
                    slot[5] = __float_as_uint(qp.scale);
                    __threadfence();
                    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(slot + 3), "r"(1u) : "memory");
                }
            }
        }

        // ================= quantise half: unit j - D =================
        if (j >= D) {
            const uint32_t jq = j - D;
            const uint32_t n = fdiv(jq, p.by_US);
            const uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
            uint32_t ready = 0, dbits = 0, sbits = 0;
            if (lane == 0 && !gave_up) {
                uint32_t polls = 0;
                uint64_t t0 = 0;
                while (true) {
                    ready = ld_acquire_u32(slot + 3);
                    if (ready) break;
                    if ((++polls & 7u) == 0) {
                        const uint64_t tn = now_ns();
                        if (t0 == 0) t0 = tn;
                        if (ld_relaxed_u32(p.ws) != 0u || tn - t0 > p.timeout_ns) {
                            atomicCAS(p.ws, 0u, (uint32_t)DIV_ERR_TIMEOUT);
                            atomicCAS(p.ws + 1, 0u, n + 1u);
                            break;
                        }
                    }
                    __nanosleep(200);
                }
                if (ready) {
                    dbits = ld_relaxed_u32(slot + 4);
                    sbits = ld_relaxed_u32(slot + 5);
                }
            }
            ready = __shfl_sync(0xFFFFFFFFu, ready, 0);
            dbits = __shfl_sync(0xFFFFFFFFu, dbits, 0);
            sbits = __shfl_sync(0xFFFFFFFFu, sbits, 0);
            __syncwarp();
            if (!ready) {
                gave_up = true;
            } else {
                const LStart t = l_start<P2>(p, jq - n * US, lane);
                if (t.nb != 0u) {
                    const unsigned char* xs = reinterpret_cast<const unsigned char*>(x + ((size_t)n * s.CHW + t.e));
                    // the low-frequency map was written by other warps: read it past the (incoherent) L1
                    const LT* lfc_n = lfc_out + (size_t)n * s.C * s.TPP + t.ts;
                    const uint64_t delta2 = pk2u(dbits, dbits), scale2 = pk2u(sbits, sbits);
                    const uint32_t g0 = t.e >> 2;
                    uint64_t ctr = rng_sample_base(p.seed, n) + K_GROUP * (uint64_t)(g0 + 1u);
                    OutT* out = packed + (((uint64_t)n * s.CHW) >> 2) + g0;
                    uint32_t bh = t.bh;
                    if (t.nb == 4u && p.tail_rows == s.B) {
                        const uint32_t band_bytes = s.B * row_bytes;
                        const float st0 = Elem<LT>::load_cg(lfc_n), st1 = Elem<LT>::load_cg(lfc_n + s.Wb);
                        const float st2 = Elem<LT>::load_cg(lfc_n + 2u * s.Wb), st3 = Elem<LT>::load_cg(lfc_n + 3u * s.Wb);
                        uint64_t axy[P2], azw[P2], bxy[P2], bzw[P2];
                        l_load_band<XT, P2>(xs, row_bytes, pol_release, axy, azw);
                        l_load_band<XT, P2>(xs + band_bytes, row_bytes, pol_release, bxy, bzw);
                        l_quant_full_band<OutT, Q, P2>(axy, azw, st0, delta2, scale2, ctr, p.rng_row_step, out, W4);
                        l_load_band<XT, P2>(xs + 2u * band_bytes, row_bytes, pol_release, axy, azw);
                        l_quant_full_band<OutT, Q, P2>(bxy, bzw, st1, delta2, scale2, ctr, p.rng_row_step, out, W4);
                        l_load_band<XT, P2>(xs + 3u * band_bytes, row_bytes, pol_release, bxy, bzw);
                        l_quant_full_band<OutT, Q, P2>(axy, azw, st2, delta2, scale2, ctr, p.rng_row_step, out, W4);
                        l_quant_full_band<OutT, Q, P2>(bxy, bzw, st3, delta2, scale2, ctr, p.rng_row_step, out, W4);
                    } else
                    for (uint32_t jb = 0; jb < t.nb; ++jb) {
                        const uint32_t rows = (bh + 1u == s.Hb) ? p.tail_rows : s.B;
                        const float stored = Elem<LT>::load_cg(lfc_n);
                        const uint64_t stored2 = pk2(stored, stored);
                        if (rows == (uint32_t)P2) {
                            uint64_t vxy[P2], vzw[P2];
#pragma unroll
                            for (int r = 0; r < P2; ++r) {
                                GlobalRow2<XT>::load(xs, pol_release, vxy[r], vzw[r]);
                                xs += row_bytes;
                            }
#pragma unroll
                            for (int r = 0; r < P2; ++r) {
                                *out = (OutT)quant_row<Q>(vxy[r], vzw[r], stored2, delta2, scale2, rng_mix(ctr));
                                out += W4;
                                ctr += p.rng_row_step;
                            }
                        } else {
                            for (uint32_t r = 0; r < rows; ++r) {
                                uint64_t xy, zw;
                                GlobalRow2<XT>::load(xs, pol_release, xy, zw);
                                xs += row_bytes;
                                *out = (OutT)quant_row<Q>(xy, zw, stored2, delta2, scale2, rng_mix(ctr));
                                out += W4;
                                ctr += p.rng_row_step;
                            }
                        }
                        lfc_n += s.Wb;
                        bh = (bh + 1u == s.Hb) ? 0u : bh + 1u;
                    }
                }
            }
        }
        // claim the next unit only now: a claimed unit that waits behind this warp's quantise half would
        // hold back its whole sample
        if (lane == 0) next = atomicAdd(claim_word, 1u);
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
template <typename XT, typename LT, int Q, int P2>
inline div_status l_occupancy(int dev, int* ctas_per_sm) {
    // resident CTAs per SM of this instance: asked once per device
    static SmemSeen cached[DEVICE_CACHE_SLOTS];          // .bytes holds the count
    const void* kern = (const void*)lagged_kernel<XT, LT, Q, P2>;
    const bool slot = dev >= 0 && dev < DEVICE_CACHE_SLOTS;
    if (slot && cached[dev].fn.load(std::memory_order_acquire) == kern) {
        const int c = cached[dev].bytes.load(std::memory_order_acquire);
        if (c > 0) {
            *ctas_per_sm = c;
            return DIV_OK;
        }
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, lagged_kernel<XT, LT, Q, P2>, L_THREADS, 0) != cudaSuccess) {
        cudaGetLastError();
        return DIV_ERR_CUDA;
    }
    if (slot && *ctas_per_sm > 0) {
        cached[dev].fn.store(nullptr, std::memory_order_release);
        cached[dev].bytes.store(*ctas_per_sm, std::memory_order_release);
        cached[dev].fn.store(kern, std::memory_order_release);
    }
    return DIV_OK;
}

template <typename XT, typename LT>
inline div_status l_occupancy_q(int dev, int qbits, uint32_t p2, int* out) {
    if (p2 == 8) {
        if (qbits == 2) return l_occupancy<XT, LT, 2, 8>(dev, out);
        if (qbits == 4) return l_occupancy<XT, LT, 4, 8>(dev, out);
        if (qbits == 8) return l_occupancy<XT, LT, 8, 8>(dev, out);
    } else if (p2 == 4) {
        if (qbits == 2) return l_occupancy<XT, LT, 2, 4>(dev, out);
        if (qbits == 4) return l_occupancy<XT, LT, 4, 4>(dev, out);
        if (qbits == 8) return l_occupancy<XT, LT, 8, 4>(dev, out);
    }
    return DIV_ERR_PARAM;
}

inline div_status plan_lagged(const div_desc* d, const Shape& s, LPlan* out) {
    typedef __nv_bfloat16 bf16;
    const uint32_t sx = d->x_dtype == DIV_F32 ? 4u : 2u;
    if (s.W % 4 != 0) return DIV_ERR_PARAM;
    if (!(s.B == 4 || s.B == 8) || s.P2 != s.B) return DIV_ERR_PARAM;
    if (!(d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return DIV_ERR_PARAM;
    // packed stores of whole bytes / half-words / words per strip row need the sample to start on one
    if (s.CHW % 4 != 0) return DIV_ERR_PARAM;
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return DIV_ERR_CUDA;

    LPlan pl = LPlan();
    pl.spb = s.Wb * (s.P2 / 4);
    const uint64_t bands = (uint64_t)s.C * s.Hb;
    if (bands >= (1ull << 31)) return DIV_ERR_PARAM;
    pl.bands = (uint32_t)bands;
    // bands per lane: DIVK_L_BANDS, fewer while a sample would not fill a couple of units
    uint32_t J = DIVK_L_BANDS;
    while (J > 1 && ((bands + J - 1) / J) * pl.spb < 64) J >>= 1;
    pl.bands_per_lane = J;
    const uint64_t slots = ((bands + J - 1) / J) * pl.spb;
    if (slots >= (1ull << 31)) return DIV_ERR_PARAM;
    pl.slots_per_sample = (uint32_t)slots;
    pl.units_per_sample = (pl.slots_per_sample + 31u) / 32u;
    pl.total_units = (uint64_t)pl.units_per_sample * s.N;
    pl.threads = L_THREADS;
    int cps = 0;
    div_status st;
    if (d->x_dtype == DIV_F32)
        st = d->lfc_dtype == DIV_F32 ? l_occupancy_q<float, float>(di.dev, d->qbits, s.P2, &cps) : l_occupancy_q<float, bf16>(di.dev, d->qbits, s.P2, &cps);
    else
        st = d->lfc_dtype == DIV_F32 ? l_occupancy_q<bf16, float>(di.dev, d->qbits, s.P2, &cps) : l_occupancy_q<bf16, bf16>(di.dev, d->qbits, s.P2, &cps);
    if (st != DIV_OK) return st;
    if (cps < 1) return DIV_ERR_CUDA;
    pl.ctas_per_sm = cps;
    uint64_t grid = (uint64_t)di.sms * (uint64_t)cps;
    const uint64_t want = (pl.total_units + L_WARPS - 1) / L_WARPS;
    if (grid > want) grid = want;
    pl.grid = (int32_t)grid;
    // lag: at least a whole sample (so that every unit of the sample has been claimed, hence is being
    // reduced by a running warp, when its first unit comes up for quantising), and about
    // DIVK_L_LAG_BYTES of x, which the L2 still holds
    const uint64_t unit_bytes = 32ull * J * s.B * 4ull * sx;
    uint64_t lag = (DIVK_L_LAG_BYTES + unit_bytes - 1) / unit_bytes;
    if (lag > pl.total_units) lag = pl.total_units;      // a tensor smaller than the span: reduce everything, then quantise
    if (lag < pl.units_per_sample) lag = pl.units_per_sample;
    // unit indices and the claim counter are 32-bit on the device (every warp overshoots by one claim)
    if (pl.total_units + lag + grid * L_WARPS >= (1ull << 30)) return DIV_ERR_PARAM;
    pl.lag_units = (uint32_t)lag;
    *out = pl;
    return DIV_OK;
}

template <typename XT, typename LT, int Q, int P2>
inline div_status launch_lagged(const LParams& prm, cudaStream_t st) {
    void* args[] = {(void*)&prm};
    if (cudaLaunchCooperativeKernel((const void*)lagged_kernel<XT, LT, Q, P2>, dim3(prm.pl.grid), dim3(prm.pl.threads), args,
                                    0, st) != cudaSuccess) {
        cudaGetLastError();
        return DIV_ERR_CUDA;
    }
    return DIV_OK;
}

template <typename XT, typename LT>
inline div_status launch_lagged_q(int qbits, uint32_t p2, const LParams& prm, cudaStream_t st) {
    if (p2 == 8) {
        if (qbits == 2) return launch_lagged<XT, LT, 2, 8>(prm, st);
        if (qbits == 4) return launch_lagged<XT, LT, 4, 8>(prm, st);
        if (qbits == 8) return launch_lagged<XT, LT, 8, 8>(prm, st);
    } else if (p2 == 4) {
        if (qbits == 2) return launch_lagged<XT, LT, 2, 4>(prm, st);
        if (qbits == 4) return launch_lagged<XT, LT, 4, 4>(prm, st);
        if (qbits == 8) return launch_lagged<XT, LT, 8, 4>(prm, st);
    }
    return DIV_ERR_PARAM;
}

inline div_status compress_lagged(const div_desc* d, const Shape& s, const div_layout& lo, const LPlan& pl,
                                  const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st,
                                  uint32_t expected_units = 0, uint64_t timeout_ns = 0) {
    LParams prm;
    prm.s = s;
    prm.pl = pl;
    prm.by_US = host_fastdiv(pl.units_per_sample);
    prm.by_spb = host_fastdiv(pl.spb);
    prm.by_hb = host_fastdiv(s.Hb);
    prm.x = x;
    prm.lfc = blob + lo.lfc_off;
    prm.packed = blob + lo.packed_off;
    prm.stats = reinterpret_cast<float*>(blob + lo.stats_off);
    prm.ws = ws;
    prm.seed = seed;
    prm.rng_row_step = K_GROUP * (uint64_t)(s.W / 4u);
    prm.timeout_ns = timeout_ns ? timeout_ns : 2000000000ull;
    prm.expected_units = expected_units ? expected_units : pl.units_per_sample;
    prm.tail_rows = s.H - (s.Hb - 1u) * s.B;
    const uint32_t tail_cols = s.W - (s.Wb - 1u) * s.B;
    for (int i = 0; i < 4; ++i) {
        const uint32_t rows = (i & 2) ? prm.tail_rows : s.B, cols = (i & 1) ? tail_cols : s.B;
        const uint32_t cnt = rows * cols;
        prm.cnt[i] = (float)cnt;
        prm.inv_cnt[i] = (cnt & (cnt - 1)) == 0 ? 1.0f / (float)cnt : 0.f;      // exact for a power of two
    }
    typedef __nv_bfloat16 bf16;
    if (d->x_dtype == DIV_F32) {
        if (d->lfc_dtype == DIV_F32) return launch_lagged_q<float, float>(d->qbits, s.P2, prm, st);
        return launch_lagged_q<float, bf16>(d->qbits, s.P2, prm, st);
    }
    if (d->lfc_dtype == DIV_F32) return launch_lagged_q<bf16, float>(d->qbits, s.P2, prm, st);
    return launch_lagged_q<bf16, bf16>(d->qbits, s.P2, prm, st);
}

}  // namespace divk
