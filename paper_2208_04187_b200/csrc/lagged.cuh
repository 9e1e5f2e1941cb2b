// Lagged single-launch compress kernel (DIVISION Sec. 4.1; Algorithm 1, forward loop) for the common
// CNN shapes: W % 4 == 0, B in {4, 8}, Q in {2, 4, 8}.
//
// The per-sample (delta, scale) of Eq. 9 depend on every residual of the sample, so each element is
// needed twice: once for the block means and the residual extremes ("reduce"), once for the codes
// ("quantise").  This kernel reads x from HBM once and takes the second read from L2: all warps of the
// grid sweep the tensor together, and in every round a warp reduces one unit of the round's span and
// quantises the unit it reduced D rounds earlier.  The span of D rounds (a few tens of MB) stays
// resident in the 126 MB L2, and by the time a unit is quantised its sample has long been completed by
// the other CTAs, so that nothing waits on the grid-wide dependency in the steady state.
//
//   * a STRIP is 4 adjacent columns of one tile row band (4 x B elements), owned by one lane: B
//     16-byte global loads, column sums in registers, one shuffle to meet the other half of a B = 8
//     tile.  A UNIT is 32 consecutive strips of one sample (4 KB of fp32).
//   * round k, CTA c, warp w reduces unit (k * gridDim + c) * warps_per_cta + w: the warps of a CTA
//     take consecutive units, which lie in one sample (or straddle one boundary), so the CTA folds
//     its residual extremes in shared memory and sends one update per sample and round to the
//     sample's slot in global scratch.  The update that completes a sample derives (delta, Delta,
//     scale), writes the first two to the blob and publishes all of it in the slot.
//   * the quantise half reads the slot (bounded wait; normally the first look succeeds), re-reads the
//     stored low-frequency value and x, and emits the 4 codes of each strip row as one byte (Q = 2),
//     half-word (Q = 4) or word (Q = 8): lanes of a warp write consecutive bytes.
//
// The launch is cooperative so that all CTAs are resident (a CTA that waits for a sample needs the
// CTAs that hold the sample's other units to be running); no grid-wide barrier is used.  Every wait is
// bounded: when a limit runs out the kernel records DIV_ERR_TIMEOUT in the workspace status word, stops
// waiting everywhere and finishes its rounds without the quantise halves that could not start.
#pragma once

#include "fused_v.cuh"

namespace divk {

#ifndef DIVK_L_WARPS
#define DIVK_L_WARPS 8
#endif
#ifndef DIVK_L_MIN_CTAS
#define DIVK_L_MIN_CTAS 4
#endif
#ifndef DIVK_L_LAG_BYTES
#define DIVK_L_LAG_BYTES (12u << 20)
#endif
constexpr int L_WARPS = DIVK_L_WARPS;
constexpr int L_THREADS = 32 * L_WARPS;

// slot words used by this kernel (see common.cuh): 0 ~key(min), 1 key(max), 2 units arrived,
// 3 ready flag, 4 delta bits, 5 scale bits

struct LPlan {
    int32_t grid, threads, ctas_per_sm;
    uint32_t spb;                 // strip slots per band
    uint32_t slots_per_sample;    // C * Hb * spb
    uint32_t units_per_sample;    // ceil(slots_per_sample / 32)
    uint32_t lag_rounds;          // D
    uint32_t rounds;              // rounds of the reduce half
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
};

// geometry of the strip of lane `lane` in unit `uu` of a sample
struct LStrip {
    uint32_t e;        // in-sample index of the strip's first element
    uint32_t rows;     // in-bounds rows of its band (0: the slot is padding)
    uint32_t ts;       // tile index inside the sample
    uint32_t q;        // slot inside the band
    uint32_t bw;       // tile column
};
template <int P2>
__device__ __forceinline__ LStrip l_strip(const LParams& p, uint32_t uu, uint32_t lane) {
    constexpr uint32_t LPT = P2 / 4;
    const Shape& s = p.s;
    LStrip t;
    const uint32_t sl = uu * 32u + lane;
    const bool valid = sl < p.pl.slots_per_sample;
    const uint32_t slc = valid ? sl : 0u;
    const uint32_t bi = fdiv(slc, p.by_spb);
    t.q = slc - bi * p.pl.spb;
    const uint32_t plane = fdiv(bi, p.by_hb);
    const uint32_t bh = bi - plane * s.Hb;
    const uint32_t col0 = 4u * t.q;
    const bool ok = valid && col0 < s.W;
    t.rows = ok ? min(s.B, s.H - bh * s.B) : 0u;
    t.e = plane * s.HW + bh * s.B * s.W + (ok ? col0 : 0u);
    t.bw = t.q / LPT;
    t.ts = plane * s.TPP + bh * s.Wb + t.bw;
    return t;
}

template <typename XT, typename LT, int Q, int P2>
__global__ void __launch_bounds__(L_THREADS, DIVK_L_MIN_CTAS)
lagged_kernel(const LParams p) {
    constexpr uint32_t LPT = P2 / 4;
    typedef typename PackedUnit<Q>::type OutT;
    // CTA-level fold of the residual extremes: [round parity][first / second sample of the CTA's span]
    __shared__ uint32_t sh_kmin[2][2], sh_kmax[2][2], sh_cnt[2][2];

    const Shape& s = p.s;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t WPC = blockDim.x >> 5;
    const uint32_t G = gridDim.x;
    const uint32_t US = p.pl.units_per_sample;
    const uint64_t TU = p.pl.total_units;
    const uint32_t D = p.pl.lag_rounds;
    const uint32_t row_elems = s.W;
    const uint32_t W4 = s.W >> 2;
    const XT* x = reinterpret_cast<const XT*>(p.x);
    LT* lfc_out = reinterpret_cast<LT*>(p.lfc);
    OutT* packed = reinterpret_cast<OutT*>(p.packed);

    if (threadIdx.x < 4) {
        sh_kmin[threadIdx.x >> 1][threadIdx.x & 1] = 0;
        sh_kmax[threadIdx.x >> 1][threadIdx.x & 1] = 0;
        sh_cnt[threadIdx.x >> 1][threadIdx.x & 1] = 0;
    }
    __syncthreads();
    bool gave_up = false;

    for (uint32_t k = 0; k < p.pl.rounds + D; ++k) {
        const uint32_t par = k & 1u;
        // ================= reduce half: unit (k * G + c) * WPC + w =================
        const uint64_t a0 = ((uint64_t)k * G + blockIdx.x) * WPC;        // first unit of the CTA's span
        const uint32_t n0 = (uint32_t)(a0 / US);                          // its sample (uniform in the CTA)
        if (k < p.pl.rounds && a0 + warp < TU) {
            const uint64_t a = a0 + warp;
            uint32_t uu = (uint32_t)(a0 - (uint64_t)n0 * US) + warp;
            uint32_t n = n0;
            if (uu >= US) {
                uu -= US;
                n += 1;
            }
            (void)a;
            const LStrip t = l_strip<P2>(p, uu, lane);
            const XT* xs = x + ((size_t)n * s.CHW + t.e);
            uint64_t vxy[P2], vzw[P2];
            if (__all_sync(0xFFFFFFFFu, t.rows == (uint32_t)P2)) {
#pragma unroll
                for (int r = 0; r < P2; ++r)
                    StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(xs + r * row_elems), vxy[r], vzw[r]);
            } else {
#pragma unroll
                for (int r = 0; r < P2; ++r) {
                    if ((uint32_t)r < t.rows) {
                        StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(xs + r * row_elems), vxy[r], vzw[r]);
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
            const uint32_t cnt = max(t.rows, 1u) * min(s.B, s.W - t.bw * s.B);
            const float cntf = (float)cnt;
            float mean;
            if ((cnt & (cnt - 1)) == 0)
                mean = __fmul_rn(sum, __uint_as_float(0x7F000000u - __float_as_uint(cntf)));   // exact 1/2^k
            else
                mean = __fdiv_rn(sum, cntf);
            const float stored = Elem<LT>::round(mean);
            if (t.rows != 0u && (t.q % LPT) == 0) Elem<LT>::store(lfc_out + (size_t)n * s.C * s.TPP + t.ts, mean);
            // extremes of x over the strip's in-bounds rows; x -> fl(x - stored) is monotone
            float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
            if (t.rows != 0u) {
#pragma unroll
                for (int r = 0; r < P2; ++r) {
                    if (t.rows == (uint32_t)P2 || (uint32_t)r < t.rows) {
                        float a_, b_, c_, d_;
                        upk2(vxy[r], a_, b_);
                        upk2(vzw[r], c_, d_);
                        lo = fmin3(lo, a_, b_);
                        lo = fmin3(lo, c_, d_);
                        hi = fmax3(hi, a_, b_);
                        hi = fmax3(hi, c_, d_);
                    }
                }
                lo = __fsub_rn(lo, stored);
                hi = __fsub_rn(hi, stored);
            }
            const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
            const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
            if (lane == 0) {
                const uint32_t which = n - n0;
                atomicMax(&sh_kmin[par][which], kmin);
                atomicMax(&sh_kmax[par][which], kmax);
                atomicAdd(&sh_cnt[par][which], 1u);
            }
        }
        __syncthreads();
        if (threadIdx.x < 2) {
            // one update per sample and round from this CTA
            const uint32_t units = sh_cnt[par][threadIdx.x];
            if (units != 0u) {
                const uint32_t n = n0 + threadIdx.x;
                uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
                red_max_relaxed(slot + 0, sh_kmin[par][threadIdx.x]);
                red_max_relaxed(slot + 1, sh_kmax[par][threadIdx.x]);
                const uint32_t before = atom_add_acq_rel(slot + 2, units);
                sh_kmin[par][threadIdx.x] = 0;
                sh_kmax[par][threadIdx.x] = 0;
                sh_cnt[par][threadIdx.x] = 0;
                if (before + units == p.expected_units) {
                    // this update completes the sample
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

        // ================= quantise half: the unit reduced D rounds ago =================
        if (k >= D) {
            const uint64_t b0 = ((uint64_t)(k - D) * G + blockIdx.x) * WPC;
            if (b0 + warp < TU) {
                const uint32_t m0 = (uint32_t)(b0 / US);
                uint32_t uu = (uint32_t)(b0 - (uint64_t)m0 * US) + warp;
                uint32_t n = m0;
                if (uu >= US) {
                    uu -= US;
                    n += 1;
                }
                const uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
                uint32_t ready = 0, dbits = 0, sbits = 0;
                if (lane == 0 && !gave_up) {
                    uint32_t polls = 0;
                    uint64_t t0 = 0;
                    while (true) {
                        ready = ld_acquire_u32(slot + 3);
                        if (ready) break;
                        if ((++polls & 7u) == 0) {
                            const uint64_t t = now_ns();
                            if (t0 == 0) t0 = t;
                            if (ld_relaxed_u32(p.ws) != 0u || t - t0 > p.timeout_ns) {
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
                    const LStrip t = l_strip<P2>(p, uu, lane);
                    if (t.rows != 0u) {
                        // the low-frequency map was written by other CTAs: read it past the (incoherent) L1
                        const float stored = Elem<LT>::load_cg(lfc_out + (size_t)n * s.C * s.TPP + t.ts);
                        const XT* xs = x + ((size_t)n * s.CHW + t.e);
                        const uint64_t stored2 = pk2(stored, stored);
                        const uint64_t delta2 = pk2u(dbits, dbits), scale2 = pk2u(sbits, sbits);
                        const uint32_t g0 = t.e >> 2;
                        uint64_t ctr = rng_sample_base(p.seed, n) + K_GROUP * (uint64_t)(g0 + 1u);
                        OutT* out = packed + (((uint64_t)n * s.CHW) >> 2) + g0;
                        if (t.rows == (uint32_t)P2) {
                            uint64_t vxy[P2], vzw[P2];
#pragma unroll
                            for (int r = 0; r < P2; ++r)
                                StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(xs + r * row_elems), vxy[r], vzw[r]);
#pragma unroll
                            for (int r = 0; r < P2; ++r) {
                                out[r * W4] = (OutT)quant_row<Q>(vxy[r], vzw[r], stored2, delta2, scale2, rng_mix(ctr));
                                ctr += p.rng_row_step;
                            }
                        } else {
                            for (uint32_t r = 0; r < t.rows; ++r) {
                                uint64_t xy, zw;
                                StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(xs + r * row_elems), xy, zw);
                                out[r * W4] = (OutT)quant_row<Q>(xy, zw, stored2, delta2, scale2, rng_mix(ctr));
                                ctr += p.rng_row_step;
                            }
                        }
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
template <typename XT, typename LT, int Q, int P2>
inline div_status l_occupancy(int* ctas_per_sm) {
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, lagged_kernel<XT, LT, Q, P2>, L_THREADS, 0) != cudaSuccess) {
        cudaGetLastError();
        return DIV_ERR_CUDA;
    }
    return DIV_OK;
}

template <typename XT, typename LT>
inline div_status l_occupancy_q(int qbits, uint32_t p2, int* out) {
    if (p2 == 8) {
        if (qbits == 2) return l_occupancy<XT, LT, 2, 8>(out);
        if (qbits == 4) return l_occupancy<XT, LT, 4, 8>(out);
        if (qbits == 8) return l_occupancy<XT, LT, 8, 8>(out);
    } else if (p2 == 4) {
        if (qbits == 2) return l_occupancy<XT, LT, 2, 4>(out);
        if (qbits == 4) return l_occupancy<XT, LT, 4, 4>(out);
        if (qbits == 8) return l_occupancy<XT, LT, 8, 4>(out);
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
    const uint64_t slots = (uint64_t)s.C * s.Hb * pl.spb;
    if (slots >= (1ull << 31)) return DIV_ERR_PARAM;
    pl.slots_per_sample = (uint32_t)slots;
    pl.units_per_sample = (pl.slots_per_sample + 31u) / 32u;
    if (pl.units_per_sample < (uint32_t)L_WARPS) return DIV_ERR_PARAM;   // a CTA's span may cross one sample boundary only
    pl.total_units = (uint64_t)pl.units_per_sample * s.N;
    pl.threads = L_THREADS;
    int cps = 0;
    div_status st;
    if (d->x_dtype == DIV_F32)
        st = d->lfc_dtype == DIV_F32 ? l_occupancy_q<float, float>(d->qbits, s.P2, &cps) : l_occupancy_q<float, bf16>(d->qbits, s.P2, &cps);
    else
        st = d->lfc_dtype == DIV_F32 ? l_occupancy_q<bf16, float>(d->qbits, s.P2, &cps) : l_occupancy_q<bf16, bf16>(d->qbits, s.P2, &cps);
    if (st != DIV_OK) return st;
    if (cps < 1) return DIV_ERR_CUDA;
    pl.ctas_per_sm = cps;
    uint64_t grid = (uint64_t)di.sms * (uint64_t)cps;
    const uint64_t span_ctas = (pl.total_units + L_WARPS - 1) / L_WARPS;
    if (grid > span_ctas) grid = span_ctas;
    pl.grid = (int32_t)grid;
    const uint64_t gw = grid * L_WARPS;                                  // units per round
    const uint64_t rounds = (pl.total_units + gw - 1) / gw;
    if (rounds >= (1ull << 30)) return DIV_ERR_PARAM;
    pl.rounds = (uint32_t)rounds;
    // lag: far enough that the sample is complete when its units come up for quantising (every CTA has
    // then finished the rounds that hold the rest of the sample), and about DIVK_L_LAG_BYTES of x apart
    const uint64_t unit_bytes = 32ull * s.B * 4ull * sx;
    uint64_t lag = (DIVK_L_LAG_BYTES + gw * unit_bytes - 1) / (gw * unit_bytes);
    const uint64_t need = 1 + (pl.units_per_sample + gw - 1) / gw;
    if (lag < need) lag = need;
    pl.lag_rounds = (uint32_t)lag;
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
    typedef __nv_bfloat16 bf16;
    if (d->x_dtype == DIV_F32) {
        if (d->lfc_dtype == DIV_F32) return launch_lagged_q<float, float>(d->qbits, s.P2, prm, st);
        return launch_lagged_q<float, bf16>(d->qbits, s.P2, prm, st);
    }
    if (d->lfc_dtype == DIV_F32) return launch_lagged_q<bf16, float>(d->qbits, s.P2, prm, st);
    return launch_lagged_q<bf16, bf16>(d->qbits, s.P2, prm, st);
}

}  // namespace divk
