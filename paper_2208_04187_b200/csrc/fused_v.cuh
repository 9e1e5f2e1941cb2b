// Vectorised fused single-pass compress kernel (DIVISION Sec. 4.1; Algorithm 1 lines 3-6) for the
// common CNN shapes: W % 4 == 0, B in {4, 8}, Q in {2, 4, 8}.
//
// Same plan as the general fused kernel (fused.cuh): x is read from HBM once, each chunk waits in a
// shared-memory ring between the "reduce" half (block means, residual extremes) and the "quantise"
// half (Eq. 9 with stochastic rounding, packing), and the per-sample (delta, scale) travel through a
// slot in global scratch.  What differs is the work decomposition, chosen for instruction count:
//
//   * a STRIP is 4 adjacent columns of one tile row band (4 x B elements); one thread owns a strip:
//     B 16-byte shared-memory loads, the column sums of its 4 columns in registers, one shuffle to
//     meet the other half of a B = 8 tile.  No predicates and no index arithmetic per element;
//   * a UNIT is 32 consecutive strips (one per lane).  Units are dealt round-robin to the consumer
//     warps; warp w runs the reduce half of unit w + i*NW and then the quantise half of the unit
//     `lag` positions earlier, so the wait for the sample's parameters is normally already over;
//   * the quantise half re-reads x from shared memory, subtracts the stored low-frequency value
//     (kept per strip in shared memory) and emits the 4 codes of each strip row as one byte (Q = 2),
//     half-word (Q = 4) or word (Q = 8) straight to the packed stream: lanes of a warp write
//     consecutive bytes.
//   * chunks are runs of `cb` consecutive tile row bands of one sample (they may cross planes);
//     chunk j goes to CTA j mod gridDim.x.
//
// All waits are bounded exactly as in fused.cuh.
#pragma once

#include "fused.cuh"

namespace divk {

#ifndef DIVK_V_CONSUMER_WARPS
#define DIVK_V_CONSUMER_WARPS 16
#endif
constexpr int V_CONSUMER_WARPS = DIVK_V_CONSUMER_WARPS;
constexpr int V_THREADS = 32 * (1 + V_CONSUMER_WARPS);
constexpr int V_MAX_STAGES = 8;

struct VPlan {
    int32_t grid, threads, stages, lag, smem_bytes;
    uint32_t cb;                 // tile row bands per full chunk
    uint32_t spb;                // strip slots per band (tiles per row * lanes per tile)
    uint32_t nf;                 // units per full chunk
    uint32_t chunk_elems;        // elements of a full chunk of full-height bands
    uint32_t chunks_per_sample;  // S
    uint32_t bands_per_sample;   // C * Hb
    uint32_t stage_bytes;
    uint32_t slots_per_stage;    // nf * 32
};

struct VParams {
    Shape s;
    VPlan pl;
    FastDiv by_S, by_spb, by_hb, by_nf, by_K;
    const void* x;
    void* lfc;
    void* packed;
    float* stats;
    uint32_t* ws;
    uint64_t seed;
    uint64_t total_chunks;
    uint32_t expected_arrivals;
    uint64_t timeout_ns;
};

struct VDesc {
    uint32_t n, e0, bi0, nslots;
};

struct VCtl {
    uint64_t full[V_MAX_STAGES];
    uint64_t empty[V_MAX_STAGES];
    uint32_t kmin[V_MAX_STAGES];
    uint32_t kmax[V_MAX_STAGES];
    uint32_t done1[V_MAX_STAGES];
    uint32_t done2[V_MAX_STAGES];
    uint32_t failed;
};

// geometry of global chunk `gc`: sample, first band, first element, number of strip slots, bytes
__device__ __forceinline__ VDesc v_chunk_desc(const VParams& p, uint32_t gc, uint32_t* nelem = nullptr) {
    const Shape& s = p.s;
    VDesc d;
    d.n = fdiv(gc, p.by_S);
    const uint32_t k = gc - d.n * p.pl.chunks_per_sample;
    d.bi0 = k * p.pl.cb;
    const uint32_t bi1 = min(p.pl.bands_per_sample, d.bi0 + p.pl.cb);
    const uint32_t pl0 = fdiv(d.bi0, p.by_hb);
    d.e0 = pl0 * s.HW + (d.bi0 - pl0 * s.Hb) * s.B * s.W;
    d.nslots = (bi1 - d.bi0) * p.pl.spb;
    if (nelem) {
        const uint32_t pl1 = fdiv(bi1, p.by_hb);
        *nelem = pl1 * s.HW + (bi1 - pl1 * s.Hb) * s.B * s.W - d.e0;
    }
    return d;
}

__device__ __forceinline__ float fmin3(float a, float b, float c) {
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ uint32_t atom_add_acq_rel(uint32_t* p, uint32_t v) {
    uint32_t old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void red_max_relaxed(uint32_t* p, uint32_t v) {
    asm volatile("red.relaxed.gpu.global.max.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// bounded waits (same policy as fused.cuh, on this kernel's control block)
__device__ __forceinline__ bool v_give_up(const VParams& p, VCtl* ctl, uint64_t& t0) {
    if (*(volatile uint32_t*)&ctl->failed || ld_relaxed_u32(p.ws) != 0u) return true;
    const uint64_t t = now_ns();
    if (t0 == 0) t0 = t;
    return t - t0 > p.timeout_ns;
}
__device__ __forceinline__ void v_record_failure(const VParams& p, VCtl* ctl, uint32_t detail) {
    atomicCAS(p.ws, 0u, (uint32_t)DIV_ERR_TIMEOUT);
    atomicCAS(p.ws + 1, 0u, detail);
    *(volatile uint32_t*)&ctl->failed = 1u;
}
__device__ __forceinline__ bool v_wait_barrier(uint64_t* bar, uint32_t parity, const VParams& p, VCtl* ctl) {
    if (mbar_try_wait(bar, parity)) return true;
    uint32_t polls = 0;
    uint64_t t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 31u) == 0 && v_give_up(p, ctl, t0)) {
            v_record_failure(p, ctl, 0x80000000u);
            return false;
        }
    }
    return true;
}

// 4 adjacent values of a staged strip row, widened to fp32
template <typename XT> struct StripRow;
template <> struct StripRow<float> {
    static __device__ __forceinline__ float4 load(const float* p) { return *reinterpret_cast<const float4*>(p); }
};
template <> struct StripRow<__nv_bfloat16> {
    static __device__ __forceinline__ float4 load(const __nv_bfloat16* p) {
        const uint2 u = *reinterpret_cast<const uint2*>(p);
        return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u),
                           __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xFFFF0000u));
    }
};

template <int Q> struct PackedUnit;
template <> struct PackedUnit<2> { typedef uint8_t type; };
template <> struct PackedUnit<4> { typedef uint16_t type; };
template <> struct PackedUnit<8> { typedef uint32_t type; };

// geometry of the strip a lane owns inside a chunk
struct Strip {
    uint32_t off;     // element offset of its first element inside the staged chunk
    uint32_t e;       // the same as in-sample flat index
    uint32_t rows;    // in-bounds rows of its band
    uint32_t ts;      // tile index inside the sample (plane * TPP + bh * Wb + bw)
    uint32_t q;       // slot inside the band
    bool ok;          // slot holds real columns
};
template <int P2>
__device__ __forceinline__ Strip strip_of(const VParams& p, const VDesc& d, uint32_t sl) {
    constexpr uint32_t LPT = P2 / 4;
    const Shape& s = p.s;
    Strip t;
    const uint32_t slc = sl < d.nslots ? sl : 0u;
    const uint32_t band_local = fdiv(slc, p.by_spb);
    t.q = slc - band_local * p.pl.spb;
    const uint32_t bi = d.bi0 + band_local;
    const uint32_t plane = fdiv(bi, p.by_hb);
    const uint32_t bh = bi - plane * s.Hb;
    t.rows = min(s.B, s.H - bh * s.B);
    const uint32_t col0 = 4u * t.q;
    t.ok = (sl < d.nslots) && (col0 < s.W);
    t.e = plane * s.HW + bh * s.B * s.W + (t.ok ? col0 : 0u);
    t.off = t.e - d.e0;
    t.ts = plane * s.TPP + bh * s.Wb + t.q / LPT;
    return t;
}

template <typename XT, typename LT, int Q, int P2>
__global__ void __launch_bounds__(V_THREADS, 1)
fused_v_kernel(const VParams p) {
    constexpr uint32_t LPT = P2 / 4;
    typedef typename PackedUnit<Q>::type OutT;

    extern __shared__ __align__(128) unsigned char smem[];
    const Shape& s = p.s;
    const uint32_t K = p.pl.stages;
    const uint32_t stage_bytes = p.pl.stage_bytes;
    float* lfcs = reinterpret_cast<float*>(smem + (size_t)K * stage_bytes);
    VCtl* ctl = reinterpret_cast<VCtl*>(lfcs + (size_t)K * p.pl.slots_per_stage);

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t NW = (blockDim.x >> 5) - 1;
    const uint32_t G = gridDim.x;
    const uint64_t total = p.total_chunks;
    const uint32_t n_my = blockIdx.x < total ? (uint32_t)((total - blockIdx.x + G - 1) / G) : 0u;

    if (threadIdx.x == 0) {
        for (uint32_t i = 0; i < K; ++i) {
            mbar_init(&ctl->full[i], 1);
            mbar_init(&ctl->empty[i], 1);
            ctl->kmin[i] = 0;
            ctl->kmax[i] = 0;
            ctl->done1[i] = 0;
            ctl->done2[i] = 0;
        }
        ctl->failed = 0;
        fence_barrier_init();
    }
    __syncthreads();

    if (warp == 0) {
        // ================= producer: one lane streams the chunks into the ring =================
        if (lane == 0) {
            for (uint32_t it = 0; it < n_my; ++it) {
                const uint32_t round = fdiv(it, p.by_K);
                const uint32_t st = it - round * K;
                if (it >= K && !v_wait_barrier(&ctl->empty[st], (round - 1) & 1, p, ctl)) break;
                uint32_t nelem;
                const VDesc d = v_chunk_desc(p, blockIdx.x + it * G, &nelem);
                const uint32_t bytes = nelem * (uint32_t)sizeof(XT);
                const XT* src = reinterpret_cast<const XT*>(p.x) + ((size_t)d.n * s.CHW + d.e0);
                mbar_arrive_expect_tx(&ctl->full[st], bytes);
                bulk_load(smem + (size_t)st * stage_bytes, src, bytes, &ctl->full[st]);
            }
        }
        return;
    }

    // ================= consumers =================
    const uint32_t cw = warp - 1;
    const uint32_t nf = p.pl.nf;
    const uint32_t n_units = n_my * nf;
    const uint32_t L = (uint32_t)p.pl.lag;
    LT* lfc_out = reinterpret_cast<LT*>(p.lfc);
    OutT* packed = reinterpret_cast<OutT*>(p.packed);
    bool alive = true;

    for (uint32_t U1 = cw; U1 < n_units + L; U1 += NW) {
        const bool has1 = U1 < n_units;
        const bool has2 = U1 >= L;

        // ---------------- reduce half of unit U1 ----------------
        if (has1) {
            const uint32_t it = fdiv(U1, p.by_nf);
            const uint32_t u = U1 - it * nf;
            const uint32_t round = fdiv(it, p.by_K);
            const uint32_t st = it - round * K;
            const VDesc d = v_chunk_desc(p, blockIdx.x + it * G);
            const bool real = u * 32u < d.nslots;      // a short chunk leaves its last unit slots empty
            if (alive && real) alive = v_wait_barrier(&ctl->full[st], round & 1, p, ctl);
            if (alive && real) {
                const uint32_t sl = u * 32u + lane;
                const Strip t = strip_of<P2>(p, d, sl);
                const XT* xs = reinterpret_cast<const XT*>(smem + (size_t)st * stage_bytes) + t.off;
                float4 v[P2];
                if (__all_sync(0xFFFFFFFFu, t.ok && t.rows == (uint32_t)P2)) {
#pragma unroll
                    for (int r = 0; r < P2; ++r) v[r] = StripRow<XT>::load(xs + r * s.W);
                } else {
#pragma unroll
                    for (int r = 0; r < P2; ++r)
                        v[r] = (t.ok && (uint32_t)r < t.rows) ? StripRow<XT>::load(xs + r * s.W)
                                                              : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                // column sums: balanced tree down the rows of each of the 4 columns
                float4 c[P2];
#pragma unroll
                for (int r = 0; r < P2; ++r) c[r] = v[r];
#pragma unroll
                for (int w = P2; w > 1; w >>= 1) {
#pragma unroll
                    for (int i = 0; i < w / 2; ++i) {
                        c[i].x = __fadd_rn(c[2 * i].x, c[2 * i + 1].x);
                        c[i].y = __fadd_rn(c[2 * i].y, c[2 * i + 1].y);
                        c[i].z = __fadd_rn(c[2 * i].z, c[2 * i + 1].z);
                        c[i].w = __fadd_rn(c[2 * i].w, c[2 * i + 1].w);
                    }
                }
                float sum = __fadd_rn(__fadd_rn(c[0].x, c[0].y), __fadd_rn(c[0].z, c[0].w));
#pragma unroll
                for (int m = 1; m < (int)LPT; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
                const uint32_t bw = t.q / LPT;
                const uint32_t cnt = t.rows * min(s.B, s.W - bw * s.B);
                const float cntf = (float)cnt;
                float mean;
                if ((cnt & (cnt - 1)) == 0)
                    mean = __fmul_rn(sum, __uint_as_float(0x7F000000u - __float_as_uint(cntf)));   // exact 1/2^k
                else
                    mean = __fdiv_rn(sum, cntf);
                const float stored = Elem<LT>::round(mean);
                if (t.ok && (t.q % LPT) == 0) Elem<LT>::store(lfc_out + (size_t)d.n * s.C * s.TPP + t.ts, mean);
                lfcs[(size_t)st * p.pl.slots_per_stage + sl] = stored;
                // extremes of x over the strip's in-bounds rows; x -> fl(x - stored) is monotone
                float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
                if (t.ok) {
                    if (t.rows == (uint32_t)P2) {
#pragma unroll
                        for (int r = 0; r < P2; ++r) {
                            lo = fmin3(lo, v[r].x, v[r].y);
                            lo = fmin3(lo, v[r].z, v[r].w);
                            hi = fmax3(hi, v[r].x, v[r].y);
                            hi = fmax3(hi, v[r].z, v[r].w);
                        }
                    } else {
#pragma unroll
                        for (int r = 0; r < P2; ++r) {
                            if ((uint32_t)r < t.rows) {
                                lo = fmin3(lo, v[r].x, v[r].y);
                                lo = fmin3(lo, v[r].z, v[r].w);
                                hi = fmax3(hi, v[r].x, v[r].y);
                                hi = fmax3(hi, v[r].z, v[r].w);
                            }
                        }
                    }
                    lo = __fsub_rn(lo, stored);
                    hi = __fsub_rn(hi, stored);
                }
                const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
                const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
                __syncwarp();
                if (lane == 0) {
                    atomicMax(&ctl->kmin[st], kmin);
                    atomicMax(&ctl->kmax[st], kmax);
                    __threadfence_block();
                    const uint32_t units = (d.nslots + 31u) >> 5;
                    if (atomicAdd(&ctl->done1[st], 1u) == units - 1u) {
                        // last unit of this chunk: fold the chunk into its sample's slot
                        __threadfence_block();
                        const uint32_t smin = atomicExch(&ctl->kmin[st], 0u);
                        const uint32_t smax = atomicExch(&ctl->kmax[st], 0u);
                        ctl->done1[st] = 0u;
                        uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)d.n * WS_SLOT_WORDS;
                        if (*(volatile uint32_t*)&ctl->failed == 0u) {
                            red_max_relaxed(slot + 0, smin);
                            red_max_relaxed(slot + 1, smax);
                            if (atom_add_acq_rel(slot + 2, 1u) == p.expected_arrivals - 1u) {
                                const float rlo = key_float(~ld_relaxed_u32(slot + 0));
                                const float rhi = key_float(ld_relaxed_u32(slot + 1));
                                const QParams qp = make_qparams(rlo, rhi, Q);
                                p.stats[2 * (size_t)d.n + 0] = qp.delta;
                                p.stats[2 * (size_t)d.n + 1] = qp.step;
                                const uint64_t word = ((uint64_t)(__float_as_uint(qp.scale) | 0x80000000u) << 32) |
                                                      (uint64_t)__float_as_uint(qp.delta);
                                st_release_u64(reinterpret_cast<uint64_t*>(slot + 4), word);
                            }
                        }
                    }
                }
            }
        }

        // ---------------- quantise half of unit U1 - L ----------------
        if (has2) {
            const uint32_t U2 = U1 - L;
            const uint32_t it = fdiv(U2, p.by_nf);
            const uint32_t u = U2 - it * nf;
            const uint32_t round = fdiv(it, p.by_K);
            const uint32_t st = it - round * K;
            const VDesc d = v_chunk_desc(p, blockIdx.x + it * G);
            const bool real = u * 32u < d.nslots;
            // the chunk landed long ago, but this warp may not have looked at its barrier yet
            if (alive && real) alive = v_wait_barrier(&ctl->full[st], round & 1, p, ctl);
            if (real) {
                uint64_t word = 0;
                if (alive) {
                    if (lane == 0) {
                        const uint64_t* pw =
                            reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)d.n * WS_SLOT_WORDS + 4);
                        uint32_t polls = 0;
                        uint64_t t0 = 0;
                        while (true) {
                            word = ld_relaxed_u64(pw);
                            if (word >> 63) break;
                            if ((++polls & 63u) == 0) {
                                if (v_give_up(p, ctl, t0)) {
                                    v_record_failure(p, ctl, d.n + 1u);
                                    word = 0;
                                    break;
                                }
                                __nanosleep(32);
                            }
                        }
                        fence_acq_rel_gpu();
                    }
                    word = __shfl_sync(0xFFFFFFFFu, word, 0);
                    alive = (word >> 63) != 0;
                }
                if (alive) {
                    const float delta = __uint_as_float((uint32_t)word);
                    const float scale = __uint_as_float((uint32_t)(word >> 32) & 0x7FFFFFFFu);
                    const uint64_t base = rng_sample_base(p.seed, d.n);
                    const uint32_t sl = u * 32u + lane;
                    const Strip t = strip_of<P2>(p, d, sl);
                    if (t.ok) {
                        const XT* xs = reinterpret_cast<const XT*>(smem + (size_t)st * stage_bytes) + t.off;
                        const float stored = lfcs[(size_t)st * p.pl.slots_per_stage + sl];
                        const uint32_t W4 = s.W >> 2;
                        const uint32_t g0 = t.e >> 2;
                        OutT* out = packed + (((uint64_t)d.n * s.CHW) >> 2) + g0;
                        if (t.rows == (uint32_t)P2) {
#pragma unroll
                            for (int r = 0; r < P2; ++r) {
                                const float4 x4 = StripRow<XT>::load(xs + r * s.W);
                                const uint64_t z = rng_group(base, g0 + r * W4);
                                out[r * W4] = (OutT)quant4<Q>(__fsub_rn(x4.x, stored), __fsub_rn(x4.y, stored),
                                                              __fsub_rn(x4.z, stored), __fsub_rn(x4.w, stored), delta,
                                                              scale, z);
                            }
                        } else {
                            for (uint32_t r = 0; r < t.rows; ++r) {
                                const float4 x4 = StripRow<XT>::load(xs + r * s.W);
                                const uint64_t z = rng_group(base, g0 + r * W4);
                                out[r * W4] = (OutT)quant4<Q>(__fsub_rn(x4.x, stored), __fsub_rn(x4.y, stored),
                                                              __fsub_rn(x4.z, stored), __fsub_rn(x4.w, stored), delta,
                                                              scale, z);
                            }
                        }
                    }
                }
                // release: the last unit of the chunk hands the stage back to the producer
                __syncwarp();
                if (lane == 0) {
                    const uint32_t units = (d.nslots + 31u) >> 5;
                    if (atomicAdd(&ctl->done2[st], 1u) == units - 1u) {
                        ctl->done2[st] = 0u;
                        __threadfence_block();
                        mbar_arrive(&ctl->empty[st]);
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
inline div_status plan_v(const div_desc* d, const Shape& s, VPlan* out) {
    const uint32_t sx = d->x_dtype == DIV_F32 ? 4u : 2u;
    if (s.W % 4 != 0) return DIV_ERR_PARAM;
    if (!(s.B == 4 || s.B == 8) || s.P2 != s.B) return DIV_ERR_PARAM;
    if (!(d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return DIV_ERR_PARAM;
    const uint32_t tma = 16u / sx;
    if (s.HW % tma != 0 || (s.B * s.W) % tma != 0) return DIV_ERR_PARAM;
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return DIV_ERR_CUDA;

    VPlan pl = VPlan();
    const uint32_t lpt = s.P2 / 4;
    pl.spb = s.Wb * lpt;
    pl.bands_per_sample = s.C * s.Hb;
    pl.threads = V_THREADS;
    const uint32_t band_bytes = s.B * s.W * sx;
    const uint32_t budget = (uint32_t)di.smem_optin - 2048u - (uint32_t)sizeof(VCtl);
    const uint32_t target = 30u * 1024u;                       // chunk bytes we aim for
    if (band_bytes + 256u > budget / 4) return DIV_ERR_PARAM;
    // whole units per chunk where the band geometry allows it
    const uint32_t cbq = 32u / gcd_u32(32u, pl.spb);
    uint32_t cb = target / band_bytes;
    if (cb >= cbq) cb = cb / cbq * cbq;
    if (cb == 0) cb = 1;
    if (cb > pl.bands_per_sample) cb = pl.bands_per_sample;
    pl.cb = cb;
    pl.nf = (cb * pl.spb + 31u) / 32u;
    pl.slots_per_stage = pl.nf * 32u;
    pl.chunk_elems = cb * s.B * s.W;
    pl.chunks_per_sample = (pl.bands_per_sample + cb - 1) / cb;
    pl.stage_bytes = (cb * band_bytes + 127u) & ~127u;
    const uint32_t per_stage = pl.stage_bytes + pl.slots_per_stage * 4u;
    uint32_t stages = budget / per_stage;
    if (stages > (uint32_t)V_MAX_STAGES) stages = V_MAX_STAGES;
    if (stages < 4) return DIV_ERR_PARAM;
    pl.stages = (int32_t)stages;
    pl.smem_bytes = (int32_t)(stages * per_stage + sizeof(VCtl) + 128u);
    const uint64_t total_chunks = (uint64_t)pl.chunks_per_sample * s.N;
    if (total_chunks * pl.nf >= (1ull << 31)) return DIV_ERR_PARAM;
    uint64_t grid = (uint64_t)di.sms;
    if (grid > total_chunks) grid = total_chunks;
    pl.grid = (int32_t)grid;
    // lag (in units): keep two stages for loads in flight and one for the chunk being reduced
    const int64_t alive_units = (int64_t)(stages - 3) * pl.nf - V_CONSUMER_WARPS;
    int64_t lag = alive_units;
    if (lag < (int64_t)pl.nf) lag = pl.nf;
    // progress guarantee: units of one sample inside one CTA must fit between the two halves
    const uint64_t span = ((pl.chunks_per_sample + grid - 1) / grid) * pl.nf;
    if (span > (uint64_t)lag + V_CONSUMER_WARPS) return DIV_ERR_PARAM;
    // and the ring must hold everything between the oldest lagging unit and the newest reduced unit
    if ((uint64_t)(lag + V_CONSUMER_WARPS + pl.nf - 1) / pl.nf + 1 > stages) return DIV_ERR_PARAM;
    pl.lag = (int32_t)lag;
    *out = pl;
    return DIV_OK;
}

template <typename XT, typename LT, int Q, int P2>
inline div_status launch_v(const VParams& prm, cudaStream_t st) {
    auto kern = fused_v_kernel<XT, LT, Q, P2>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, prm.pl.smem_bytes) != cudaSuccess) {
        cudaGetLastError();
        return DIV_ERR_CUDA;
    }
    void* args[] = {(void*)&prm};
    if (cudaLaunchCooperativeKernel((const void*)kern, dim3(prm.pl.grid), dim3(prm.pl.threads), args,
                                    (size_t)prm.pl.smem_bytes, st) != cudaSuccess) {
        cudaGetLastError();
        return DIV_ERR_CUDA;
    }
    return DIV_OK;
}

template <typename XT, typename LT>
inline div_status launch_v_q(int qbits, uint32_t p2, const VParams& prm, cudaStream_t st) {
    if (p2 == 8) {
        if (qbits == 2) return launch_v<XT, LT, 2, 8>(prm, st);
        if (qbits == 4) return launch_v<XT, LT, 4, 8>(prm, st);
        if (qbits == 8) return launch_v<XT, LT, 8, 8>(prm, st);
    } else if (p2 == 4) {
        if (qbits == 2) return launch_v<XT, LT, 2, 4>(prm, st);
        if (qbits == 4) return launch_v<XT, LT, 4, 4>(prm, st);
        if (qbits == 8) return launch_v<XT, LT, 8, 4>(prm, st);
    }
    return DIV_ERR_PARAM;
}

inline div_status compress_fused_v(const div_desc* d, const Shape& s, const div_layout& lo, const VPlan& pl,
                                   const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st,
                                   uint32_t expected_arrivals = 0, uint64_t timeout_ns = 0) {
    VParams prm;
    prm.s = s;
    prm.pl = pl;
    prm.by_S = host_fastdiv(pl.chunks_per_sample);
    prm.by_spb = host_fastdiv(pl.spb);
    prm.by_hb = host_fastdiv(s.Hb);
    prm.by_nf = host_fastdiv(pl.nf);
    prm.by_K = host_fastdiv((uint32_t)pl.stages);
    prm.x = x;
    prm.lfc = blob + lo.lfc_off;
    prm.packed = blob + lo.packed_off;
    prm.stats = reinterpret_cast<float*>(blob + lo.stats_off);
    prm.ws = ws;
    prm.seed = seed;
    prm.total_chunks = (uint64_t)pl.chunks_per_sample * s.N;
    prm.expected_arrivals = expected_arrivals ? expected_arrivals : pl.chunks_per_sample;
    prm.timeout_ns = timeout_ns ? timeout_ns : 2000000000ull;
    typedef __nv_bfloat16 bf16;
    if (d->x_dtype == DIV_F32) {
        if (d->lfc_dtype == DIV_F32) return launch_v_q<float, float>(d->qbits, s.P2, prm, st);
        return launch_v_q<float, bf16>(d->qbits, s.P2, prm, st);
    }
    if (d->lfc_dtype == DIV_F32) return launch_v_q<bf16, float>(d->qbits, s.P2, prm, st);
    return launch_v_q<bf16, bf16>(d->qbits, s.P2, prm, st);
}

}  // namespace divk
