// Vectorised fused single-pass compress kernel (DIVISION Sec. 4.1; Algorithm 1, forward loop) for the
// common CNN shapes: W % 4 == 0, B in {4, 8}, Q in {2, 4, 8}.
//
// x is read from HBM once.  Each chunk waits in a shared-memory ring between the "reduce" half (block
// means, residual extremes) and the "quantise" half (Eq. 9 with stochastic rounding, packing), because
// the per-sample (delta, scale) are only known once every CTA has reduced its share of the sample.
//
// Roles inside a CTA (one CTA per SM, persistent):
//   warp 0   producer: one lane streams the chunks into the ring with bulk asynchronous copies;
//   warp 1   watcher: one lane waits, per chunk, until the chunk's sample is complete grid-wide (it
//            polls the sample's arrival counter in global scratch, slowly, so that the counter's L2
//            slice is not flooded), derives (delta, scale) and posts them in shared memory;
//   others   workers.  Work is cut into UNITS of 32 strips (a strip = 4 adjacent columns of one tile
//            row band, 4 x B elements, owned by one lane: B 16-byte shared-memory loads, column sums
//            in registers, one shuffle to meet the other half of a B = 8 tile).  Units are dealt
//            round-robin to the worker warps.  Each warp keeps two cursors, "next unit to reduce" and
//            "next unit to quantise", and always does whichever is possible, quantising first: nobody
//            blocks on the grid-wide dependency while loaded chunks are waiting to be reduced, so the
//            whole ring is available to hide that dependency's latency.
//   * the reduce half leaves, per strip, a 16-byte record in shared memory (stored low-frequency value,
//     where the strip sits in the stage, its index in the sample, its in-bounds rows); the quantise
//     half re-reads x from shared memory, subtracts the stored low-frequency value and emits the 4
//     codes of each strip row as one byte (Q = 2), half-word (Q = 4) or word (Q = 8) straight to the
//     packed stream: lanes of a warp write consecutive bytes.  Its fp32 arithmetic runs on packed
//     pairs (add/sub/mul/fma .f32x2: two IEEE results per instruction, same roundings as the scalar
//     forms).
//   * chunks are runs of `cb` consecutive tile row bands of one sample (they may cross planes);
//     chunk j goes to CTA j mod gridDim.x, so the CTAs sweep the samples together.
//
// Every wait is bounded: when a limit runs out the kernel records DIV_ERR_TIMEOUT in the workspace
// status word, stops waiting everywhere, lets its own copies land and returns.  The launch is
// cooperative only to be certain that all CTAs are resident (no grid-wide barrier is used).
#pragma once

#include "fused.cuh"

namespace divk {

#ifndef DIVK_V_WORKER_WARPS
#define DIVK_V_WORKER_WARPS 22
#endif
#ifndef DIVK_V_TARGET_BYTES
#define DIVK_V_TARGET_BYTES (32 * 1024)
#endif
#ifndef DIVK_V_POLL_NS
#define DIVK_V_POLL_NS 200
#endif
constexpr int V_WORKER_WARPS = DIVK_V_WORKER_WARPS;
constexpr int V_THREADS = 32 * (2 + V_WORKER_WARPS);
constexpr int V_MAX_STAGES = 16;

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
    uint32_t last_slots;          // strip slots of a sample's last (possibly short) chunk
    uint64_t rng_row_step;        // counter increment of the random stream from one row to the next (K_GROUP * W/4)
    uint64_t timeout_ns;
};

struct VDesc {
    uint32_t n, e0, bi0, nslots;
};

// per-stage descriptor, written by the producer before it issues the stage's copy
struct VStage {
    uint32_t n;          // sample
    uint32_t e0;         // in-sample index of the chunk's first element
    uint32_t bi0;        // first band
    uint32_t nslots;     // strip slots of the chunk
};

struct VCtl {
    uint64_t full[V_MAX_STAGES];        // producer -> workers: chunk landed
    uint64_t empty[V_MAX_STAGES];       // workers -> producer: stage may be overwritten
    uint32_t issued[V_MAX_STAGES];      // 1 + index of the chunk whose copy was last issued into the stage
    uint32_t reduced[V_MAX_STAGES];     // 1 + index of the chunk whose reduce half is complete in this CTA
    uint32_t posted[V_MAX_STAGES];      // 1 + index of the chunk whose (delta, scale) are posted below
    float par_delta[V_MAX_STAGES];
    float par_scale[V_MAX_STAGES];
    uint32_t kmin[V_MAX_STAGES];        // ~key(min r), key(max r) folded over the units of the chunk
    uint32_t kmax[V_MAX_STAGES];
    uint32_t done1[V_MAX_STAGES];       // units of the chunk that finished the reduce half
    uint32_t done2[V_MAX_STAGES];       // units of the chunk that finished the quantise half
    VStage desc[V_MAX_STAGES];
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
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t lds_volatile(const uint32_t* p) { return *(const volatile uint32_t*)p; }
__device__ __forceinline__ void sts_volatile(uint32_t* p, uint32_t v) { *(volatile uint32_t*)p = v; }

// bounded waits (same policy as fused.cuh, on this kernel's control block)
__device__ __forceinline__ bool v_give_up(const VParams& p, VCtl* ctl, uint64_t& t0) {
    if (lds_volatile(&ctl->failed) || ld_relaxed_u32(p.ws) != 0u) return true;
    const uint64_t t = now_ns();
    if (t0 == 0) t0 = t;
    return t - t0 > p.timeout_ns;
}
__device__ __forceinline__ void v_record_failure(const VParams& p, VCtl* ctl, uint32_t detail) {
    atomicCAS(p.ws, 0u, (uint32_t)DIV_ERR_TIMEOUT);
    atomicCAS(p.ws + 1, 0u, detail);
    sts_volatile(&ctl->failed, 1u);
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

template <int Q> struct PackedUnit;
template <> struct PackedUnit<2> { typedef uint8_t type; };
template <> struct PackedUnit<4> { typedef uint16_t type; };
template <> struct PackedUnit<8> { typedef uint32_t type; };

// ------------------------------------------------------------------------------------------------
// packed fp32 pairs (one instruction works on two values; IEEE, one rounding per value)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ uint64_t pk2u(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void upk2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void upk2u(uint64_t v, uint32_t& lo, uint32_t& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2_rn(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t add2_rp(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rp.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t sub2_rn(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul2_rn(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma2_rn(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t fma2_rp(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rp.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// a staged strip row as two packed pairs (x, y) and (z, w), widened to fp32
template <typename XT> struct StripRow2;
template <> struct StripRow2<float> {
    static __device__ __forceinline__ void load(const unsigned char* p, uint64_t& xy, uint64_t& zw) {
        const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(p);
        xy = v.x;
        zw = v.y;
    }
};
template <> struct StripRow2<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const unsigned char* p, uint64_t& xy, uint64_t& zw) {
        const uint2 u = *reinterpret_cast<const uint2*>(p);
        xy = pk2u(u.x << 16, u.x & 0xFFFF0000u);
        zw = pk2u(u.y << 16, u.y & 0xFFFF0000u);
    }
};

// Codes of two elements sharing the 32-bit half `h` of a random word (Eq. 9 with stochastic
// rounding); returns the two results QUANT2_BITS + code.  Same integer as quant_bits(): with
// F = 2^23 + field (the field dropped into the mantissa of 2^23), F * -2^-16 = -128 - u exactly, so one
// fused multiply-add rounded towards +inf gives d = RU(t - u - 128), and ceil(d) = ceil(t - u) - 128
// (rounding up never carries a value across an integer); the second add, of 1.5 * 2^23 + 128 and rounded up
// onto the integer grid of [2^23, 2^24), leaves ceil(t - u) in the low mantissa bits.  QUANT2_BITS has its
// low 22 bits clear, so where the packed codes are stored as a byte or a half-word (Q = 2, 4) the bias of the
// four results drops out of the stored bits by itself.
constexpr uint32_t QUANT2_BITS = MAGIC_CEIL_BITS;
constexpr float QUANT2_MAGIC = MAGIC_CEIL + 128.0f;
__device__ __forceinline__ void quant2(uint64_t x01, uint64_t stored2, uint64_t delta2, uint64_t scale2, float qmax,
                                       uint32_t h, uint32_t& b0, uint32_t& b1) {
    const uint64_t t01 = mul2_rn(sub2_rn(sub2_rn(x01, stored2), delta2), scale2);
    float t0, t1;
    upk2(t01, t0, t1);
    t0 = fminf(t0, qmax);
    t1 = fminf(t1, qmax);
    const uint64_t f01 = pk2u(__byte_perm(h, 0x4B000000u, 0x7610), __byte_perm(h, 0x4B000000u, 0x7632));   // 2^23 + field
    const uint64_t d01 = fma2_rp(f01, pk2(-1.52587890625e-05f, -1.52587890625e-05f), pk2(t0, t1));         // RU(t - u - 128)
    upk2u(add2_rp(d01, pk2(QUANT2_MAGIC, QUANT2_MAGIC)), b0, b1);
}

// four elements of one strip row -> their codes packed Q bits apart (low bits first)
template <int Q>
__device__ __forceinline__ uint32_t quant_row(uint64_t xy, uint64_t zw, uint64_t stored2, uint64_t delta2,
                                              uint64_t scale2, uint64_t z) {
    constexpr float qmax = (float)((1 << Q) - 1);
    uint32_t b0, b1, b2, b3;
    quant2(xy, stored2, delta2, scale2, qmax, (uint32_t)z, b0, b1);
    quant2(zw, stored2, delta2, scale2, qmax, (uint32_t)(z >> 32), b2, b3);
    constexpr uint32_t BIAS = QUANT2_BITS * (1u + (1u << Q) + (1u << (2 * Q)) + (1u << (3 * Q)));   // mod 2^32
    const uint32_t acc = b0 + (b1 << Q) + (b2 << (2 * Q)) + (b3 << (3 * Q));
    if constexpr (4 * Q < 22) return acc;      // the caller stores the low 4 * Q bits only: the bias does not reach them
    return acc - BIAS;
}

// the mixing function of the random stream (see rng_group) applied to a prepared counter
__device__ __forceinline__ uint64_t rng_mix(uint64_t z) {
    z ^= z >> 32;
    z *= K_MIX;
    z ^= z >> 32;
    z *= K_MIX;
    z ^= z >> 32;
    return z;
}

// per-slot record, written by the reduce half for the quantise half
//   x: stored low-frequency value (bits)   y: byte offset of the strip inside the stage
//   z: in-sample index of the strip's first element / 4   w: in-bounds rows (0: the slot is padding)

// position of a worker warp's cursor: unit U of this CTA = unit `u` of the CTA's chunk number `it`
struct VCursor {
    uint32_t U, it, u, st, round;
    bool real;        // the unit holds strips (a short chunk leaves its last unit slots empty)
};
__device__ __forceinline__ void v_seek(const VParams& p, VCursor& c, uint32_t U, uint32_t n_units) {
    c.U = U;
    if (U >= n_units) {
        c.real = false;
        return;
    }
    c.it = fdiv(U, p.by_nf);
    c.u = U - c.it * p.pl.nf;
    c.round = fdiv(c.it, p.by_K);
    c.st = c.it - c.round * (uint32_t)p.pl.stages;
    const uint32_t gc = blockIdx.x + c.it * gridDim.x;
    const uint32_t k = gc - fdiv(gc, p.by_S) * p.pl.chunks_per_sample;
    const uint32_t nslots = (k + 1u == p.pl.chunks_per_sample) ? p.last_slots : p.pl.cb * p.pl.spb;
    c.real = c.u * 32u < nslots;
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
    uint4* recs = reinterpret_cast<uint4*>(smem + (size_t)K * stage_bytes);
    VCtl* ctl = reinterpret_cast<VCtl*>(recs + (size_t)K * p.pl.slots_per_stage);

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t NW = (blockDim.x >> 5) - 2;
    const uint32_t G = gridDim.x;
    const uint64_t total = p.total_chunks;
    const uint32_t n_my = blockIdx.x < total ? (uint32_t)((total - blockIdx.x + G - 1) / G) : 0u;

    if (threadIdx.x == 0) {
        for (uint32_t i = 0; i < K; ++i) {
            mbar_init(&ctl->full[i], 1);
            mbar_init(&ctl->empty[i], 1);
            ctl->issued[i] = 0;
            ctl->reduced[i] = 0;
            ctl->posted[i] = 0;
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
            uint32_t it = 0;
            for (; it < n_my; ++it) {
                const uint32_t round = fdiv(it, p.by_K);
                const uint32_t st = it - round * K;
                if (it >= K && !v_wait_barrier(&ctl->empty[st], (round - 1) & 1, p, ctl)) break;
                uint32_t nelem;
                const VDesc d = v_chunk_desc(p, blockIdx.x + it * G, &nelem);
                const uint32_t bytes = nelem * (uint32_t)sizeof(XT);
                const XT* src = reinterpret_cast<const XT*>(p.x) + ((size_t)d.n * s.CHW + d.e0);
                VStage sd;
                sd.n = d.n;
                sd.e0 = d.e0;
                sd.bi0 = d.bi0;
                sd.nslots = d.nslots;
                ctl->desc[st] = sd;
                mbar_arrive_expect_tx(&ctl->full[st], bytes);
                bulk_load(smem + (size_t)st * stage_bytes, src, bytes, &ctl->full[st]);
                __threadfence_block();
                sts_volatile(&ctl->issued[st], it + 1u);
            }
            if (it < n_my || lds_volatile(&ctl->failed)) {
                // a wait gave up somewhere: let the copies still in flight land before the CTA may exit
                const uint32_t first = it > K ? it - K : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const uint32_t round = fdiv(j, p.by_K);
                    uint32_t polls = 0;
                    while (!mbar_try_wait(&ctl->full[j - round * K], round & 1) && ++polls < (1u << 20)) {
                    }
                }
            }
        }
        return;
    }

    if (warp == 1) {
        // ================= watcher: per chunk, wait for its sample's parameters and post them =================
        if (lane == 0) {
            uint32_t have_n = 0xFFFFFFFFu;
            float delta = 0.f, scale = 0.f;
            for (uint32_t it = 0; it < n_my; ++it) {
                const uint32_t round = fdiv(it, p.by_K);
                const uint32_t st = it - round * K;
                const VDesc d = v_chunk_desc(p, blockIdx.x + it * G);
                bool ok = true;
                if (d.n != have_n) {
                    uint32_t polls = 0;
                    uint64_t t0 = 0;
                    // first the cheap local condition: this CTA's own chunk has been reduced
                    while (lds_volatile(&ctl->reduced[st]) != it + 1u) {
                        if ((++polls & 63u) == 0 && v_give_up(p, ctl, t0)) {
                            ok = false;
                            break;
                        }
                        __nanosleep(40);
                    }
                    const uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)d.n * WS_SLOT_WORDS;
                    polls = 0;
                    t0 = 0;
                    while (ok && ld_acquire_u32(slot + 2) != p.expected_arrivals) {
                        if ((++polls & 7u) == 0 && v_give_up(p, ctl, t0)) {
                            ok = false;
                            break;
                        }
                        __nanosleep(DIVK_V_POLL_NS);
                    }
                    if (!ok) {
                        v_record_failure(p, ctl, d.n + 1u);
                        break;
                    }
                    const QParams qp = make_qparams(key_float(~ld_relaxed_u32(slot + 0)), key_float(ld_relaxed_u32(slot + 1)), Q);
                    delta = qp.delta;
                    scale = qp.scale;
                    have_n = d.n;
                }
                ctl->par_delta[st] = delta;
                ctl->par_scale[st] = scale;
                __threadfence_block();
                sts_volatile(&ctl->posted[st], it + 1u);
            }
        }
        return;
    }

    // ================= workers =================
    const uint32_t cw = warp - 2;
    const uint32_t n_units = n_my * p.pl.nf;
    const uint32_t row_bytes = s.W * (uint32_t)sizeof(XT);
    const uint32_t W4 = s.W >> 2;
    LT* lfc_out = reinterpret_cast<LT*>(p.lfc);
    OutT* packed = reinterpret_cast<OutT*>(p.packed);

    VCursor cr, cq;              // next unit to reduce / to quantise
    v_seek(p, cr, cw, n_units);
    v_seek(p, cq, cw, n_units);
    uint32_t idle = 0;
    uint64_t t0 = 0;

    while (cq.U < n_units) {
        // ---------------- quantise half of the oldest reduced unit, if its parameters are posted ----------------
        if (cq.U < cr.U) {
            if (!cq.real) {
                v_seek(p, cq, cq.U + NW, n_units);
                continue;
            }
            const uint32_t st = cq.st;
            if (__shfl_sync(0xFFFFFFFFu, lds_volatile(&ctl->posted[st]), 0) == cq.it + 1u) {
                __threadfence_block();
                const float delta = ctl->par_delta[st];
                const float scale = ctl->par_scale[st];
                const uint32_t n = ctl->desc[st].n;
                const uint32_t sl = cq.u * 32u + lane;
                const uint4 rec = recs[(size_t)st * p.pl.slots_per_stage + sl];
                if (rec.w != 0u) {
                    const unsigned char* xs = smem + (size_t)st * stage_bytes + rec.y;
                    const uint64_t stored2 = pk2u(rec.x, rec.x);
                    const uint64_t delta2 = pk2(delta, delta), scale2 = pk2(scale, scale);
                    uint64_t ctr = rng_sample_base(p.seed, n) + K_GROUP * (uint64_t)(rec.z + 1u);
                    OutT* out = packed + (((uint64_t)n * s.CHW) >> 2) + rec.z;
                    if (rec.w == (uint32_t)P2) {
#pragma unroll
                        for (int r = 0; r < P2; ++r) {
                            uint64_t xy, zw;
                            StripRow2<XT>::load(xs + r * row_bytes, xy, zw);
                            out[r * W4] = (OutT)quant_row<Q>(xy, zw, stored2, delta2, scale2, rng_mix(ctr));
                            ctr += p.rng_row_step;
                        }
                    } else {
                        for (uint32_t r = 0; r < rec.w; ++r) {
                            uint64_t xy, zw;
                            StripRow2<XT>::load(xs + r * row_bytes, xy, zw);
                            out[r * W4] = (OutT)quant_row<Q>(xy, zw, stored2, delta2, scale2, rng_mix(ctr));
                            ctr += p.rng_row_step;
                        }
                    }
                }
                // release: the last unit of the chunk hands the stage back to the producer
                __syncwarp();
                if (lane == 0) {
                    const uint32_t units = (ctl->desc[st].nslots + 31u) >> 5;
                    if (atomicAdd(&ctl->done2[st], 1u) == units - 1u) {
                        ctl->done2[st] = 0u;
                        __threadfence_block();
                        mbar_arrive(&ctl->empty[st]);
                    }
                }
                v_seek(p, cq, cq.U + NW, n_units);
                idle = 0;
                t0 = 0;
                continue;
            }
        }

        // ---------------- reduce half of the next unit, if its chunk has landed ----------------
        if (cr.U < n_units) {
            if (!cr.real) {
                v_seek(p, cr, cr.U + NW, n_units);
                continue;
            }
            const uint32_t st = cr.st;
            bool landed = __shfl_sync(0xFFFFFFFFu, lds_volatile(&ctl->issued[st]), 0) == cr.it + 1u;
            if (landed) landed = __any_sync(0xFFFFFFFFu, mbar_try_wait(&ctl->full[st], cr.round & 1));
            if (landed) {
                const VStage sd = ctl->desc[st];
                // geometry of this lane's strip
                const uint32_t sl = cr.u * 32u + lane;
                const bool valid = sl < sd.nslots;
                const uint32_t slc = valid ? sl : 0u;
                const uint32_t band_local = fdiv(slc, p.by_spb);
                const uint32_t q = slc - band_local * p.pl.spb;
                const uint32_t bi = sd.bi0 + band_local;
                const uint32_t plane = fdiv(bi, p.by_hb);
                const uint32_t bh = bi - plane * s.Hb;
                const uint32_t rows = min(s.B, s.H - bh * s.B);
                const uint32_t col0 = 4u * q;
                const bool ok = valid && col0 < s.W;
                const uint32_t e = plane * s.HW + bh * s.B * s.W + (ok ? col0 : 0u);
                const uint32_t off_bytes = (e - sd.e0) * (uint32_t)sizeof(XT);
                const unsigned char* xs = smem + (size_t)st * stage_bytes + off_bytes;

                uint64_t vxy[P2], vzw[P2];
                if (__all_sync(0xFFFFFFFFu, ok && rows == (uint32_t)P2)) {
#pragma unroll
                    for (int r = 0; r < P2; ++r) StripRow2<XT>::load(xs + r * row_bytes, vxy[r], vzw[r]);
                } else {
#pragma unroll
                    for (int r = 0; r < P2; ++r) {
                        if (ok && (uint32_t)r < rows) {
                            StripRow2<XT>::load(xs + r * row_bytes, vxy[r], vzw[r]);
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
                const uint32_t bw = q / LPT;
                const uint32_t cnt = rows * min(s.B, s.W - bw * s.B);
                const float cntf = (float)cnt;
                float mean;
                if ((cnt & (cnt - 1)) == 0)
                    mean = __fmul_rn(sum, __uint_as_float(0x7F000000u - __float_as_uint(cntf)));   // exact 1/2^k
                else
                    mean = __fdiv_rn(sum, cntf);
                const float stored = Elem<LT>::round(mean);
                if (ok && (q % LPT) == 0)
                    Elem<LT>::store(lfc_out + (size_t)sd.n * s.C * s.TPP + (plane * s.TPP + bh * s.Wb + bw), mean);
                recs[(size_t)st * p.pl.slots_per_stage + sl] =
                    make_uint4(__float_as_uint(stored), off_bytes, e >> 2, ok ? rows : 0u);
                // extremes of x over the strip's in-bounds rows; x -> fl(x - stored) is monotone
                float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
                if (ok) {
#pragma unroll
                    for (int r = 0; r < P2; ++r) {
                        if (rows == (uint32_t)P2 || (uint32_t)r < rows) {
                            float a, b, c, d;
                            upk2(vxy[r], a, b);
                            upk2(vzw[r], c, d);
                            lo = fmin3(lo, a, b);
                            lo = fmin3(lo, c, d);
                            hi = fmax3(hi, a, b);
                            hi = fmax3(hi, c, d);
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
                    const uint32_t units = (sd.nslots + 31u) >> 5;
                    if (atomicAdd(&ctl->done1[st], 1u) == units - 1u) {
                        // last unit of this chunk: fold the chunk into its sample's slot
                        __threadfence_block();
                        const uint32_t smin = atomicExch(&ctl->kmin[st], 0u);
                        const uint32_t smax = atomicExch(&ctl->kmax[st], 0u);
                        ctl->done1[st] = 0u;
                        uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)sd.n * WS_SLOT_WORDS;
                        if (lds_volatile(&ctl->failed) == 0u) {
                            red_max_relaxed(slot + 0, smin);
                            red_max_relaxed(slot + 1, smax);
                            const uint32_t before = atom_add_acq_rel(slot + 2, 1u);
                            sts_volatile(&ctl->reduced[st], cr.it + 1u);
                            if (before == p.expected_arrivals - 1u) {
                                // the arrival that completes the sample writes its (delta, Delta) to the blob
                                const QParams qp = make_qparams(key_float(~ld_relaxed_u32(slot + 0)),
                                                                key_float(ld_relaxed_u32(slot + 1)), Q);
                                p.stats[2 * (size_t)sd.n + 0] = qp.delta;
                                p.stats[2 * (size_t)sd.n + 1] = qp.step;
                            }
                        }
                    }
                }
                v_seek(p, cr, cr.U + NW, n_units);
                idle = 0;
                t0 = 0;
                continue;
            }
        }

        // ---------------- nothing to do right now ----------------
        if ((++idle & 15u) == 0) {
            bool stop = false;
            if (lane == 0) {
                stop = v_give_up(p, ctl, t0);
                if (stop) v_record_failure(p, ctl, 0x40000000u | cq.U);
            }
            if (__any_sync(0xFFFFFFFFu, stop)) break;
        }
        __nanosleep(100);
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
    const uint32_t target = DIVK_V_TARGET_BYTES;               // chunk bytes we aim for
    if (band_bytes + 256u > budget / 4) return DIV_ERR_PARAM;
    // bands per chunk: near the target size, a count that fills whole units of 32 strips where possible
    const uint32_t cbq = 32u / gcd_u32(32u, pl.spb);
    uint32_t cb = target / band_bytes;
    if (cb == 0) cb = 1;
    if (cb >= cbq) cb = cb / cbq * cbq;
    if (cb > pl.bands_per_sample) cb = pl.bands_per_sample;
    pl.cb = cb;
    pl.nf = (cb * pl.spb + 31u) / 32u;
    pl.slots_per_stage = pl.nf * 32u;
    pl.chunk_elems = cb * s.B * s.W;
    pl.chunks_per_sample = (pl.bands_per_sample + cb - 1) / cb;
    pl.stage_bytes = (cb * band_bytes + 127u) & ~127u;
    const uint32_t per_stage = pl.stage_bytes + pl.slots_per_stage * 16u;
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
    // progress guarantee: a sample completes only when every CTA has reduced all of its chunks of that
    // sample, so those chunks (plus room for the next copy) must fit in a CTA's ring together
    const uint64_t span = (pl.chunks_per_sample + grid - 1) / grid;
    if (span + 2 > stages) return DIV_ERR_PARAM;
    pl.lag = (int32_t)(stages - span);      // chunks the reduce half may run ahead of the quantise half
    *out = pl;
    return DIV_OK;
}

template <typename XT, typename LT, int Q, int P2>
inline div_status launch_v(const VParams& prm, cudaStream_t st) {
    auto kern = fused_v_kernel<XT, LT, Q, P2>;
    static SmemSeen smem_set[DEVICE_CACHE_SLOTS];
    if (!ensure_dynamic_smem((const void*)kern, prm.pl.smem_bytes, smem_set)) return DIV_ERR_CUDA;
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
    prm.last_slots = (pl.bands_per_sample - (pl.chunks_per_sample - 1u) * pl.cb) * pl.spb;
    prm.rng_row_step = K_GROUP * (uint64_t)(s.W / 4u);
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
