// Staged single-launch compress kernel (DIVISION Sec. 4.1; Algorithm 1, forward loop) for the common CNN
// shapes: W % 4 == 0, B in {4, 8}, Q in {2, 4, 8}.
//
// Like the lagged kernel, x is read from HBM once ("reduce": block means, residual extremes) and a second
// time a little later from L2 ("quantise": Eq. 9 with stochastic rounding, packing), because the
// per-sample (delta, scale) of Eq. 9 depend on every residual of the sample.  Unlike it, no warp ever waits
// for a global load: both reads are bulk asynchronous copies (cp.async.bulk, completion on an mbarrier)
// into two shared-memory rings, issued far ahead by two producer threads, and the worker warps touch
// shared memory only.
//
//   * a CHUNK is a run of G tile row bands of one sample, contiguous in memory (about 28 KB).  Chunks are
//     claimed from a counter in global scratch.  The CTA that claims chunk j brings chunk j into its
//     reduce ring (L2 hint: keep) and chunk j - D into its quantise ring (L2 hint: release), D chunks
//     being at least one sample and about 16 MB of x, which the L2 still holds.
//   * a STRIP is 4 adjacent columns of one band (4 x B elements), owned by one lane: B 16-byte
//     shared-memory loads, column sums in registers, one shuffle to meet the other half of a B = 8 tile.
//     Where a strip sits inside a chunk is the same for every chunk, so it comes from a table built once
//     per CTA.  A UNIT is 32 strips; the units of the chunks are dealt round-robin to the worker warps.
//   * reduce unit: tile mean in the fixed order, stored low-frequency value, extremes of the residual; the
//     last unit of a chunk folds the chunk's extremes into the sample's slot in global scratch and counts
//     the chunk as arrived; the arrival that completes a sample derives (delta, Delta, scale), writes the
//     first two to the blob and publishes delta and scale as one 64-bit word in the slot.
//   * quantise unit: the tile mean is computed again from the staged rows (cheaper than fetching it from
//     the other CTA that stored it), then the 4 codes of each strip row are emitted as one byte (Q = 2),
//     half-word (Q = 4) or word (Q = 8); lanes of a warp write consecutive bytes.  The quantise producer
//     reads the sample's published word before it issues the copy (bounded wait; normally the first look
//     succeeds) and posts it beside the stage.
//
// The launch is cooperative so that all CTAs are resident; no grid-wide barrier is used.  Every wait is
// bounded: when a limit runs out the kernel records DIV_ERR_TIMEOUT in the workspace status word, stops
// waiting everywhere, lets its own copies land and returns.
//
// Why no wait can last: a CTA's workers take units in order, reduce units of a step before its quantise
// unit, and the quantise producer of a CTA that holds claim j waits for the sample of chunk j - D only.
// D is at least a sample, so every chunk of that sample has an index below j: it has been claimed, and
// its claimer is not waiting for it (what a CTA has claimed and not yet reduced lies at or after its own
// j).  By induction over the samples in order, the sample completes.
#pragma once

#include "lagged.cuh"

namespace divk {

#ifndef DIVK_S_WORKER_WARPS
#define DIVK_S_WORKER_WARPS 22
#endif
#ifndef DIVK_S_TARGET_BYTES
#define DIVK_S_TARGET_BYTES (28 * 1024)
#endif
#ifndef DIVK_S_LAG_BYTES
#define DIVK_S_LAG_BYTES (16u << 20)
#endif
constexpr int S_WORKER_WARPS = DIVK_S_WORKER_WARPS;
constexpr int S_THREADS = 32 * (2 + S_WORKER_WARPS);
constexpr int S_MAX_STAGES = 8;
constexpr uint32_t S_CLAIM_RING = 32;

struct SPlan {
    int32_t grid, threads, smem_bytes;
    uint32_t kr, kq;               // stages of the reduce ring / of the quantise ring
    uint32_t G;                    // bands per full chunk
    uint32_t spb;                  // strip slots per band
    uint32_t slots;                // G * spb strip slots per full chunk
    uint32_t nf;                   // units per full chunk
    uint32_t chunk_elems;          // elements of a full chunk
    uint32_t chunks_per_sample;    // S
    uint32_t bands_per_sample;     // C * Hb
    uint32_t stage_bytes;
    uint32_t lag_chunks;           // D
    uint32_t uniform;              // 1: every band has B rows (H % B == 0); 0: chunks are whole planes
    uint64_t total_chunks;
};

struct SParams {
    Shape s;
    SPlan pl;
    FastDiv by_S, by_kr, by_kq;
    const void* x;
    void* lfc;
    void* packed;
    float* stats;
    uint32_t* ws;
    uint64_t seed;
    uint64_t rng_row_step;         // K_GROUP * (W / 4)
    uint64_t timeout_ns;
    uint32_t expected_chunks;      // arrivals that complete a sample (a test may ask for an unreachable count)
    uint32_t tail_rows;
    float inv_cnt[4];              // 1 / (rows * cols) for [tail row band][tail column tile] when a power of two, else 0
    float cnt[4];
};

// what a producer posts beside a stage before it issues the copy
struct SDesc {
    uint32_t nslots;               // strip slots of the chunk (0: the step has no chunk for this ring)
    uint32_t n;                    // sample
    uint32_t tile0;                // first tile of the chunk inside the sample
    uint32_t seq;                  // 1 + the step whose chunk the stage holds; written last (see s_wait_step)
    uint64_t quad0;                // (n * CHW + e0) / 4: first group of 4 elements of the chunk in the tensor
    uint64_t ctr0;                 // counter of the random stream of that group, minus K_GROUP (see rng_group)
    float delta, scale;            // quantise ring only
};

struct SCtl {
    uint64_t full_r[S_MAX_STAGES], empty_r[S_MAX_STAGES];
    uint64_t full_q[S_MAX_STAGES], empty_q[S_MAX_STAGES];
    SDesc desc_r[S_MAX_STAGES], desc_q[S_MAX_STAGES];
    uint32_t kmin[S_MAX_STAGES], kmax[S_MAX_STAGES];      // ~key(min r), key(max r) folded over the units of a chunk
    uint32_t done_r[S_MAX_STAGES], done_q[S_MAX_STAGES];  // units of the chunk that are finished
    uint32_t claims[S_CLAIM_RING];                        // claimed chunk index of step i at [i % S_CLAIM_RING]
    uint32_t claims_n;                                    // steps published by the reduce producer
    uint32_t q_steps;                                     // steps taken over by the quantise producer
    uint32_t end_step;                                    // first step that does not exist (0xFFFFFFFF: not known yet)
    uint32_t failed;
};

__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar,
                                               uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_u32(smem_dst)),
        "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

__device__ __forceinline__ bool s_give_up(const SParams& p, SCtl* ctl, uint64_t& t0) {
    if (lds_volatile(&ctl->failed) || ld_relaxed_u32(p.ws) != 0u) return true;
    const uint64_t t = now_ns();
    if (t0 == 0) t0 = t;
    return t - t0 > p.timeout_ns;
}
__device__ __forceinline__ void s_record_failure(const SParams& p, SCtl* ctl, uint32_t detail) {
    atomicCAS(p.ws, 0u, (uint32_t)DIV_ERR_TIMEOUT);
    atomicCAS(p.ws + 1, 0u, detail);
    sts_volatile(&ctl->failed, 1u);
}
// producer side: bounded wait for a phase of a barrier
__device__ __forceinline__ bool s_wait(uint64_t* bar, uint32_t parity, const SParams& p, SCtl* ctl, uint32_t detail) {
    if (mbar_try_wait(bar, parity)) return true;
    uint32_t polls = 0;
    uint64_t t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 31u) == 0 && s_give_up(p, ctl, t0)) {
            s_record_failure(p, ctl, detail);
            return false;
        }
    }
    return true;
}
// worker side: wait for the chunk of `step`; false when the step does not exist or a wait gave up.
// Worker warps skip steps (units are dealt round-robin), so a warp may look at a stage a whole turn of the
// ring before the producer does, when the barrier's phase of that parity is still the one two turns back,
// which counts as complete.  Hence the sequence number: the parity wait starts only once the producer has
// posted this step's descriptor and its arrival on the barrier.
__device__ __forceinline__ bool s_wait_step(uint64_t* bar, uint32_t parity, const uint32_t* seq, uint32_t step,
                                            const SParams& p, SCtl* ctl) {
    uint32_t polls = 0;
    uint64_t t0 = 0;
    while (lds_volatile(seq) != step + 1u) {
        if (lds_volatile(&ctl->end_step) <= step) return false;
        if ((++polls & 63u) == 0 && s_give_up(p, ctl, t0)) {
            s_record_failure(p, ctl, 0x40000000u | step);
            return false;
        }
    }
    __threadfence_block();
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 63u) == 0 && s_give_up(p, ctl, t0)) {
            s_record_failure(p, ctl, 0x40000000u | step);
            return false;
        }
    }
    return true;
}

// the B rows of a strip from a stage; rows at or past `rows` read as zero (full: every lane has all B rows)
template <typename XT, int P2>
__device__ __forceinline__ void s_load_strip(const unsigned char* xs, uint32_t row_bytes, uint32_t rows, bool full,
                                             uint64_t (&vxy)[P2], uint64_t (&vzw)[P2]) {
    if (full) {
#pragma unroll
        for (int r = 0; r < P2; ++r) StripRow2<XT>::load(xs + r * row_bytes, vxy[r], vzw[r]);
    } else {
#pragma unroll
        for (int r = 0; r < P2; ++r) {
            if ((uint32_t)r < rows) {
                StripRow2<XT>::load(xs + r * row_bytes, vxy[r], vzw[r]);
            } else {
                vxy[r] = 0ull;
                vzw[r] = 0ull;
            }
        }
    }
}

// tile mean in the fixed order (balanced tree down the rows of each of the 4 columns, then across the
// columns of the strip, then across the strips of the tile); every lane of the warp must call it
template <int P2>
__device__ __forceinline__ float s_tile_mean(const uint64_t (&vxy)[P2], const uint64_t (&vzw)[P2], bool active, float inv,
                                             float cnt) {
    constexpr uint32_t LPT = P2 / 4;
    uint64_t cxy[P2 / 2], czw[P2 / 2];
#pragma unroll
    for (int i = 0; i < P2 / 2; ++i) {
        cxy[i] = add2_rn(vxy[2 * i], vxy[2 * i + 1]);
        czw[i] = add2_rn(vzw[2 * i], vzw[2 * i + 1]);
    }
#pragma unroll
    for (int w = P2 / 2; w > 1; w >>= 1) {
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
    if (!active) sum = 0.f;                                 // a padding lane stands for columns past the right edge
#pragma unroll
    for (int m = 1; m < (int)LPT; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
    return (inv != 0.f) ? __fmul_rn(sum, inv) : __fdiv_rn(sum, cnt);
}

template <typename XT, typename LT, int Q, int P2>
__global__ void __launch_bounds__(S_THREADS, 1)
staged_kernel(const SParams p) {
    constexpr uint32_t LPT = P2 / 4;
    constexpr uint32_t QSHIFT = sizeof(XT) == 4 ? 4u : 3u;      // bytes of 4 elements = 1 << QSHIFT
    typedef typename PackedUnit<Q>::type OutT;

    extern __shared__ __align__(128) unsigned char smem[];
    const Shape& s = p.s;
    const uint32_t KR = p.pl.kr, KQ = p.pl.kq;
    const uint32_t stage_bytes = p.pl.stage_bytes;
    unsigned char* ring_r = smem;
    unsigned char* ring_q = smem + (size_t)KR * stage_bytes;
    uint2* table = reinterpret_cast<uint2*>(ring_q + (size_t)KQ * stage_bytes);
    SCtl* ctl = reinterpret_cast<SCtl*>(reinterpret_cast<unsigned char*>(table) + (((size_t)p.pl.slots * 8u + 15u) & ~(size_t)15u));

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t S = p.pl.chunks_per_sample;
    const uint32_t TU = (uint32_t)p.pl.total_chunks;      // < 2^30 (checked by the planner)
    const uint32_t D = p.pl.lag_chunks;

    // ---- set-up: strip table, barriers ----
    //   x: offset of the strip's first element inside the chunk, in groups of 4 elements
    //   y: in-bounds rows (0: padding slot) | kind of tile << 4 | writes the tile's mean << 6 | tile inside the chunk << 8
    for (uint32_t sl = threadIdx.x; sl < p.pl.slots; sl += blockDim.x) {
        const uint32_t band = sl / p.pl.spb, q = sl - band * p.pl.spb;
        const uint32_t col0 = 4u * q;
        const bool ok = col0 < s.W;
        uint32_t eoff, rows;
        if (p.pl.uniform) {
            eoff = band * s.B * s.W + col0;
            rows = s.B;
        } else {
            const uint32_t pl_ = band / s.Hb, bh = band - pl_ * s.Hb;
            eoff = pl_ * s.HW + bh * s.B * s.W + col0;
            rows = (bh + 1u == s.Hb) ? p.tail_rows : s.B;
        }
        const uint32_t bw = q / LPT;
        const uint32_t which = ((rows != s.B) ? 2u : 0u) + ((bw == s.Wb - 1u && (s.W % s.B) != 0u) ? 1u : 0u);
        const uint32_t writer = (q % LPT) == 0 ? 1u : 0u;
        table[sl] = make_uint2(ok ? (eoff >> 2) : 0u, (ok ? rows : 0u) | (which << 4) | (writer << 6) | ((band * s.Wb + bw) << 8));
    }
    if (threadIdx.x == 0) {
        for (uint32_t i = 0; i < (uint32_t)S_MAX_STAGES; ++i) {
            mbar_init(&ctl->full_r[i], 1);
            mbar_init(&ctl->empty_r[i], 1);
            mbar_init(&ctl->full_q[i], 1);
            mbar_init(&ctl->empty_q[i], 1);
            ctl->kmin[i] = 0;
            ctl->kmax[i] = 0;
            ctl->done_r[i] = 0;
            ctl->done_q[i] = 0;
            ctl->desc_r[i].seq = 0;
            ctl->desc_q[i].seq = 0;
        }
        ctl->claims_n = 0;
        ctl->q_steps = 0;
        ctl->end_step = 0xFFFFFFFFu;
        ctl->failed = 0;
        fence_barrier_init();
    }
    __syncthreads();

    if (warp == 0) {
        // ================= reduce producer: claims chunks, streams them from HBM =================
        if (lane == 0) {
            uint32_t* claim_word = p.ws + WS_CLAIM_WORD;
            const uint64_t pol_keep = l2_policy_keep();
            uint32_t i = 0;
            uint32_t j = atomicAdd(claim_word, 1u);
            bool ok = true;
            while (j < TU + D) {
                const uint32_t jn = atomicAdd(claim_word, 1u);          // needed only at the next turn
                // hand the claim to the quantise producer
                {
                    uint32_t polls = 0;
                    uint64_t t0 = 0;
                    while (i - lds_volatile(&ctl->q_steps) >= S_CLAIM_RING) {
                        if ((++polls & 31u) == 0 && s_give_up(p, ctl, t0)) {
                            s_record_failure(p, ctl, 0x80000001u);
                            ok = false;
                            break;
                        }
                    }
                    if (!ok) break;
                }
                ctl->claims[i % S_CLAIM_RING] = j;
                __threadfence_block();
                sts_volatile(&ctl->claims_n, i + 1u);
                const uint32_t round = fdiv(i, p.by_kr);
                const uint32_t st = i - round * KR;
                if (i >= KR && !s_wait(&ctl->empty_r[st], (round - 1u) & 1u, p, ctl, 0x80000002u)) {
                    ok = false;
                    break;
                }
                SDesc d;
                d.nslots = 0;
                d.n = 0;
                d.tile0 = 0;
                d.seq = 0;
                d.quad0 = 0;
                d.ctr0 = 0;
                d.delta = 0.f;
                d.scale = 0.f;
                if (j < TU) {
                    const uint32_t n = fdiv(j, p.by_S);
                    const uint32_t k = j - n * S;
                    const uint32_t e0 = k * p.pl.chunk_elems;
                    const uint32_t nelem = min(p.pl.chunk_elems, s.CHW - e0);
                    const uint32_t nbands = min(p.pl.G, p.pl.bands_per_sample - k * p.pl.G);
                    d.nslots = nbands * p.pl.spb;
                    d.n = n;
                    d.tile0 = k * p.pl.G * s.Wb;
                    ctl->desc_r[st] = d;
                    const uint32_t bytes = nelem * (uint32_t)sizeof(XT);
                    const XT* src = reinterpret_cast<const XT*>(p.x) + ((size_t)n * s.CHW + e0);
                    mbar_arrive_expect_tx(&ctl->full_r[st], bytes);
                    bulk_load_hint(ring_r + (size_t)st * stage_bytes, src, bytes, &ctl->full_r[st], pol_keep);
                } else {
                    ctl->desc_r[st] = d;
                    mbar_arrive(&ctl->full_r[st]);
                }
                __threadfence_block();
                sts_volatile(&ctl->desc_r[st].seq, i + 1u);
                ++i;
                j = jn;
            }
            __threadfence_block();
            sts_volatile(&ctl->end_step, i);
            if (!ok || lds_volatile(&ctl->failed)) {
                // a wait gave up somewhere: let the copies still in flight land before the CTA may exit
                const uint32_t first = i > KR ? i - KR : 0u;
                for (uint32_t t = first; t < i; ++t) {
                    const uint32_t round = fdiv(t, p.by_kr);
                    uint32_t polls = 0;
                    while (!mbar_try_wait(&ctl->full_r[t - round * KR], round & 1u) && ++polls < (1u << 20)) {
                    }
                }
            }
        }
        return;
    }

    if (warp == 1) {
        // ================= quantise producer: chunk j - D from L2, with its sample's parameters =================
        if (lane == 0) {
            const uint64_t pol_release = l2_policy_release();
            uint32_t i = 0;
            bool ok = true;
            uint64_t pre_word = 0;          // parameter word looked up ahead of time for step pre_step
            uint32_t pre_step = 0xFFFFFFFFu;
            while (true) {
                // the claim of step i
                {
                    uint32_t polls = 0;
                    uint64_t t0 = 0;
                    bool ended = false;
                    while (lds_volatile(&ctl->claims_n) <= i) {
                        if (lds_volatile(&ctl->end_step) <= i) {
                            ended = true;
                            break;
                        }
                        if ((++polls & 31u) == 0 && s_give_up(p, ctl, t0)) {
                            s_record_failure(p, ctl, 0x80000003u);
                            ok = false;
                            break;
                        }
                    }
                    if (ended || !ok) break;
                }
                __threadfence_block();
                const uint32_t j = ctl->claims[i % S_CLAIM_RING];
                // look ahead: the claim of the next step, if it is there already
                uint32_t jnext = 0xFFFFFFFFu;
                if (lds_volatile(&ctl->claims_n) > i + 1u) jnext = ctl->claims[(i + 1u) % S_CLAIM_RING];
                __threadfence_block();
                sts_volatile(&ctl->q_steps, i + 1u);

                const bool has = j >= D && j - D < TU;
                uint32_t n = 0, k = 0;
                uint64_t word = 0;
                if (has) {
                    n = fdiv(j - D, p.by_S);
                    k = (j - D) - n * S;
                    const uint64_t* pw = reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS + 4);
                    word = (pre_step == i) ? pre_word : ld_relaxed_u64(pw);
                }
                // issue the look-up for the next step now; its answer is used a turn later
                if (jnext != 0xFFFFFFFFu && jnext >= D && jnext - D < TU) {
                    const uint32_t nn = fdiv(jnext - D, p.by_S);
                    pre_word = ld_relaxed_u64(reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)nn * WS_SLOT_WORDS + 4));
                    pre_step = i + 1u;
                }
                const uint32_t round = fdiv(i, p.by_kq);
                const uint32_t st = i - round * KQ;
                if (i >= KQ && !s_wait(&ctl->empty_q[st], (round - 1u) & 1u, p, ctl, 0x80000004u)) {
                    ok = false;
                    break;
                }
                SDesc d;
                d.nslots = 0;
                d.n = 0;
                d.tile0 = 0;
                d.seq = 0;
                d.quad0 = 0;
                d.ctr0 = 0;
                d.delta = 0.f;
                d.scale = 0.f;
                if (has) {
                    if (!(word >> 63)) {
                        const uint64_t* pw = reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS + 4);
                        uint32_t polls = 0;
                        uint64_t t0 = 0;
                        while (true) {
                            word = ld_relaxed_u64(pw);
                            if (word >> 63) break;
                            if ((++polls & 7u) == 0 && s_give_up(p, ctl, t0)) {
                                s_record_failure(p, ctl, n + 1u);
                                ok = false;
                                break;
                            }
                            __nanosleep(100);
                        }
                        if (!ok) break;
                    }
                    const uint32_t e0 = k * p.pl.chunk_elems;
                    const uint32_t nelem = min(p.pl.chunk_elems, s.CHW - e0);
                    const uint32_t nbands = min(p.pl.G, p.pl.bands_per_sample - k * p.pl.G);
                    d.nslots = nbands * p.pl.spb;
                    d.n = n;
                    d.tile0 = k * p.pl.G * s.Wb;
                    d.quad0 = ((uint64_t)n * s.CHW + e0) >> 2;
                    d.ctr0 = rng_sample_base(p.seed, n) + K_GROUP * (uint64_t)((e0 >> 2) + 1u);
                    d.delta = __uint_as_float((uint32_t)word);
                    d.scale = __uint_as_float((uint32_t)(word >> 32) & 0x7FFFFFFFu);
                    ctl->desc_q[st] = d;
                    const uint32_t bytes = nelem * (uint32_t)sizeof(XT);
                    const XT* src = reinterpret_cast<const XT*>(p.x) + ((size_t)n * s.CHW + e0);
                    mbar_arrive_expect_tx(&ctl->full_q[st], bytes);
                    bulk_load_hint(ring_q + (size_t)st * stage_bytes, src, bytes, &ctl->full_q[st], pol_release);
                } else {
                    ctl->desc_q[st] = d;
                    mbar_arrive(&ctl->full_q[st]);
                }
                __threadfence_block();
                sts_volatile(&ctl->desc_q[st].seq, i + 1u);
                ++i;
            }
            if (!ok || lds_volatile(&ctl->failed)) {
                const uint32_t first = i > KQ ? i - KQ : 0u;
                for (uint32_t t = first; t < i; ++t) {
                    const uint32_t round = fdiv(t, p.by_kq);
                    uint32_t polls = 0;
                    while (!mbar_try_wait(&ctl->full_q[t - round * KQ], round & 1u) && ++polls < (1u << 20)) {
                    }
                }
            }
        }
        return;
    }

    // ================= workers =================
    const uint32_t NW = (blockDim.x >> 5) - 2;
    const uint32_t nf = p.pl.nf;
    const uint32_t row_bytes = s.W * (uint32_t)sizeof(XT);
    const uint32_t W4 = s.W >> 2;
    LT* lfc_out = reinterpret_cast<LT*>(p.lfc);
    OutT* packed = reinterpret_cast<OutT*>(p.packed);

    // unit k of step `step`: k < nf reduce unit k, else quantise unit k - nf
    uint32_t step = 0, k = warp - 2;
    while (k >= 2u * nf) {
        k -= 2u * nf;
        ++step;
    }

    while (true) {
        if (k < nf) {
            // ---------------- reduce unit ----------------
            const uint32_t round = fdiv(step, p.by_kr);
            const uint32_t st = step - round * KR;
            if (!s_wait_step(&ctl->full_r[st], round & 1u, &ctl->desc_r[st].seq, step, p, ctl)) break;
            // every unit index of the step takes part in the closing count, also where a short chunk has no
            // strips for it: a stage is recycled only after each of its nf readers has looked at it
            const uint32_t nslots = ctl->desc_r[st].nslots;
            const bool work = k * 32u < nslots;
            {
                uint32_t kmin = 0, kmax = 0;
                if (work) {
                    const uint32_t n = ctl->desc_r[st].n;
                    const uint32_t sl = k * 32u + lane;
                    uint2 rec = make_uint2(0u, 0u);
                    if (sl < nslots) rec = table[sl];
                    const uint32_t rows = rec.y & 15u;
                    const bool active = rows != 0u;
                    const uint32_t which = (rec.y >> 4) & 3u;
                    const unsigned char* xs = ring_r + (size_t)st * stage_bytes + ((size_t)rec.x << QSHIFT);
                    const bool full = __all_sync(0xFFFFFFFFu, rows == (uint32_t)P2 || rows == 0u);
                    uint64_t vxy[P2], vzw[P2];
                    s_load_strip<XT, P2>(xs, row_bytes, rows, full, vxy, vzw);
                    const float mean = s_tile_mean<P2>(vxy, vzw, active, p.inv_cnt[which], p.cnt[which]);
                    const float stored = Elem<LT>::round(mean);
                    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
                    if (active) {
                        if (rec.y & 64u)
                            Elem<LT>::store(lfc_out + (size_t)n * s.C * s.TPP + ctl->desc_r[st].tile0 + (rec.y >> 8), mean);
                        // extremes of x over the strip's in-bounds rows; x -> fl(x - stored) is monotone
                        float blo = 3.402823466e+38f, bhi = -3.402823466e+38f;
#pragma unroll
                        for (int r = 0; r < P2; ++r) {
                            if (full || (uint32_t)r < rows) {
                                float a_, b_, c_, d_;
                                upk2(vxy[r], a_, b_);
                                upk2(vzw[r], c_, d_);
                                blo = fmin3(blo, a_, b_);
                                blo = fmin3(blo, c_, d_);
                                bhi = fmax3(bhi, a_, b_);
                                bhi = fmax3(bhi, c_, d_);
                            }
                        }
                        lo = __fsub_rn(blo, stored);
                        hi = __fsub_rn(bhi, stored);
                    }
                    kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
                    kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
                }
                __syncwarp();
                if (lane == 0) {
                    if (work) {
                        atomicMax(&ctl->kmin[st], kmin);
                        atomicMax(&ctl->kmax[st], kmax);
                        __threadfence_block();
                    }
                    if (atomicAdd(&ctl->done_r[st], 1u) == nf - 1u) {
                        // last unit of this chunk: fold the chunk into its sample's slot, hand the stage back
                        __threadfence_block();
                        const uint32_t smin = atomicExch(&ctl->kmin[st], 0u);
                        const uint32_t smax = atomicExch(&ctl->kmax[st], 0u);
                        ctl->done_r[st] = 0u;
                        if (nslots && lds_volatile(&ctl->failed) == 0u) {
                            const uint32_t n = ctl->desc_r[st].n;
                            uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
                            red_max_relaxed(slot + 0, smin);
                            red_max_relaxed(slot + 1, smax);
                            const uint32_t before = atom_add_acq_rel(slot + 2, 1u);
                            if (before + 1u == p.expected_chunks) {
                                // this arrival completes the sample
                                const QParams qp = make_qparams(key_float(~ld_relaxed_u32(slot + 0)), key_float(ld_relaxed_u32(slot + 1)), Q);
                                p.stats[2 * (size_t)n + 0] = qp.delta;
                                p.stats[2 * (size_t)n + 1] = qp.step;
                                const uint64_t word = ((uint64_t)(__float_as_uint(qp.scale) | 0x80000000u) << 32) |
                                                      (uint64_t)__float_as_uint(qp.delta);
                                st_release_u64(reinterpret_cast<uint64_t*>(slot + 4), word);
                            }
                        }
                        __threadfence_block();
                        mbar_arrive(&ctl->empty_r[st]);
                    }
                }
            }
        } else {
            // ---------------- quantise unit ----------------
            const uint32_t kk = k - nf;
            const uint32_t round = fdiv(step, p.by_kq);
            const uint32_t st = step - round * KQ;
            if (!s_wait_step(&ctl->full_q[st], round & 1u, &ctl->desc_q[st].seq, step, p, ctl)) break;
            const uint32_t nslots = ctl->desc_q[st].nslots;
            {
                if (kk * 32u < nslots) {
                    const uint32_t sl = kk * 32u + lane;
                    uint2 rec = make_uint2(0u, 0u);
                    if (sl < nslots) rec = table[sl];
                    const uint32_t rows = rec.y & 15u;
                    const bool active = rows != 0u;
                    const uint32_t which = (rec.y >> 4) & 3u;
                    const unsigned char* xs = ring_q + (size_t)st * stage_bytes + ((size_t)rec.x << QSHIFT);
                    const bool full = __all_sync(0xFFFFFFFFu, rows == (uint32_t)P2 || rows == 0u);
                    uint64_t vxy[P2], vzw[P2];
                    s_load_strip<XT, P2>(xs, row_bytes, rows, full, vxy, vzw);
                    const float mean = s_tile_mean<P2>(vxy, vzw, active, p.inv_cnt[which], p.cnt[which]);
                    const float stored = Elem<LT>::round(mean);
                    if (active) {
                        const float delta = ctl->desc_q[st].delta, scale = ctl->desc_q[st].scale;
                        const uint64_t stored2 = pk2(stored, stored);
                        const uint64_t delta2 = pk2(delta, delta), scale2 = pk2(scale, scale);
                        uint64_t ctr = ctl->desc_q[st].ctr0 + K_GROUP * (uint64_t)rec.x;
                        OutT* out = packed + ctl->desc_q[st].quad0 + rec.x;
                        if (full) {
#pragma unroll
                            for (int r = 0; r < P2; ++r) {
                                *out = (OutT)quant_row<Q>(vxy[r], vzw[r], stored2, delta2, scale2, rng_mix(ctr));
                                out += W4;
                                ctr += p.rng_row_step;
                            }
                        } else {
#pragma unroll
                            for (int r = 0; r < P2; ++r) {
                                if ((uint32_t)r < rows) {
                                    *out = (OutT)quant_row<Q>(vxy[r], vzw[r], stored2, delta2, scale2, rng_mix(ctr));
                                    out += W4;
                                    ctr += p.rng_row_step;
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    if (atomicAdd(&ctl->done_q[st], 1u) == nf - 1u) {
                        ctl->done_q[st] = 0u;
                        __threadfence_block();
                        mbar_arrive(&ctl->empty_q[st]);
                    }
                }
            }
        }
        k += NW;
        while (k >= 2u * nf) {
            k -= 2u * nf;
            ++step;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
inline uint32_t lcm_u32(uint32_t a, uint32_t b) { return a / gcd_u32(a, b) * b; }

inline div_status plan_staged(const div_desc* d, const Shape& s, SPlan* out) {
    const uint32_t sx = d->x_dtype == DIV_F32 ? 4u : 2u;
    if (s.W % 4 != 0) return DIV_ERR_PARAM;
    if (!(s.B == 4 || s.B == 8) || s.P2 != s.B) return DIV_ERR_PARAM;
    if (!(d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return DIV_ERR_PARAM;
    // bulk copies start on 16-byte boundaries and move multiples of 16 bytes
    if (((uint64_t)s.CHW * sx) % 16u != 0 || ((uint64_t)s.HW * sx) % 16u != 0 || ((uint64_t)s.B * s.W * sx) % 16u != 0)
        return DIV_ERR_PARAM;
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return DIV_ERR_CUDA;

    SPlan pl = SPlan();
    pl.spb = s.Wb * (s.P2 / 4);
    const uint64_t bands = (uint64_t)s.C * s.Hb;
    if (bands >= (1ull << 31)) return DIV_ERR_PARAM;
    pl.bands_per_sample = (uint32_t)bands;
    pl.uniform = (s.H % s.B == 0) ? 1u : 0u;
    // bands per chunk: a count that keeps the chunk's inner geometry the same for every chunk (any count when
    // all bands are alike, whole planes otherwise) and, where possible, fills whole units of 32 strips
    const uint32_t geo = pl.uniform ? 1u : s.Hb;
    const uint64_t geo_bytes = pl.uniform ? (uint64_t)s.B * s.W * sx : (uint64_t)s.HW * sx;     // bytes of `geo` bands
    const uint32_t fill = 32u / gcd_u32(32u, pl.spb);
    const uint32_t both = lcm_u32(geo, fill);
    const uint64_t both_bytes = geo_bytes * (both / geo);
    const uint64_t target = DIVK_S_TARGET_BYTES;
    uint32_t G;
    if (both_bytes <= target) G = (uint32_t)(target / both_bytes) * both;
    else if (geo_bytes <= target) G = (uint32_t)(target / geo_bytes) * geo;
    else return DIV_ERR_PARAM;
    const uint32_t bands_up = (pl.bands_per_sample + geo - 1u) / geo * geo;
    if (G > bands_up) G = bands_up;
    pl.G = G;
    pl.slots = G * pl.spb;
    if (pl.slots > 4096u) return DIV_ERR_PARAM;
    pl.nf = (pl.slots + 31u) / 32u;
    pl.chunk_elems = pl.uniform ? G * s.B * s.W : (G / s.Hb) * s.HW;
    if (pl.chunk_elems >= (1u << 20)) return DIV_ERR_PARAM;
    pl.chunks_per_sample = (pl.bands_per_sample + G - 1u) / G;
    pl.stage_bytes = (pl.chunk_elems * sx + 127u) & ~127u;
    const uint32_t fixed = ((pl.slots * 8u + 15u) & ~15u) + (uint32_t)sizeof(SCtl) + 256u;
    if ((uint32_t)di.smem_optin < fixed + 4u * pl.stage_bytes + 1024u) return DIV_ERR_PARAM;
    uint32_t stages = ((uint32_t)di.smem_optin - 1024u - fixed) / pl.stage_bytes;
    if (stages > 2u * S_MAX_STAGES) stages = 2u * S_MAX_STAGES;
    uint32_t kq = (stages * 3u + 4u) / 8u;
    if (kq < 2u) kq = 2u;
    if (kq > (uint32_t)S_MAX_STAGES) kq = S_MAX_STAGES;
    uint32_t kr = stages - kq;
    if (kr > (uint32_t)S_MAX_STAGES) kr = S_MAX_STAGES;
    if (kr < 2u) return DIV_ERR_PARAM;
    pl.kr = kr;
    pl.kq = kq;
    pl.smem_bytes = (int32_t)((kr + kq) * pl.stage_bytes + fixed);
    pl.total_chunks = (uint64_t)pl.chunks_per_sample * s.N;
    // lag: at least a whole sample (see the progress argument at the top), and about DIVK_S_LAG_BYTES of x
    const uint64_t chunk_bytes = (uint64_t)pl.chunk_elems * sx;
    uint64_t lag = (DIVK_S_LAG_BYTES + chunk_bytes - 1) / chunk_bytes;
    if (lag < (uint64_t)pl.chunks_per_sample + 2u) lag = (uint64_t)pl.chunks_per_sample + 2u;
    if (lag > pl.total_chunks) lag = pl.total_chunks;     // a tensor smaller than the span: reduce everything, then quantise
    uint64_t grid = (uint64_t)di.sms;
    if (grid > pl.total_chunks) grid = pl.total_chunks;
    pl.grid = (int32_t)grid;
    pl.threads = S_THREADS;
    // chunk indices and the claim counter are 32-bit on the device (every CTA overshoots by two claims)
    if (pl.total_chunks + lag + 2u * grid >= (1ull << 30)) return DIV_ERR_PARAM;
    pl.lag_chunks = (uint32_t)lag;
    *out = pl;
    return DIV_OK;
}

template <typename XT, typename LT, int Q, int P2>
inline div_status launch_staged(const SParams& prm, cudaStream_t st) {
    auto kern = staged_kernel<XT, LT, Q, P2>;
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
inline div_status launch_staged_q(int qbits, uint32_t p2, const SParams& prm, cudaStream_t st) {
    if (p2 == 8) {
        if (qbits == 2) return launch_staged<XT, LT, 2, 8>(prm, st);
        if (qbits == 4) return launch_staged<XT, LT, 4, 8>(prm, st);
        if (qbits == 8) return launch_staged<XT, LT, 8, 8>(prm, st);
    } else if (p2 == 4) {
        if (qbits == 2) return launch_staged<XT, LT, 2, 4>(prm, st);
        if (qbits == 4) return launch_staged<XT, LT, 4, 4>(prm, st);
        if (qbits == 8) return launch_staged<XT, LT, 8, 4>(prm, st);
    }
    return DIV_ERR_PARAM;
}

inline div_status compress_staged(const div_desc* d, const Shape& s, const div_layout& lo, const SPlan& pl,
                                  const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st,
                                  uint32_t expected_chunks = 0, uint64_t timeout_ns = 0) {
    SParams prm;
    prm.s = s;
    prm.pl = pl;
    prm.by_S = host_fastdiv(pl.chunks_per_sample);
    prm.by_kr = host_fastdiv(pl.kr);
    prm.by_kq = host_fastdiv(pl.kq);
    prm.x = x;
    prm.lfc = blob + lo.lfc_off;
    prm.packed = blob + lo.packed_off;
    prm.stats = reinterpret_cast<float*>(blob + lo.stats_off);
    prm.ws = ws;
    prm.seed = seed;
    prm.rng_row_step = K_GROUP * (uint64_t)(s.W / 4u);
    prm.timeout_ns = timeout_ns ? timeout_ns : 2000000000ull;
    prm.expected_chunks = expected_chunks ? expected_chunks : pl.chunks_per_sample;
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
        if (d->lfc_dtype == DIV_F32) return launch_staged_q<float, float>(d->qbits, s.P2, prm, st);
        return launch_staged_q<float, bf16>(d->qbits, s.P2, prm, st);
    }
    if (d->lfc_dtype == DIV_F32) return launch_staged_q<bf16, float>(d->qbits, s.P2, prm, st);
    return launch_staged_q<bf16, bf16>(d->qbits, s.P2, prm, st);
}

}  // namespace divk
