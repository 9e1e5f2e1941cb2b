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
//   * a CHUNK is a run of G tile row bands of one sample, contiguous in memory (about 28 KB).  Chunk j
//     belongs to CTA j mod gridDim.x, so the CTAs sweep the tensor together, one round of gridDim.x chunks
//     after the other.  A CTA brings its i-th chunk into its reduce ring (L2 hint: keep) and, L rounds
//     later, the same chunk into its quantise ring (L2 hint: release).  L rounds are at least a sample
//     plus a round, and about 16 MB of x, which the L2 still holds.
//   * a STRIP is 4 adjacent columns of one band (4 x B elements), owned by one lane: B 16-byte
//     shared-memory loads, column sums in registers, one shuffle to meet the other half of a B = 8 tile.
//     Where a strip sits inside a chunk is the same for every chunk, so it comes from a table built once
//     per CTA.  A UNIT is 32 strips.  A CTA's work is the sequence of steps s = 0, 1, ...: the reduce units
//     of its chunk s, then the quantise units of its chunk s - L; the units are dealt round-robin to the
//     worker warps, each of which takes its units in order.
//   * reduce unit: tile mean in the fixed order, stored low-frequency value, extremes of the residual; the
//     last unit of a chunk folds the chunk's extremes into the sample's slot in global scratch and counts
//     the chunk as arrived (the count is sent by the CTA's watcher thread, behind a release fence).  The
//     watcher also polls the counts of the samples blockIdx.x, blockIdx.x + gridDim.x, ...; when a sample is
//     complete it derives (delta, Delta, scale), writes the first two to the blob and publishes delta and
//     scale as one 64-bit word in the slot.
//   * quantise unit: the tile mean is computed again from the staged rows, then the 4 codes of each strip
//     row are emitted as one byte (Q = 2), half-word (Q = 4) or word (Q = 8); lanes of a warp write
//     consecutive bytes.  The quantise producer reads the sample's published word before it issues the
//     copy (bounded wait; the look-up is started two chunks ahead, so normally it has long arrived) and
//     posts it beside the stage.
//
// The launch is cooperative so that all CTAs are resident; no grid-wide barrier is used.  Every wait is
// bounded: when a limit runs out the kernel records DIV_ERR_TIMEOUT in the workspace status word, stops
// waiting everywhere, lets its own copies land and returns.
//
// Why no wait can last: the watchers wait for counts and nobody waits for them but the quantise producers;
// the only other wait on other CTAs is the quantise producer's, for the sample of its chunk s - L.  The chunks of that sample lie in rounds up to s - L + ceil((S - 1) / gridDim.x) <= s - 1 (S chunks
// per sample; L is chosen that large).  Take the first sample that is not complete and one of its chunks
// that has not been reduced, chunk t of CTA Y.  Y's reduce producer issues its copies in order and waits only
// for its own workers; Y's workers take units in order, and the only thing they can be stuck on is a
// quantise chunk that Y's quantise producer has not issued, chunk u - L with u <= t.  But that producer waits
// for a sample whose chunks all lie in rounds before u, i.e. for an earlier sample, which is complete.
#pragma once

#include "lagged.cuh"

namespace divk {

#ifndef DIVK_S_WORKER_WARPS
#define DIVK_S_WORKER_WARPS 29
#endif
#ifndef DIVK_S_AHEAD
#define DIVK_S_AHEAD 4
#endif
#ifndef DIVK_S_Q_STAGES_PER_8
#define DIVK_S_Q_STAGES_PER_8 4
#endif
#ifndef DIVK_S_REDUCE_WARPS
#define DIVK_S_REDUCE_WARPS 14
#endif
#ifndef DIVK_S_TARGET_BYTES
#define DIVK_S_TARGET_BYTES (28 * 1024)
#endif
#ifndef DIVK_S_LAG_BYTES
#define DIVK_S_LAG_BYTES (48u << 20)
#endif
constexpr int S_WORKER_WARPS = DIVK_S_WORKER_WARPS;
constexpr int S_REDUCE_WARPS = DIVK_S_REDUCE_WARPS;      // of the worker warps
static_assert(S_REDUCE_WARPS >= 1 && S_REDUCE_WARPS < S_WORKER_WARPS, "both worker classes need a warp");
constexpr int S_SERVICE_WARPS = 3;          // reduce producer, quantise producer, watcher
constexpr int S_THREADS = 32 * (S_SERVICE_WARPS + S_WORKER_WARPS);
constexpr int S_MAX_STAGES = 8;
constexpr uint32_t S_MAILBOX = 16;
constexpr int S_AHEAD = DIVK_S_AHEAD;       // chunks the reduce half may lead the quantise half by, beyond the lag

struct SPlan {
    int32_t grid, threads, smem_bytes;
    uint32_t kr, kq;               // stages of the reduce ring / of the quantise ring
    uint32_t G;                    // bands per full chunk
    uint32_t spb;                  // strip slots per band
    uint32_t paired;               // 1: bands are laid out in pairs, their single-strip last tiles side by side (see the table)
    uint32_t slots;                // G * spb strip slots per full chunk
    uint32_t nf;                   // units per full chunk
    uint32_t chunk_elems;          // elements of a full chunk
    uint32_t chunks_per_sample;    // S
    uint32_t bands_per_sample;     // C * Hb
    uint32_t stage_bytes;
    uint32_t lag_steps;            // L: rounds between the reduce and the quantise half of a chunk
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
    uint32_t ntiles;               // tiles of the chunk (a short last chunk of a sample has fewer)
    uint32_t n;                    // sample
    uint32_t tile0;                // first tile of the chunk inside the sample
    uint32_t seq;                  // 1 + index (in this CTA's list) of the chunk the stage holds; written last (see s_wait_chunk)
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
    uint32_t q_closed;                                    // chunks whose quantise half is finished
    uint32_t mb_n[S_MAILBOX], mb_seq[S_MAILBOX];          // reduce closers -> watcher: chunk it of this CTA (slot it % S_MAILBOX)
                                                          // has been folded into sample mb_n; mb_seq = it + 1, written last
    uint32_t mb_done;                                     // chunks the watcher has counted
    uint32_t failed;
};

__device__ __forceinline__ void red_add_relaxed(uint32_t* p, uint32_t v) {
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar,
                                               uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_u32(smem_dst)),
        "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// Bounded waits.  The polling loops below stay on chip: a look at the clock every few polls, and only once a
// wait has lasted S_SLOW_CYCLES (far longer than any wait of a healthy run) the slow check, which reads the
// status word in global memory (has any wait of this launch given up?) and the wall clock.
constexpr long long S_SLOW_CYCLES = 1ll << 15;
struct SWait {
    long long c0;        // clock at the last slow check (0: none yet)
    uint64_t t0;         // wall clock at the first slow check
};
__device__ __forceinline__ bool s_give_up(const SParams& p, SCtl* ctl, SWait& w) {
    const long long c = clock64();
    if (w.c0 == 0) {
        w.c0 = c;
        w.t0 = 0;
        return false;
    }
    if (c - w.c0 < S_SLOW_CYCLES) return false;
    w.c0 = c;
    if (lds_volatile(&ctl->failed) || ld_relaxed_u32(p.ws) != 0u) return true;
    const uint64_t t = now_ns();
    if (w.t0 == 0) w.t0 = t;
    return t - w.t0 > p.timeout_ns;
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
    SWait w = {0, 0};
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 7u) == 0 && s_give_up(p, ctl, w)) {
            s_record_failure(p, ctl, detail);
            return false;
        }
    }
    return true;
}
// worker side: wait for the CTA's chunk number `it` in a ring; false when a wait gave up.
// Worker warps skip chunks (units are dealt round-robin), so a warp may look at a stage a whole turn of the
// ring before the producer does, when the barrier's phase of that parity is still the one two turns back,
// which counts as complete.  Hence the sequence number: the parity wait starts only once the producer has
// posted this chunk's descriptor and its arrival on the barrier.
__device__ __forceinline__ bool s_wait_chunk(uint64_t* bar, uint32_t parity, const uint32_t* seq, uint32_t it,
                                             const SParams& p, SCtl* ctl) {
    uint32_t polls = 0;
    SWait w = {0, 0};
    while (lds_volatile(seq) != it + 1u) {
        __nanosleep(32);
        if ((++polls & 7u) == 0 && s_give_up(p, ctl, w)) {
            s_record_failure(p, ctl, 0x40000000u | it);
            return false;
        }
    }
    __threadfence_block();
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 7u) == 0 && s_give_up(p, ctl, w)) {
            s_record_failure(p, ctl, 0x40000000u | it);
            return false;
        }
    }
    return true;
}

// the B rows of a strip from a stage; rows at or past `rows` read as zero (full: every lane has all B rows)
template <typename XT, int P2>
__device__ __forceinline__ void s_load_strip(const unsigned char* xs, uint32_t row_bytes, uint32_t rows, bool full,
                                             uint32_t rmax, uint64_t (&vxy)[P2], uint64_t (&vzw)[P2]) {
    if (full) {
#pragma unroll
        for (int r = 0; r < P2; ++r) StripRow2<XT>::load(xs + r * row_bytes, vxy[r], vzw[r]);
    } else {
#pragma unroll
        for (int r = 0; r < P2; ++r) {
            vxy[r] = 0ull;
            vzw[r] = 0ull;
            // rmax, the largest row count in the warp, is the same in every lane: a unit of short bands only
            // steps over its missing rows without issuing anything for them
            if ((uint32_t)r < rmax) {
                if ((uint32_t)r < rows) StripRow2<XT>::load(xs + r * row_bytes, vxy[r], vzw[r]);
            }
        }
    }
}

// tile mean in the fixed order (balanced tree down the rows of each of the 4 columns, then across the
// columns of the strip, then across the strips of the tile); every lane of the warp must call it
template <int P2>
__device__ __forceinline__ float s_tile_mean(const uint64_t (&vxy)[P2], const uint64_t (&vzw)[P2], bool active, bool mate,
                                             float inv, float cnt) {
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
    if (LPT == 2u) {
        // the tile's other strip is next door; a tile of one strip adds the zero its missing columns stand for
        const float other = __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
        sum = __fadd_rn(sum, mate ? other : 0.f);
    }
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
    uint32_t* table = reinterpret_cast<uint32_t*>(ring_q + (size_t)KQ * stage_bytes);
    SCtl* ctl = reinterpret_cast<SCtl*>(reinterpret_cast<unsigned char*>(table) + (((size_t)p.pl.slots * 4u + 15u) & ~(size_t)15u));

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t S = p.pl.chunks_per_sample;
    const uint32_t TU = (uint32_t)p.pl.total_chunks;      // < 2^30 (checked by the planner)
    const uint32_t L = p.pl.lag_steps;
    const uint32_t G = gridDim.x;
    // this CTA's chunks: blockIdx.x + it * G for it < n_my
    const uint32_t n_my = blockIdx.x < TU ? (TU - blockIdx.x + G - 1u) / G : 0u;

    // ---- set-up: strip table, barriers ----
    // One entry per strip slot of a full chunk; slot sl is lane sl % 32 of unit sl / 32.
    //   bits 0-12 offset of the strip's first element inside the chunk, in groups of 4 elements; 13-16 in-bounds rows
    //   (0: padding slot); 17-18 kind of tile; 19 writes the tile's mean (first strip of its tile); 20 the tile has a
    //   second strip, held by the lane next door (lane ^ 1); 21-31 tile inside the chunk.
    // Order of the slots: bands of full height first, then the short last bands of the planes, so that most units
    // hold strips of one height only.  Inside a band the strips follow each other, 2 per tile for B = 8.  Where W / 4
    // is odd the last tile of a band has one strip; bands are then laid out in pairs, their two-strip tiles first and
    // the two single strips side by side, so that every two-strip tile starts on an even lane and no lane is idle.
    {
        const uint32_t spr = s.W >> 2;                                       // strips per band that exist
        const uint32_t full_bands = p.pl.uniform ? p.pl.G : (p.pl.G / s.Hb) * (s.Hb - 1u);
        for (uint32_t sl = threadIdx.x; sl < p.pl.slots; sl += blockDim.x) {
            uint32_t ob, q;                                                  // band in the order above, strip inside the band
            if (p.pl.paired) {
                const uint32_t pair = sl / (2u * spr), r = sl - pair * 2u * spr;
                const uint32_t two = 2u * (spr - 1u);                        // lanes of the pair's two-strip tiles
                if (r < two) {
                    const uint32_t t = r >> 1, per = (spr - 1u) >> 1;        // two-strip tiles per band
                    const uint32_t wb = t / per;
                    ob = 2u * pair + wb;
                    q = 2u * (t - wb * per) + (r & 1u);
                } else {
                    ob = 2u * pair + (r - two);
                    q = spr - 1u;
                }
            } else {
                ob = sl / p.pl.spb;
                q = sl - ob * p.pl.spb;
            }
            uint32_t band;                                                   // band inside the chunk, in memory order
            if (p.pl.uniform) band = ob;
            else if (ob < full_bands) band = ob + ob / (s.Hb - 1u);
            else band = (ob - full_bands) * s.Hb + (s.Hb - 1u);
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
            const uint32_t mate = (LPT == 2u && !(p.pl.paired && q == spr - 1u)) ? 1u : 0u;
            table[sl] = (ok ? (eoff >> 2) : 0u) | ((ok ? rows : 0u) << 13) | (which << 17) | (writer << 19) | (mate << 20) |
                        ((band * s.Wb + bw) << 21);
        }
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
        ctl->q_closed = 0;
        ctl->mb_done = 0;
        for (uint32_t i = 0; i < S_MAILBOX; ++i) ctl->mb_seq[i] = 0;
        ctl->failed = 0;
        fence_barrier_init();
    }
    __syncthreads();

    if (warp == 2) {
        // ================= watcher (one thread).  Two duties, taken in turns:
        //   * count this CTA's folded chunks as arrived: the reduce closers post them in a mailbox; the watcher
        //     takes what is there, issues ONE release fence at gpu scope (the closers' folds happen before their
        //     posts, so the fence orders them before the counts; it costs a round trip to the L2, which is why
        //     no reduce warp issues it) and sends the counts, reductions without an answer;
        //   * complete the samples n = blockIdx.x, blockIdx.x + gridDim.x, ...: when every chunk of the sample has
        //     been counted, derive (delta, Delta, scale) from the folded extremes, write the first two to the blob
        //     and publish delta and scale in the slot.
        if (lane != 0) return;
        uint32_t next = 0;                       // next chunk of this CTA to count
        uint32_t n = blockIdx.x;                 // next sample to complete
        uint32_t polls = 0;
        SWait w = {0, 0};
        while (next < n_my || n < s.N) {
            bool progress = false;
            uint32_t cnt = 0;
            while (next + cnt < n_my && cnt < S_MAILBOX && lds_volatile(&ctl->mb_seq[(next + cnt) % S_MAILBOX]) == next + cnt + 1u) ++cnt;
            if (cnt) {
                __threadfence_block();
                fence_acq_rel_gpu();
                for (uint32_t i = 0; i < cnt; ++i)
                    red_add_relaxed(p.ws + WS_HEADER_WORDS + (size_t)ctl->mb_n[(next + i) % S_MAILBOX] * WS_SLOT_WORDS + 2, 1u);
                next += cnt;
                __threadfence_block();
                sts_volatile(&ctl->mb_done, next);
                progress = true;
            }
            if (n < s.N) {
                uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
                if (ld_acquire_u32(slot + 2) == p.expected_chunks) {
                    const QParams qp = make_qparams(key_float(~ld_relaxed_u32(slot + 0)), key_float(ld_relaxed_u32(slot + 1)), Q);
                    p.stats[2 * (size_t)n + 0] = qp.delta;
                    p.stats[2 * (size_t)n + 1] = qp.step;
                    const uint64_t word = ((uint64_t)(__float_as_uint(qp.scale) | 0x80000000u) << 32) | (uint64_t)__float_as_uint(qp.delta);
                    st_release_u64(reinterpret_cast<uint64_t*>(slot + 4), word);
                    n += G;
                    progress = true;
                }
            } else if (!cnt) {
                __nanosleep(100);
            }
            if (progress) {
                polls = 0;
                w.c0 = 0;
            } else if ((++polls & 7u) == 0 && s_give_up(p, ctl, w)) {
                s_record_failure(p, ctl, n < s.N ? n + 1u : 0x80000007u);
                break;
            }
        }
        return;
    }

    if (warp < 2) {
        // ================= producers: warp 0 streams the chunks from HBM into the reduce ring, warp 1 streams
        // ================= them again, from L2 and with their sample's parameters, into the quantise ring
        if (lane != 0) return;
        const bool quant = warp == 1;
        const uint32_t K = quant ? KQ : KR;
        const FastDiv by_K = quant ? p.by_kq : p.by_kr;
        uint64_t* full = quant ? ctl->full_q : ctl->full_r;
        uint64_t* empty = quant ? ctl->empty_q : ctl->empty_r;
        SDesc* desc = quant ? ctl->desc_q : ctl->desc_r;
        unsigned char* ring = quant ? ring_q : ring_r;
        const uint64_t policy = quant ? l2_policy_release() : l2_policy_keep();
        // parameter words of the samples of the next two chunks, asked for ahead of time
        uint64_t w0 = 0, w1 = 0;
        if (quant) {
            if (n_my > 0u) w0 = ld_relaxed_u64(reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)fdiv(blockIdx.x, p.by_S) * WS_SLOT_WORDS + 4));
            if (n_my > 1u) w1 = ld_relaxed_u64(reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)fdiv(blockIdx.x + G, p.by_S) * WS_SLOT_WORDS + 4));
        }
        uint32_t it = 0;
        bool ok = true;
        for (; it < n_my; ++it) {
            const uint32_t round = fdiv(it, by_K);
            const uint32_t st = it - round * K;
            const uint32_t j = blockIdx.x + it * G;
            const uint32_t n = fdiv(j, p.by_S);
            const uint32_t k = j - n * S;
            uint64_t word = w0;
            if (quant) {
                w0 = w1;
                if (it + 2u < n_my)
                    w1 = ld_relaxed_u64(reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)fdiv(j + 2u * G, p.by_S) * WS_SLOT_WORDS + 4));
            }
            if (it >= K && !s_wait(&empty[st], (round - 1u) & 1u, p, ctl, 0x80000002u + (quant ? 2u : 0u))) {
                ok = false;
                break;
            }
            if (!quant && it >= L + (uint32_t)S_AHEAD) {
                // the first read must not run away from the second one: what it brought into the L2 would be gone
                // by the time it is read again.  (The quantise half of chunk c needs reduce halves up to round
                // c + L - 1 only, so this wait always ends.)
                uint32_t polls = 0;
                SWait w = {0, 0};
                while (it - lds_volatile(&ctl->q_closed) >= L + (uint32_t)S_AHEAD) {
                    __nanosleep(32);
                    if ((++polls & 7u) == 0 && s_give_up(p, ctl, w)) {
                        s_record_failure(p, ctl, 0x80000006u);
                        ok = false;
                        break;
                    }
                }
                if (!ok) break;
            }
            if (quant && !(word >> 63)) {
                const uint64_t* pw = reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS + 4);
                uint32_t polls = 0;
                SWait w = {0, 0};
                while (true) {
                    word = ld_relaxed_u64(pw);
                    if (word >> 63) break;
                    if ((++polls & 7u) == 0 && s_give_up(p, ctl, w)) {
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
            SDesc d;
            d.ntiles = nbands * s.Wb;
            d.n = n;
            d.tile0 = k * p.pl.G * s.Wb;
            d.seq = 0;
            d.quad0 = ((uint64_t)n * s.CHW + e0) >> 2;
            d.ctr0 = rng_sample_base(p.seed, n) + K_GROUP * (uint64_t)((e0 >> 2) + 1u);
            d.delta = __uint_as_float((uint32_t)word);
            d.scale = __uint_as_float((uint32_t)(word >> 32) & 0x7FFFFFFFu);
            desc[st] = d;
            const uint32_t bytes = nelem * (uint32_t)sizeof(XT);
            const XT* src = reinterpret_cast<const XT*>(p.x) + ((size_t)n * s.CHW + e0);
            mbar_arrive_expect_tx(&full[st], bytes);
            bulk_load_hint(ring + (size_t)st * stage_bytes, src, bytes, &full[st], policy);
            __threadfence_block();
            sts_volatile(&desc[st].seq, it + 1u);
        }
        if (!ok || lds_volatile(&ctl->failed)) {
            // a wait gave up somewhere: let the copies still in flight land before the CTA may exit
            const uint32_t first = it > K ? it - K : 0u;
            for (uint32_t t = first; t < it; ++t) {
                const uint32_t round = fdiv(t, by_K);
                uint32_t polls = 0;
                while (!mbar_try_wait(&full[t - round * K], round & 1u) && ++polls < (1u << 20)) {
                }
            }
        }
        return;
    }

    // ================= workers: the first S_REDUCE_WARPS warps take the reduce units, the others the quantise
    // ================= units, each class dealing its units round-robin and taking them in order
    const uint32_t nf = p.pl.nf;
    const uint32_t row_bytes = s.W * (uint32_t)sizeof(XT);
    const uint32_t W4 = s.W >> 2;
    LT* lfc_out = reinterpret_cast<LT*>(p.lfc);
    OutT* packed = reinterpret_cast<OutT*>(p.packed);
    const bool reducer = warp < (uint32_t)S_SERVICE_WARPS + (uint32_t)S_REDUCE_WARPS;
    const uint32_t NW = reducer ? (uint32_t)S_REDUCE_WARPS : (blockDim.x >> 5) - (uint32_t)S_SERVICE_WARPS - (uint32_t)S_REDUCE_WARPS;
    // unit k of this CTA's chunk number `it`
    uint32_t it = 0, k = reducer ? warp - (uint32_t)S_SERVICE_WARPS : warp - (uint32_t)S_SERVICE_WARPS - (uint32_t)S_REDUCE_WARPS;
    while (k >= nf) {
        k -= nf;
        ++it;
    }

    if (reducer) {
        for (; it < n_my;) {
            const uint32_t round = fdiv(it, p.by_kr);
            const uint32_t st = it - round * KR;
            const bool landed = __all_sync(0xFFFFFFFFu, s_wait_chunk(&ctl->full_r[st], round & 1u, &ctl->desc_r[st].seq, it, p, ctl));
            if (!landed) break;
            // every unit index takes part in the closing count, also where a short chunk has no strips for it:
            // a stage is recycled only after each of its nf readers has looked at it
            // (a short last chunk of a sample holds a prefix of the tiles in memory order, not of the table: its
            // lanes are masked one by one)
            const uint32_t ntiles = ctl->desc_r[st].ntiles;
            uint32_t rec = 0u;
            {
                const uint32_t sl = k * 32u + lane;
                if (sl < p.pl.slots) rec = table[sl];
                if ((rec >> 21) >= ntiles) rec = 0u;
            }
            const bool work = __any_sync(0xFFFFFFFFu, rec != 0u);
            uint32_t kmin = 0, kmax = 0;
            if (work) {
                const uint32_t n = ctl->desc_r[st].n;
                const uint32_t rows = (rec >> 13) & 15u;
                const bool active = rows != 0u;
                const uint32_t which = (rec >> 17) & 3u;
                const unsigned char* xs = ring_r + (size_t)st * stage_bytes + ((size_t)(rec & 0x1FFFu) << QSHIFT);
                const bool full = __all_sync(0xFFFFFFFFu, rows == (uint32_t)P2 || rows == 0u);
                uint64_t vxy[P2], vzw[P2];
                const uint32_t rmax = full ? (uint32_t)P2 : __reduce_max_sync(0xFFFFFFFFu, rows);
                s_load_strip<XT, P2>(xs, row_bytes, rows, full, rmax, vxy, vzw);
                const float mean = s_tile_mean<P2>(vxy, vzw, active, (rec >> 20) & 1u, p.inv_cnt[which], p.cnt[which]);
                const float stored = Elem<LT>::round(mean);
                float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
                if (active) {
                    if (rec & (1u << 19))
                        Elem<LT>::store(lfc_out + (size_t)n * s.C * s.TPP + ctl->desc_r[st].tile0 + (rec >> 21), mean);
                    // extremes of x over the strip's in-bounds rows; x -> fl(x - stored) is monotone
                    float blo = 3.402823466e+38f, bhi = -3.402823466e+38f;
#pragma unroll
                    for (int r = 0; r < P2; ++r) {
                        if (full || ((uint32_t)r < rmax && (uint32_t)r < rows)) {
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
                    const uint32_t n = ctl->desc_r[st].n;
                    __threadfence_block();
                    mbar_arrive(&ctl->empty_r[st]);
                    if (lds_volatile(&ctl->failed) == 0u) {
                        // fold the chunk's extremes into the sample's slot in global scratch (reductions without an
                        // answer: an atomic that returns the old count to 148 CTAs was measured to cost more than the
                        // rest of the kernel) and tell the watcher, who counts the chunk as arrived
                        uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
                        red_max_relaxed(slot + 0, smin);
                        red_max_relaxed(slot + 1, smax);
                        uint32_t polls = 0;
                        SWait w = {0, 0};
                        bool room = true;
                        while (it - lds_volatile(&ctl->mb_done) >= S_MAILBOX) {          // never in practice
                            __nanosleep(64);
                            if ((++polls & 7u) == 0 && s_give_up(p, ctl, w)) {
                                s_record_failure(p, ctl, 0x80000008u);
                                room = false;
                                break;
                            }
                        }
                        if (room) {
                            ctl->mb_n[it % S_MAILBOX] = n;
                            __threadfence_block();
                            sts_volatile(&ctl->mb_seq[it % S_MAILBOX], it + 1u);
                        }
                    }
                }
            }
            k += NW;
            while (k >= nf) {
                k -= nf;
                ++it;
            }
        }
        return;
    }

    for (; it < n_my;) {
        const uint32_t round = fdiv(it, p.by_kq);
        const uint32_t st = it - round * KQ;
        if (!__all_sync(0xFFFFFFFFu, s_wait_chunk(&ctl->full_q[st], round & 1u, &ctl->desc_q[st].seq, it, p, ctl))) break;
        const uint32_t ntiles = ctl->desc_q[st].ntiles;
        uint32_t rec = 0u;
        {
            const uint32_t sl = k * 32u + lane;
            if (sl < p.pl.slots) rec = table[sl];
            if ((rec >> 21) >= ntiles) rec = 0u;
        }
        if (__any_sync(0xFFFFFFFFu, rec != 0u)) {
            const uint32_t rows = (rec >> 13) & 15u;
            const bool active = rows != 0u;
            const uint32_t which = (rec >> 17) & 3u;
            const uint32_t quad = rec & 0x1FFFu;
            const unsigned char* xs = ring_q + (size_t)st * stage_bytes + ((size_t)quad << QSHIFT);
            const bool full = __all_sync(0xFFFFFFFFu, rows == (uint32_t)P2 || rows == 0u);
            uint64_t vxy[P2], vzw[P2];
            const uint32_t rmax = full ? (uint32_t)P2 : __reduce_max_sync(0xFFFFFFFFu, rows);
            s_load_strip<XT, P2>(xs, row_bytes, rows, full, rmax, vxy, vzw);
            const float mean = s_tile_mean<P2>(vxy, vzw, active, (rec >> 20) & 1u, p.inv_cnt[which], p.cnt[which]);
            const float stored = Elem<LT>::round(mean);
            if (active) {
                const float delta = ctl->desc_q[st].delta, scale = ctl->desc_q[st].scale;
                const uint64_t stored2 = pk2(stored, stored);
                const uint64_t delta2 = pk2(delta, delta), scale2 = pk2(scale, scale);
                uint64_t ctr = ctl->desc_q[st].ctr0 + K_GROUP * (uint64_t)quad;
                OutT* out = packed + ctl->desc_q[st].quad0 + quad;
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
                        if ((uint32_t)r < rmax) {
                            if ((uint32_t)r < rows) {
                                *out = (OutT)quant_row<Q>(vxy[r], vzw[r], stored2, delta2, scale2, rng_mix(ctr));
                                out += W4;
                                ctr += p.rng_row_step;
                            }
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
                atomicAdd(&ctl->q_closed, 1u);
            }
        }
        k += NW;
        while (k >= nf) {
            k -= nf;
            ++it;
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
    pl.spb = s.W / 4u;
    pl.paired = (s.P2 == 8u && (pl.spb & 1u)) ? 1u : 0u;
    const uint64_t bands = (uint64_t)s.C * s.Hb;
    if (bands >= (1ull << 31)) return DIV_ERR_PARAM;
    pl.bands_per_sample = (uint32_t)bands;
    pl.uniform = (s.H % s.B == 0) ? 1u : 0u;
    // bands per chunk: a count that keeps the chunk's inner geometry the same for every chunk (any count when
    // all bands are alike, whole planes otherwise) and, where possible, fills whole units of 32 strips
    // (an even count where the table lays bands out in pairs)
    const uint32_t geo1 = pl.uniform ? 1u : s.Hb;
    const uint32_t geo = (pl.paired && (geo1 & 1u)) ? 2u * geo1 : geo1;
    const uint64_t geo_bytes = (pl.uniform ? (uint64_t)s.B * s.W * sx : (uint64_t)s.HW * sx) * (geo / geo1);     // bytes of `geo` bands
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
    if (pl.slots > 4096u || G * s.Wb > 2048u) return DIV_ERR_PARAM;         // widths of the strip table's fields
    pl.nf = (pl.slots + 31u) / 32u;
    pl.chunk_elems = pl.uniform ? G * s.B * s.W : (G / s.Hb) * s.HW;
    if (pl.chunk_elems >= (1u << 15)) return DIV_ERR_PARAM;
    pl.chunks_per_sample = (pl.bands_per_sample + G - 1u) / G;
    pl.stage_bytes = (pl.chunk_elems * sx + 127u) & ~127u;
    // shared memory: the two rings, the strip table, the control block; as many stages as fit, DIVK_S_Q_STAGES_PER_8
    // eighths of them (rounded down) for the quantise ring
    const uint32_t fixed = ((pl.slots * 4u + 15u) & ~15u) + (uint32_t)sizeof(SCtl) + 16u;
    if ((uint32_t)di.smem_optin < fixed + 4u * pl.stage_bytes) return DIV_ERR_PARAM;
    uint32_t stages = ((uint32_t)di.smem_optin - fixed) / pl.stage_bytes;
    if (stages > 2u * S_MAX_STAGES) stages = 2u * S_MAX_STAGES;
    uint32_t kq = stages * DIVK_S_Q_STAGES_PER_8 / 8u;
    if (kq < 2u) kq = 2u;
    if (kq > stages - 2u) kq = stages - 2u;
    if (kq > (uint32_t)S_MAX_STAGES) kq = S_MAX_STAGES;
    uint32_t kr = stages - kq;
    if (kr > (uint32_t)S_MAX_STAGES) kr = S_MAX_STAGES;
    pl.kr = kr;
    pl.kq = kq;
    pl.smem_bytes = (int32_t)((kr + kq) * pl.stage_bytes + fixed);
    pl.total_chunks = (uint64_t)pl.chunks_per_sample * s.N;
    uint64_t grid = (uint64_t)di.sms;
    if (grid > pl.total_chunks) grid = pl.total_chunks;
    pl.grid = (int32_t)grid;
    pl.threads = S_THREADS;
    if (pl.total_chunks + grid >= (1ull << 30)) return DIV_ERR_PARAM;        // chunk indices are 32-bit on the device
    // lag in rounds of `grid` chunks: the rounds a sample can spread over plus one (see the progress argument at
    // the top), and about DIVK_S_LAG_BYTES of x
    const uint64_t round_bytes = (uint64_t)pl.chunk_elems * sx * grid;
    uint64_t lag = (DIVK_S_LAG_BYTES + round_bytes - 1) / round_bytes;
    const uint64_t need = ((uint64_t)pl.chunks_per_sample - 1u + grid - 1u) / grid + 1u;
    if (lag < need) lag = need;
    if (lag >= (1ull << 20)) return DIV_ERR_PARAM;
    pl.lag_steps = (uint32_t)lag;
    *out = pl;
    return DIV_OK;
}

template <typename XT, typename LT, int Q, int P2>
inline div_status launch_staged(const SParams& prm, cudaStream_t st) {
    auto kern = staged_kernel<XT, LT, Q, P2>;
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
