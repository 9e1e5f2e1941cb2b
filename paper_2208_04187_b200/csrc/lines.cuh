// Compress kernels for 1-D activation maps (the paper's appendix "Compression of 1D and 3D Activation Maps":
// Minibatch x Channel x N, average pooling and nearest up-sampling along the last axis; Eq. 9 unchanged).
// A 1-D map is described as N x C x 1 x W.  Conditions: W % 4 == 0, B a power of two in [4, 128], Q in {2, 4, 8}.
//
// line_fused_kernel does both halves in one launch (see there); where its CTAs cannot all be resident the pair
// below runs instead.  Two launches, no dependency inside a kernel (token / MLP activations of one layer are tens
// of MB: the second read of x comes from the 126 MB L2; larger tensors are still handled correctly, reading x
// twice from HBM):
//   line_stats_kernel   a lane owns 4 consecutive elements; the B/4 lanes of a block meet through xor shuffles
//                       (the balanced pairwise tree over the B positions, neighbours first); stored
//                       low-frequency values; residual extremes -> per-sample min / max keys in the scratch slots
//   line_quant_kernel   one thread per 4 consecutive elements (they share a block): Eq. 9 with stochastic
//                       rounding on packed pairs, one byte / half-word / word of codes per thread and step
#pragma once

#include "fused_v.cuh"

namespace divk {

struct LineGeom {
    uint32_t C, W, Wb, CHW;
    uint32_t qpr;            // quads per row = W / 4
    uint32_t cpr;            // warp chunks (32 quads) per row
    uint32_t chunks;         // C * cpr: warp chunks per sample
    uint32_t log2lpt;        // log2(B / 4): lanes per block
    uint32_t B, tail_cnt;    // in-bounds elements of a row's last block
    float inv_full, inv_tail;   // 1 / count of a full block and of a row's last block when that is a power of two, else 0
    float cnt_full, cnt_tail;
    uint32_t qps;            // quads per sample
    // single-launch kernel: a lane owns a segment of min(B, 16) consecutive elements of one block
    uint32_t log2B;
    uint32_t eq;             // quads per segment: 1, 2 or 4
    uint32_t log2spb;        // log2(segments per block) = log2(B / (4 * eq))
    uint32_t sps;            // segment slots per row = Wb * segments per block (slots past the row's end are empty)
    FastDiv by_cpr, by_qpr, by_sps;
};

constexpr int LINE_U = 4;     // warp chunks a warp works on at a time (their loads are issued together)

template <typename XT, typename LT>
__global__ void __launch_bounds__(256)
line_stats_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, LineGeom g) {
    const uint32_t n = blockIdx.y;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t lpt = 1u << g.log2lpt;
    const XT* x_n = x + (size_t)n * g.CHW;
    LT* lfc_n = lfc + (size_t)n * g.C * g.Wb;
    float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
    for (uint32_t wg = blockIdx.x * 8u + warp; wg * LINE_U < g.chunks; wg += gridDim.x * 8u) {
        uint64_t xy[LINE_U], zw[LINE_U];
        uint32_t row[LINE_U], q[LINE_U];
        bool ok[LINE_U];
#pragma unroll
        for (int u = 0; u < LINE_U; ++u) {
            const uint32_t wc = wg * LINE_U + u;
            const bool live = wc < g.chunks;
            row[u] = fdiv(live ? wc : 0u, g.by_cpr);
            q[u] = ((live ? wc : 0u) - row[u] * g.cpr) * 32u + lane;          // quad inside the row
            ok[u] = live && q[u] < g.qpr;
            xy[u] = 0ull;
            zw[u] = 0ull;
            if (ok[u]) StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(x_n + (row[u] * g.W + 4u * q[u])), xy[u], zw[u]);   // < CHW < 2^31
        }
#pragma unroll
        for (int u = 0; u < LINE_U; ++u) {
            float a, b, c, d;
            upk2(xy[u], a, b);
            upk2(zw[u], c, d);
            float sum = __fadd_rn(__fadd_rn(a, b), __fadd_rn(c, d));
            for (uint32_t m = 1; m < lpt; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
            const uint32_t t = q[u] >> g.log2lpt;                         // block inside the row
            const bool tail = t + 1u == g.Wb;
            const float inv = tail ? g.inv_tail : g.inv_full;
            const float mean = (inv != 0.f) ? __fmul_rn(sum, inv) : __fdiv_rn(sum, tail ? g.cnt_tail : g.cnt_full);
            const float stored = Elem<LT>::round(mean);
            if (ok[u]) {
                if ((q[u] & (lpt - 1u)) == 0u) Elem<LT>::store(lfc_n + (row[u] * g.Wb + t), mean);
                // x -> fl(x - stored) is monotone: the residual extremes are those of the extreme x
                lo = fminf(lo, __fsub_rn(fminf(fminf(a, b), fminf(c, d)), stored));
                hi = fmaxf(hi, __fsub_rn(fmaxf(fmaxf(a, b), fmaxf(c, d)), stored));
            }
        }
    }
    const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
    const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
    if (lane == 0) {
        uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
        atomicMax(slot + 0, kmin);       // neutral keys when this warp had no chunk
        atomicMax(slot + 1, kmax);
    }
}

template <typename XT, typename LT, int Q, int QPT>
__global__ void __launch_bounds__(256)
line_quant_kernel(const XT* __restrict__ x, const LT* __restrict__ lfc, const uint32_t* __restrict__ ws,
                  void* __restrict__ packed_v, float* __restrict__ stats, LineGeom g, uint64_t seed) {
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
    const XT* x_n = x + (size_t)n * g.CHW;
    const LT* lfc_n = lfc + (size_t)n * g.C * g.Wb;
    OutT* packed = reinterpret_cast<OutT*>(packed_v) + (uint64_t)n * g.qps;
    const uint32_t q0 = blockIdx.x * (256u * QPT) + threadIdx.x;
    uint64_t xy[QPT], zw[QPT];
    float lf[QPT];
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;                            // quad inside the sample
        if (q < g.qps) {
            StripRow2<XT>::load(reinterpret_cast<const unsigned char*>(x_n + q * 4u), xy[k], zw[k]);
            const uint32_t row = fdiv(q, g.by_qpr);
            lf[k] = Elem<LT>::load(lfc_n + (row * g.Wb + ((q - row * g.qpr) >> g.log2lpt)));
        }
    }
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < g.qps)
            packed[q] = (OutT)quant_row<Q>(xy[k], zw[k], pk2(lf[k], lf[k]), delta2, scale2, rng_group(base, q));
    }
}

// One launch for both halves.  CTA (b, n) owns the rows [b * rpc, (b + 1) * rpc) of sample n:
//   1. block means, stored low-frequency values and residual extremes of its rows: the same values as
//      line_stats_kernel in another layout (a lane owns a segment of min(B, 16) consecutive elements of one block);
//      the CTA's extremes are folded into the sample's slot (two reductions without an answer), then, behind a
//      release fence, the CTA is counted as arrived;
//   2. thread 0 waits (bounded) until all CTAs of the sample have arrived and derives (delta, Delta, scale);
//   3. Eq. 9 and packing of the same rows, segment by segment (one low-frequency load and one counter per segment):
//      x is read a second time (it is still in this SM's L1 or in the L2), the low-frequency values are the ones
//      this CTA stored in step 1.
// The launch is cooperative so that the CTAs a wait depends on are resident; no grid-wide barrier is used.
struct LineFused {
    uint32_t rpc;                 // rows per CTA
    uint32_t ctas_per_sample;
    uint32_t expected;            // arrivals that complete a sample
    uint64_t timeout_ns;
};

template <typename XT, typename LT, int Q, int EQ>
__global__ void __launch_bounds__(256)
line_fused_kernel(const XT* __restrict__ x, LT* __restrict__ lfc, uint32_t* __restrict__ ws, void* __restrict__ packed_v,
                  float* __restrict__ stats, LineGeom g, LineFused f, uint64_t seed) {
    typedef typename PackedUnit<Q>::type OutT;
    __shared__ uint32_t s_kmin, s_kmax, s_delta, s_scale, s_ok;
    const uint32_t n = blockIdx.y;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t row0 = blockIdx.x * f.rpc;
    const uint32_t nrows = row0 < g.C ? min(f.rpc, g.C - row0) : 0u;
    const XT* x_n = x + (size_t)n * g.CHW;
    LT* lfc_n = lfc + (size_t)n * g.C * g.Wb;
    if (threadIdx.x == 0) {
        s_kmin = 0;
        s_kmax = 0;
        s_ok = 0;
    }
    __syncthreads();

    // ---------------- half 1: a lane owns a segment of EQ quads of one block ----------------
    // Slot j of a row: block j >> log2spb, part j & (spb - 1) of it; the parts of a block sit in neighbouring lanes
    // (sps is a multiple of spb, which divides 32).  The block sum is the balanced pairwise tree over its positions:
    // inside the lane over the segment's elements, then by xor shuffles over the parts.
    const uint32_t spb = 1u << g.log2spb;
    const uint32_t s0 = row0 * g.sps, s1 = (row0 + nrows) * g.sps;           // this CTA's slots [s0, s1)
    {
        float lo = 3.402823466e+38f, hi = -3.402823466e+38f;
        for (uint32_t sb = s0 + warp * 32u; sb < s1; sb += 256u) {
            const uint32_t sl = sb + lane;
            const bool live = sl < s1;
            const uint32_t row = fdiv(live ? sl : s0, g.by_sps);
            const uint32_t j = (live ? sl : s0) - row * g.sps;
            const uint32_t t = j >> g.log2spb;                               // block inside the row
            const uint32_t col = (t << g.log2B) + (j & (spb - 1u)) * (4u * EQ);
            const uint32_t nq = (live && col < g.W) ? min((uint32_t)EQ, (g.W - col) >> 2) : 0u;
            const unsigned char* xp = reinterpret_cast<const unsigned char*>(x_n + (row * g.W + (nq ? col : 0u)));
            uint64_t xy[EQ], zw[EQ];
#pragma unroll
            for (int i = 0; i < EQ; ++i) {
                xy[i] = 0ull;
                zw[i] = 0ull;
                if ((uint32_t)i < nq) StripRow2<XT>::load(xp + i * 4 * (int)sizeof(XT), xy[i], zw[i]);
            }
            float part[EQ];
            float blo = 3.402823466e+38f, bhi = -3.402823466e+38f;
#pragma unroll
            for (int i = 0; i < EQ; ++i) {
                float a, b, c, d;
                upk2(xy[i], a, b);
                upk2(zw[i], c, d);
                part[i] = __fadd_rn(__fadd_rn(a, b), __fadd_rn(c, d));
                if ((uint32_t)i < nq) {
                    blo = fmin3(blo, a, b);
                    blo = fmin3(blo, c, d);
                    bhi = fmax3(bhi, a, b);
                    bhi = fmax3(bhi, c, d);
                }
            }
#pragma unroll
            for (int w = EQ; w > 1; w >>= 1) {
#pragma unroll
                for (int i = 0; i < w / 2; ++i) part[i] = __fadd_rn(part[2 * i], part[2 * i + 1]);
            }
            float sum = part[0];
            for (uint32_t m = 1; m < spb; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
            if (nq) {
                const bool tail = t + 1u == g.Wb;
                const float inv = tail ? g.inv_tail : g.inv_full;
                const float mean = (inv != 0.f) ? __fmul_rn(sum, inv) : __fdiv_rn(sum, tail ? g.cnt_tail : g.cnt_full);
                const float stored = Elem<LT>::round(mean);
                if ((j & (spb - 1u)) == 0u) Elem<LT>::store(lfc_n + (row * g.Wb + t), mean);
                // x -> fl(x - stored) is monotone: the residual extremes are those of the extreme x
                lo = fminf(lo, __fsub_rn(blo, stored));
                hi = fmaxf(hi, __fsub_rn(bhi, stored));
            }
        }
        const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(lo));
        const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(hi));
        if (lane == 0) {
            atomicMax(&s_kmin, kmin);
            atomicMax(&s_kmax, kmax);
        }
    }
    // the barrier also orders this CTA's stores of low-frequency values before its loads of them in half 2
    __syncthreads();

    // ---------------- the sample's extremes: fold, count, wait for the other CTAs of the sample ----------------
    if (threadIdx.x == 0) {
        uint32_t* slot = ws + WS_HEADER_WORDS + (size_t)n * WS_SLOT_WORDS;
        if (nrows) {
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
    if (!s_ok || nrows == 0) return;

    // ---------------- half 2: the same segments; one low-frequency value and one counter per segment ----------------
    const float delta = __uint_as_float(s_delta), scale = __uint_as_float(s_scale);
    const uint64_t delta2 = pk2(delta, delta), scale2 = pk2(scale, scale);
    const uint64_t base = rng_sample_base(seed, n);
    OutT* packed = reinterpret_cast<OutT*>(packed_v) + (uint64_t)n * g.qps;
    for (uint32_t sl = s0 + threadIdx.x; sl < s1; sl += 256u) {
        const uint32_t row = fdiv(sl, g.by_sps);
        const uint32_t j = sl - row * g.sps;
        const uint32_t t = j >> g.log2spb;
        const uint32_t col = (t << g.log2B) + (j & (spb - 1u)) * (4u * EQ);
        if (col >= g.W) continue;
        const uint32_t nq = min((uint32_t)EQ, (g.W - col) >> 2);
        const uint32_t q0 = (row * g.W + col) >> 2;                              // first quad of the segment inside the sample
        const unsigned char* xp = reinterpret_cast<const unsigned char*>(x_n + (size_t)q0 * 4u);
        uint64_t xy[EQ], zw[EQ];
#pragma unroll
        for (int i = 0; i < EQ; ++i)
            if ((uint32_t)i < nq) StripRow2<XT>::load(xp + i * 4 * (int)sizeof(XT), xy[i], zw[i]);
        const float lf = Elem<LT>::load_cg(lfc_n + (row * g.Wb + t));            // stored by this CTA in half 1
        const uint64_t lf2 = pk2(lf, lf);
        uint64_t ctr = base + K_GROUP * (uint64_t)(q0 + 1u);
#pragma unroll
        for (int i = 0; i < EQ; ++i) {
            if ((uint32_t)i < nq) packed[q0 + i] = (OutT)quant_row<Q>(xy[i], zw[i], lf2, delta2, scale2, rng_mix(ctr));
            ctr += K_GROUP;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
constexpr int LINE_QPT = 4;

inline bool plan_lines(const div_desc* d, const Shape& s, LineGeom* out) {
    if (s.H != 1 || s.W % 4 != 0) return false;
    if (!(d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return false;
    if (s.B < 4 || s.B > 128 || (s.B & (s.B - 1)) != 0) return false;
    if (s.CHW >= (1u << 31) || s.N > 65535u) return false;
    LineGeom g;
    g.C = s.C; g.W = s.W; g.Wb = s.Wb; g.CHW = s.CHW; g.B = s.B;
    g.qpr = s.W / 4;
    g.cpr = (g.qpr + 31u) / 32u;
    const uint64_t chunks = (uint64_t)s.C * g.cpr;
    if (chunks >= (1ull << 31)) return false;
    g.chunks = (uint32_t)chunks;
    g.log2lpt = 0;
    while ((4u << g.log2lpt) < s.B) ++g.log2lpt;
    g.tail_cnt = s.W - (s.Wb - 1u) * s.B;
    g.cnt_full = (float)s.B;
    g.cnt_tail = (float)g.tail_cnt;
    g.inv_full = 1.0f / (float)s.B;                                                   // B is a power of two: exact
    g.inv_tail = (g.tail_cnt & (g.tail_cnt - 1u)) == 0u ? 1.0f / (float)g.tail_cnt : 0.f;
    g.qps = s.CHW / 4;
    g.by_cpr = host_fastdiv(g.cpr);
    g.by_qpr = host_fastdiv(g.qpr);
    g.log2B = g.log2lpt + 2u;
    g.eq = s.B >= 16u ? 4u : s.B / 4u;
    g.log2spb = 0;
    while (((4u * g.eq) << g.log2spb) < s.B) ++g.log2spb;
    g.sps = s.Wb << g.log2spb;
    if ((uint64_t)s.C * g.sps >= (1ull << 31)) return false;
    g.by_sps = host_fastdiv(g.sps);
    *out = g;
    return true;
}

template <typename XT, typename LT, int Q, int EQ>
inline int line_fused_occupancy(int dev) {
    static SmemSeen cached[DEVICE_CACHE_SLOTS];          // .bytes holds the count
    const void* kern = (const void*)line_fused_kernel<XT, LT, Q, EQ>;
    const bool slot = dev >= 0 && dev < DEVICE_CACHE_SLOTS;
    if (slot && cached[dev].fn.load(std::memory_order_acquire) == kern) {
        const int c = cached[dev].bytes.load(std::memory_order_acquire);
        if (c > 0) return c;
    }
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, line_fused_kernel<XT, LT, Q, EQ>, 256, 0) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (slot && n > 0) {
        cached[dev].fn.store(nullptr, std::memory_order_release);
        cached[dev].bytes.store(n, std::memory_order_release);
        cached[dev].fn.store(kern, std::memory_order_release);
    }
    return n;
}

// rows per CTA and CTAs per sample of the single-launch form; false when its CTAs could not all be resident
template <typename XT, typename LT, int Q, int EQ>
inline bool plan_line_fused(const Shape& s, const DeviceInfo& di, LineFused* out) {
    const int occ = line_fused_occupancy<XT, LT, Q, EQ>(di.dev);
    if (occ < 1) return false;
    const uint64_t capacity = (uint64_t)occ * di.sms;
    if (s.N > capacity) return false;
    uint64_t want = (8ull * di.sms + s.N - 1) / s.N;                     // CTAs per sample: about 8 per SM in all ...
    if (want * s.N > capacity) want = capacity / s.N;                    // ... and never more than fit at once
    if (want > s.C) want = s.C;
    if (want < 1) want = 1;
    out->rpc = (uint32_t)((s.C + want - 1) / want);
    out->ctas_per_sample = (s.C + out->rpc - 1) / out->rpc;
    out->expected = out->ctas_per_sample;
    out->timeout_ns = 2000000000ull;
    return true;
}

template <typename XT, typename LT, int Q, int EQ>
inline bool launch_line_fused(const Shape& s, const div_layout& lo, const LineGeom& g, const DeviceInfo& di, const void* x,
                              uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st) {
    LineFused f;
    if (!plan_line_fused<XT, LT, Q, EQ>(s, di, &f)) return false;
    const XT* xt = (const XT*)x;
    LT* lfc = (LT*)(blob + lo.lfc_off);
    void* packed = blob + lo.packed_off;
    float* stats = (float*)(blob + lo.stats_off);
    LineGeom gg = g;
    void* args[] = {(void*)&xt, (void*)&lfc, (void*)&ws, (void*)&packed, (void*)&stats, (void*)&gg, (void*)&f, (void*)&seed};
    if (cudaLaunchCooperativeKernel((const void*)line_fused_kernel<XT, LT, Q, EQ>, dim3(f.ctas_per_sample, s.N), dim3(256), args, 0, st) !=
        cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return true;
}

template <typename XT, typename LT>
inline div_status compress_lines_t(const div_desc* d, const Shape& s, const div_layout& lo, const LineGeom& g,
                                   const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st, bool allow_fused) {
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return DIV_ERR_CUDA;
    if (allow_fused) {
        bool done = false;
#define DIVK_LF(QQ)                                                                                          \
    (g.eq == 4 ? launch_line_fused<XT, LT, QQ, 4>(s, lo, g, di, x, blob, ws, seed, st)                        \
               : g.eq == 2 ? launch_line_fused<XT, LT, QQ, 2>(s, lo, g, di, x, blob, ws, seed, st)            \
                           : launch_line_fused<XT, LT, QQ, 1>(s, lo, g, di, x, blob, ws, seed, st))
        switch (d->qbits) {
            case 2: done = DIVK_LF(2); break;
            case 4: done = DIVK_LF(4); break;
            case 8: done = DIVK_LF(8); break;
            default: return DIV_ERR_PARAM;
        }
#undef DIVK_LF
        if (done) return DIV_OK;
    }
    // pass 1: enough CTAs per sample to fill the GPU a few times over, never more than there are warp chunks
    uint32_t bx = (uint32_t)((16ull * di.sms + s.N - 1) / s.N);
    const uint32_t bx_max = (g.chunks + 8u * LINE_U - 1u) / (8u * LINE_U);
    if (bx > bx_max) bx = bx_max;
    if (bx < 1) bx = 1;
    const XT* xt = (const XT*)x;
    LT* lfc = (LT*)(blob + lo.lfc_off);
    line_stats_kernel<XT, LT><<<dim3(bx, s.N), 256, 0, st>>>(xt, lfc, ws, g);
    if (cudaGetLastError() != cudaSuccess) return DIV_ERR_CUDA;
    const uint32_t per_block = 256u * LINE_QPT;
    const dim3 grid2((g.qps + per_block - 1) / per_block, s.N);
    void* packed = blob + lo.packed_off;
    float* stats = (float*)(blob + lo.stats_off);
    switch (d->qbits) {
        case 2: line_quant_kernel<XT, LT, 2, LINE_QPT><<<grid2, 256, 0, st>>>(xt, lfc, ws, packed, stats, g, seed); break;
        case 4: line_quant_kernel<XT, LT, 4, LINE_QPT><<<grid2, 256, 0, st>>>(xt, lfc, ws, packed, stats, g, seed); break;
        case 8: line_quant_kernel<XT, LT, 8, LINE_QPT><<<grid2, 256, 0, st>>>(xt, lfc, ws, packed, stats, g, seed); break;
        default: return DIV_ERR_PARAM;
    }
    return cudaGetLastError() == cudaSuccess ? DIV_OK : DIV_ERR_CUDA;
}

inline div_status compress_lines(const div_desc* d, const Shape& s, const div_layout& lo, const LineGeom& g,
                                 const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st, bool allow_fused = true) {
    typedef __nv_bfloat16 bf16;
    if (d->x_dtype == DIV_F32) {
        if (d->lfc_dtype == DIV_F32) return compress_lines_t<float, float>(d, s, lo, g, x, blob, ws, seed, st, allow_fused);
        return compress_lines_t<float, bf16>(d, s, lo, g, x, blob, ws, seed, st, allow_fused);
    }
    if (d->lfc_dtype == DIV_F32) return compress_lines_t<bf16, float>(d, s, lo, g, x, blob, ws, seed, st, allow_fused);
    return compress_lines_t<bf16, bf16>(d, s, lo, g, x, blob, ws, seed, st, allow_fused);
}

// would the single-launch form run this descriptor?
inline bool line_fused_applies(const div_desc* d, const Shape& s, const LineGeom& g, LineFused* out) {
    typedef __nv_bfloat16 bf16;
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return false;
#define DIVK_LE(XT, LT, QQ) \
    (g.eq == 4 ? plan_line_fused<XT, LT, QQ, 4>(s, di, out) : g.eq == 2 ? plan_line_fused<XT, LT, QQ, 2>(s, di, out) : plan_line_fused<XT, LT, QQ, 1>(s, di, out))
#define DIVK_LQ(XT, LT) (d->qbits == 2 ? DIVK_LE(XT, LT, 2) : d->qbits == 4 ? DIVK_LE(XT, LT, 4) : DIVK_LE(XT, LT, 8))
    if (d->x_dtype == DIV_F32) return d->lfc_dtype == DIV_F32 ? DIVK_LQ(float, float) : DIVK_LQ(float, bf16);
    return d->lfc_dtype == DIV_F32 ? DIVK_LQ(bf16, float) : DIVK_LQ(bf16, bf16);
#undef DIVK_LQ
#undef DIVK_LE
}

}  // namespace divk
