// Fused single-pass compress kernel (DIVISION Sec. 4.1; Algorithm 1, forward loop) for sm_100a.
//
// x is read from HBM exactly once.  The per-sample min / max of the residual is a dependency that
// spans the whole sample, so the residuals wait ON CHIP between the two halves of the work:
//
//   * the tensor is cut into chunks (a run of whole tile rows of one plane, or a run of whole planes)
//     that never straddle a sample; chunk j goes to CTA j mod gridDim.x, so the CTAs sweep the
//     samples together;
//   * a producer warp streams each chunk into a shared-memory ring with one bulk asynchronous copy
//     (cp.async.bulk, completion on an mbarrier);
//   * consumer warps, half 1 ("reduce"): block means in the fixed summation order, store the
//     low-frequency values, replace x by the residual r = x - stored_lfc in shared memory, fold the
//     residual extremes into the per-sample slot in global scratch (integer atomics on
//     order-preserving keys) and count the chunk as arrived; the CTA whose arrival completes a sample
//     publishes (delta, scale) in the slot and (delta, Delta) in the blob;
//   * consumer warps, half 2 ("quantise"), `lag` chunks later: wait (bounded) until the sample's
//     parameters are published, then quantise the residuals still sitting in shared memory with
//     stochastic rounding (Eq. 9) and write whole packed 32-bit words, coalesced.
//
// Every wait is bounded: when a limit runs out the kernel records DIV_ERR_TIMEOUT in the workspace
// status word, stops waiting everywhere and drains normally.  The launch is cooperative only to be
// certain that all CTAs are resident (no grid-wide barrier is used).
#pragma once

#include <atomic>

#include "../../include/division.h"
#include "common.cuh"
#include "twopass.cuh"   // Shape

namespace divk {

// slot words (see common.cuh): 0 ~key(min), 1 key(max), 2 arrivals; words 4..5 hold the published
// 64-bit parameter word: low 32 bits = delta, high 32 bits = scale | 0x80000000 (scale >= 0, so the
// sign bit means "ready").

struct FusedPlan {
    int32_t grid, threads, stages, lag, smem_bytes;
    uint32_t mode;               // 0: chunk = cb tile rows of one plane; 1: chunk = cb whole planes
    uint32_t cb;                 // tile rows (mode 0) or planes (mode 1) per full chunk
    uint32_t cpp;                // chunks per plane (mode 0)
    uint32_t chunk_elems;        // elements of a full chunk
    uint32_t chunks_per_sample;  // S
    uint32_t stage_bytes;
    uint32_t p2;                 // lanes per tile / padded tile side
};

struct FusedParams {
    Shape s;
    FusedPlan pl;
    FastDiv by_S, by_cpp, by_tpp;
    const void* x;
    void* lfc;
    uint32_t* packed;
    float* stats;
    uint32_t* ws;
    uint64_t seed;
    uint64_t total_chunks;
    uint32_t expected_arrivals;   // S (a test may ask for an unreachable count)
    uint64_t timeout_ns;          // how long any single wait may last before it gives up
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(smem_dst)),
        "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ uint64_t ld_relaxed_u64(const uint64_t* p) {
    uint64_t v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u64(uint64_t* p, uint64_t v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }

// ------------------------------------------------------------------------------------------------
// chunk geometry
// ------------------------------------------------------------------------------------------------
struct Chunk {
    uint32_t n, e0, nelem, tile0, ntiles;
};
__device__ __forceinline__ Chunk get_chunk(const FusedParams& p, uint32_t gc) {
    Chunk c;
    const Shape& s = p.s;
    c.n = fdiv(gc, p.by_S);
    const uint32_t k = gc - c.n * p.pl.chunks_per_sample;
    if (p.pl.mode == 0) {
        const uint32_t plane = fdiv(k, p.by_cpp);
        const uint32_t kb = k - plane * p.pl.cpp;
        const uint32_t band0 = kb * p.pl.cb;
        const uint32_t band1 = min(s.Hb, band0 + p.pl.cb);
        const uint32_t row0 = band0 * s.B, row1 = min(s.H, band1 * s.B);
        c.e0 = plane * s.HW + row0 * s.W;
        c.nelem = (row1 - row0) * s.W;
        c.tile0 = plane * s.TPP + band0 * s.Wb;
        c.ntiles = (band1 - band0) * s.Wb;
    } else {
        const uint32_t plane0 = k * p.pl.cb;
        const uint32_t plane1 = min(s.C, plane0 + p.pl.cb);
        c.e0 = plane0 * s.HW;
        c.nelem = (plane1 - plane0) * s.HW;
        c.tile0 = plane0 * s.TPP;
        c.ntiles = (plane1 - plane0) * s.TPP;
    }
    return c;
}

// shared-memory control block (placed after the tile table)
struct FusedCtl {
    uint64_t full[8];      // producer -> consumers: chunk landed
    uint64_t empty[8];     // consumers -> producer: stage may be overwritten
    uint32_t kmin[8];      // per stage: ~key(min r), key(max r) folded over the consumer warps
    uint32_t kmax[8];
    uint32_t done[8];      // per stage: consumer warps that finished half 1
    uint32_t failed;       // a wait gave up somewhere in this CTA
};
constexpr int FUSED_MAX_STAGES = 8;

__device__ __forceinline__ uint64_t now_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Has this wait lasted too long, or has any wait of this launch already given up?
__device__ __forceinline__ bool give_up(const FusedParams& p, FusedCtl* ctl, uint64_t& t0) {
    if (*(volatile uint32_t*)&ctl->failed || ld_relaxed_u32(p.ws) != 0u) return true;
    const uint64_t t = now_ns();
    if (t0 == 0) t0 = t;
    return t - t0 > p.timeout_ns;
}
__device__ __forceinline__ void record_failure(const FusedParams& p, FusedCtl* ctl, uint32_t detail) {
    atomicCAS(p.ws, 0u, (uint32_t)DIV_ERR_TIMEOUT);
    atomicCAS(p.ws + 1, 0u, detail);
    *(volatile uint32_t*)&ctl->failed = 1u;
}

// bounded wait on an mbarrier phase; false when it gave up (and the failure is recorded)
__device__ __forceinline__ bool wait_barrier(uint64_t* bar, uint32_t parity, const FusedParams& p, FusedCtl* ctl) {
    uint32_t polls = 0;
    uint64_t t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 31u) == 0 && give_up(p, ctl, t0)) {
            record_failure(p, ctl, 0x80000000u);
            return false;
        }
    }
    return true;
}

// element load from the staged chunk
template <typename XT> __device__ __forceinline__ float stage_load(const XT* xs, uint32_t i);
template <> __device__ __forceinline__ float stage_load<float>(const float* xs, uint32_t i) { return xs[i]; }
template <> __device__ __forceinline__ float stage_load<__nv_bfloat16>(const __nv_bfloat16* xs, uint32_t i) {
    return __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(xs)[i] << 16);
}

template <int P2> __device__ __forceinline__ float tree8(const float (&v)[P2]) {
    float t[P2];
#pragma unroll
    for (int i = 0; i < P2; ++i) t[i] = v[i];
#pragma unroll
    for (int w = P2; w > 1; w >>= 1) {
#pragma unroll
        for (int i = 0; i < w / 2; ++i) t[i] = __fadd_rn(t[2 * i], t[2 * i + 1]);
    }
    return t[0];
}

// ------------------------------------------------------------------------------------------------
// the kernel.  P2 = padded tile side = lanes cooperating on one tile (4, 8, 16 or 32).
// blockDim.x = 32 * (1 + consumer warps); warp 0 is the producer.
// ------------------------------------------------------------------------------------------------
template <typename XT, typename LT, int Q, int P2>
__global__ void __launch_bounds__(288, 2)
fused_compress_kernel(const FusedParams p) {
    constexpr bool IN_PLACE = sizeof(XT) == 4;
    constexpr uint32_t PER = 32 / Q;          // elements per packed word
    constexpr uint32_t NQ = PER / 4;          // quads per word
    constexpr uint32_t TG = 32 / P2;          // tiles per warp step

    extern __shared__ __align__(128) unsigned char smem[];
    const Shape& s = p.s;
    const uint32_t K = p.pl.stages, D = p.pl.lag;
    const uint32_t stage_bytes = p.pl.stage_bytes;
    unsigned char* stages = smem;
    uint32_t* table = reinterpret_cast<uint32_t*>(smem + (size_t)K * stage_bytes);
    FusedCtl* ctl = reinterpret_cast<FusedCtl*>(reinterpret_cast<unsigned char*>(table) + ((s.TPP * 4u + 15u) & ~15u));

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t NW = (blockDim.x >> 5) - 1;
    const uint32_t G = gridDim.x;
    const uint64_t total = p.total_chunks;
    const uint32_t n_my = blockIdx.x < total ? (uint32_t)((total - blockIdx.x + G - 1) / G) : 0u;

    // ---- set-up: tile table, barriers ----
    for (uint32_t idx = threadIdx.x; idx < s.TPP; idx += blockDim.x) {
        const uint32_t bh = idx / s.Wb, bw = idx - bh * s.Wb;
        const uint32_t rows = min(s.B, s.H - bh * s.B), cols = min(s.B, s.W - bw * s.B);
        table[idx] = (bh * s.B * s.W + bw * s.B) | ((rows - 1) << 22) | ((cols - 1) << 27);
    }
    if (threadIdx.x == 0) {
        for (uint32_t i = 0; i < K; ++i) {
            mbar_init(&ctl->full[i], 1);
            mbar_init(&ctl->empty[i], NW);
            ctl->kmin[i] = 0;
            ctl->kmax[i] = 0;
            ctl->done[i] = 0;
        }
        ctl->failed = 0;
        fence_barrier_init();
    }
    __syncthreads();

    if (warp == 0) {
        // ================= producer =================
        if (lane == 0) {
            for (uint32_t it = 0; it < n_my; ++it) {
                const uint32_t st = it % K;
                if (it >= K && !wait_barrier(&ctl->empty[st], ((it / K) - 1) & 1, p, ctl)) break;
                const Chunk c = get_chunk(p, blockIdx.x + it * G);
                const uint32_t bytes = c.nelem * (uint32_t)sizeof(XT);
                const XT* src = reinterpret_cast<const XT*>(p.x) + ((size_t)c.n * s.CHW + c.e0);
                mbar_arrive_expect_tx(&ctl->full[st], bytes);
                bulk_load(stages + (size_t)st * stage_bytes, src, bytes, &ctl->full[st]);
            }
        }
        return;
    }

    // ================= consumers =================
    const uint32_t cw = warp - 1;
    const uint32_t sub = lane / P2, col = lane % P2;
    const uint32_t rot = (NQ > 1) ? ((lane / (8 / NQ)) % NQ) : 0u;
    LT* lfc_out = reinterpret_cast<LT*>(p.lfc);
    bool alive = true;

    for (uint32_t it = 0; it < n_my + D; ++it) {
        // ---------------- half 1: block means, residuals, extremes ----------------
        if (it < n_my) {
            const uint32_t st = it % K;
            const Chunk c = get_chunk(p, blockIdx.x + it * G);
            XT* xs = reinterpret_cast<XT*>(stages + (size_t)st * stage_bytes);
            float* rs = IN_PLACE ? reinterpret_cast<float*>(xs)
                                 : reinterpret_cast<float*>(stages + (size_t)st * stage_bytes + p.pl.chunk_elems * sizeof(XT));
            if (alive) alive = wait_barrier(&ctl->full[st], (it / K) & 1, p, ctl);
            float rmin = 3.402823466e+38f, rmax = -3.402823466e+38f;
            if (alive) {
                LT* lfc_n = lfc_out + (size_t)c.n * s.C * s.TPP;
                const uint32_t ngroups = (c.ntiles + TG - 1) / TG;
                for (uint32_t g = (cw + it) % NW; g < ngroups; g += NW) {
                    const uint32_t t = g * TG + sub;
                    const bool tile_ok = t < c.ntiles;
                    const uint32_t ts = c.tile0 + (tile_ok ? t : 0u);
                    const uint32_t plane = fdiv(ts, p.by_tpp);
                    const uint32_t entry = table[ts - plane * s.TPP];
                    const uint32_t rows = ((entry >> 22) & 31u) + 1u, cols = (entry >> 27) + 1u;
                    const uint32_t o = plane * s.HW + (entry & 0x3FFFFFu) - c.e0 + col;
                    const bool lane_ok = tile_ok && col < cols;
                    float v[P2];
#pragma unroll
                    for (int r = 0; r < P2; ++r)
                        v[r] = (lane_ok && (uint32_t)r < rows) ? stage_load<XT>(xs, o + r * s.W) : 0.f;
                    float sum = tree8<P2>(v);
#pragma unroll
                    for (int m = 1; m < P2; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
                    const uint32_t cnt = rows * cols;
                    const float cntf = (float)cnt;
                    float mean;
                    if ((cnt & (cnt - 1)) == 0)
                        mean = __fmul_rn(sum, __uint_as_float(0x7F000000u - __float_as_uint(cntf)));   // exact 1/2^k
                    else
                        mean = __fdiv_rn(sum, cntf);
                    const float stored = Elem<LT>::round(mean);
                    if (tile_ok && col == 0) Elem<LT>::store(lfc_n + ts, mean);
                    if (lane_ok) {
#pragma unroll
                        for (int r = 0; r < P2; ++r) {
                            if ((uint32_t)r < rows) {
                                const float res = __fsub_rn(v[r], stored);
                                rs[o + r * s.W] = res;
                                rmin = fminf(rmin, res);
                                rmax = fmaxf(rmax, res);
                            }
                        }
                    }
                }
            }
            // fold the warp's extremes into the stage, then the stage into the sample
            const uint32_t kmin = __reduce_max_sync(0xFFFFFFFFu, ~float_key(rmin));
            const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, float_key(rmax));
            __syncwarp();
            if (lane == 0) {
                atomicMax(&ctl->kmin[st], kmin);
                atomicMax(&ctl->kmax[st], kmax);
                __threadfence_block();
                if (atomicAdd(&ctl->done[st], 1u) == NW - 1) {
                    // last consumer warp of this CTA on this chunk: publish to the sample slot
                    __threadfence_block();
                    const uint32_t smin = atomicExch(&ctl->kmin[st], 0u);
                    const uint32_t smax = atomicExch(&ctl->kmax[st], 0u);
                    ctl->done[st] = 0u;
                    uint32_t* slot = p.ws + WS_HEADER_WORDS + (size_t)c.n * WS_SLOT_WORDS;
                    if (*(volatile uint32_t*)&ctl->failed == 0u) {
                        atomicMax(slot + 0, smin);
                        atomicMax(slot + 1, smax);
                        __threadfence();
                        if (atomicAdd(slot + 2, 1u) == p.expected_arrivals - 1u) {
                            __threadfence();
                            const float lo = key_float(~ld_relaxed_u32(slot + 0));
                            const float hi = key_float(ld_relaxed_u32(slot + 1));
                            const QParams qp = make_qparams(lo, hi, Q);
                            p.stats[2 * (size_t)c.n + 0] = qp.delta;
                            p.stats[2 * (size_t)c.n + 1] = qp.step;
                            const uint64_t word = ((uint64_t)(__float_as_uint(qp.scale) | 0x80000000u) << 32) |
                                                  (uint64_t)__float_as_uint(qp.delta);
                            st_release_u64(reinterpret_cast<uint64_t*>(slot + 4), word);
                        }
                    }
                }
            }
        }
        // ---------------- half 2: quantise and pack the chunk seen `lag` iterations ago ----------------
        if (it >= D && it - D < n_my) {
            const uint32_t jt = it - D;
            const uint32_t st = jt % K;
            const Chunk c = get_chunk(p, blockIdx.x + jt * G);
            const float* rs = IN_PLACE ? reinterpret_cast<const float*>(stages + (size_t)st * stage_bytes)
                                       : reinterpret_cast<const float*>(stages + (size_t)st * stage_bytes +
                                                                        p.pl.chunk_elems * sizeof(XT));
            uint64_t word = 0;
            if (alive) {
                if (lane == 0) {
                    const uint64_t* pw = reinterpret_cast<const uint64_t*>(p.ws + WS_HEADER_WORDS + (size_t)c.n * WS_SLOT_WORDS + 4);
                    uint32_t polls = 0;
                    uint64_t t0 = 0;
                    while (true) {
                        word = ld_relaxed_u64(pw);
                        if (word >> 63) break;
                        if ((++polls & 63u) == 0) {
                            if (give_up(p, ctl, t0)) {
                                record_failure(p, ctl, c.n + 1u);
                                word = 0;
                                break;
                            }
                            __nanosleep(64);
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
                const uint64_t base = rng_sample_base(p.seed, c.n);
                const uint32_t nunits = c.nelem / PER;
                uint32_t* out = p.packed + ((uint64_t)c.n * s.CHW + c.e0) / PER;
                const uint32_t g0 = c.e0 >> 2;
                for (uint32_t u = ((cw + it) % NW) * 32u + lane; u < nunits; u += NW * 32u) {
                    const float4* src = reinterpret_cast<const float4*>(rs + (size_t)u * PER);
                    uint32_t acc = 0;
#pragma unroll
                    for (uint32_t k = 0; k < NQ; ++k) {
                        const uint32_t qi = (k + rot) % NQ;
                        const float4 r4 = src[qi];
                        const uint64_t z = rng_group(base, g0 + u * NQ + qi);
                        acc += quant4<Q>(r4.x, r4.y, r4.z, r4.w, delta, scale, z) << ((4 * Q * qi) & 31u);
                    }
                    __stcs(out + u, acc);
                }
            }
            // release the stage to the producer
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->empty[st]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side: planning and launch
// ------------------------------------------------------------------------------------------------
inline FastDiv host_fastdiv(uint32_t d) {
    FastDiv f;
    f.d = d;
    uint32_t sh = 0;
    while ((1ull << sh) < d) ++sh;
    f.shift = 31 + sh;
    f.mul = (uint32_t)((((1ull << f.shift) - 1) / d) + 1);
    return f;
}

inline uint32_t gcd_u32(uint32_t a, uint32_t b) {
    while (b) {
        const uint32_t t = a % b;
        a = b;
        b = t;
    }
    return a;
}

constexpr int FUSED_CONSUMER_WARPS = 8;
constexpr int FUSED_THREADS = 32 * (1 + FUSED_CONSUMER_WARPS);

struct DeviceInfo {
    int sms;
    int smem_optin;
    bool ok;
    int dev;
};

// What the planners need to know about a device is asked from the runtime once per device and kept (a few words
// of host memory per device ordinal): a call of div_compress then costs one cudaGetDevice instead of attribute,
// occupancy and function-attribute queries.  Ordinals of DEVICE_CACHE_SLOTS or above are served without the cache.
constexpr int DEVICE_CACHE_SLOTS = 64;
inline DeviceInfo device_info() {
    static std::atomic<int> cached_sms[DEVICE_CACHE_SLOTS];
    static std::atomic<int> cached_smem[DEVICE_CACHE_SLOTS];
    DeviceInfo di = {0, 0, false, -1};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return di;
    }
    di.dev = dev;
    const bool slot = dev >= 0 && dev < DEVICE_CACHE_SLOTS;
    if (slot) {
        di.sms = cached_sms[dev].load(std::memory_order_acquire);
        di.smem_optin = cached_smem[dev].load(std::memory_order_acquire);
        if (di.sms > 0 && di.smem_optin > 0) {
            di.ok = true;
            return di;
        }
    }
    if (cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&di.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
        cudaGetLastError();
        return di;
    }
    if (slot) {
        cached_smem[dev].store(di.smem_optin, std::memory_order_release);
        cached_sms[dev].store(di.sms, std::memory_order_release);
    }
    di.ok = true;
    return di;
}

// cudaFuncAttributeMaxDynamicSharedMemorySize of one kernel: set once per device and size, not once per launch.
// `seen` is the per-kernel table of what has been set on each device; an entry also names the kernel it is
// about, so that a table shared by accident (two copies of the library in one process) is never trusted for
// another copy's kernel.
struct SmemSeen {
    std::atomic<const void*> fn;
    std::atomic<int> bytes;
};
inline bool ensure_dynamic_smem(const void* kern, int bytes, SmemSeen* seen) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    const bool slot = dev >= 0 && dev < DEVICE_CACHE_SLOTS;
    if (slot && seen[dev].fn.load(std::memory_order_acquire) == kern && seen[dev].bytes.load(std::memory_order_acquire) >= bytes)
        return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    if (slot) {
        seen[dev].fn.store(nullptr, std::memory_order_release);
        seen[dev].bytes.store(bytes, std::memory_order_release);
        seen[dev].fn.store(kern, std::memory_order_release);
    }
    return true;
}

// Decide whether and how the fused kernel runs a descriptor.  DIV_OK: plan filled in.
inline div_status plan_fused(const div_desc* d, const Shape& s, FusedPlan* out) {
    const uint32_t sx = d->x_dtype == DIV_F32 ? 4u : 2u;
    const uint32_t per = 32u / (uint32_t)d->qbits;
    if (s.P2 < 4 || s.P2 > 32) return DIV_ERR_PARAM;
    if (s.TPP > 4096 || s.HW >= (1u << 22)) return DIV_ERR_PARAM;
    // chunk boundaries must fall on packed-word boundaries and on 16-byte boundaries of x
    uint32_t unit = per;
    const uint32_t tma = 16u / sx;
    unit = unit / gcd_u32(unit, tma) * tma;
    if (s.CHW % unit != 0) return DIV_ERR_PARAM;
    const DeviceInfo di = device_info();
    if (!di.ok || di.sms < 1) return DIV_ERR_CUDA;

    const uint32_t elem_bytes = sx == 4 ? 4u : 6u;             // bf16 keeps a separate fp32 residual copy
    const uint32_t table_bytes = ((s.TPP * 4u + 15u) & ~15u) + (uint32_t)sizeof(FusedCtl) + 128u;
    for (int ctas_per_sm = 2; ctas_per_sm >= 1; --ctas_per_sm) {
        const uint32_t budget = (uint32_t)((di.smem_optin - 2048) / ctas_per_sm) - (ctas_per_sm == 2 ? 1024u : 0u);
        if (budget <= table_bytes + 4096) continue;
        for (uint32_t lag = 1; lag <= 4; ++lag) {
            const uint32_t stages = lag + 3;
            const uint32_t max_elems = ((budget - table_bytes) / stages / elem_bytes) & ~31u;
            FusedPlan pl = FusedPlan();
            pl.threads = FUSED_THREADS;
            pl.stages = (int32_t)stages;
            pl.lag = (int32_t)lag;
            pl.p2 = s.P2;
            const uint32_t band = s.B * s.W;                   // elements of a full tile row
            if ((uint64_t)s.HW <= max_elems / 2 || s.HW % unit != 0 || band > max_elems) {
                // whole planes per chunk
                const uint32_t step = unit / gcd_u32(unit, s.HW);
                uint32_t cb = max_elems / s.HW / step * step;
                if (cb == 0) continue;
                if (cb > s.C) cb = (s.C + step - 1) / step * step;
                pl.mode = 1;
                pl.cb = cb;
                pl.cpp = 0;
                pl.chunk_elems = cb * s.HW;
                pl.chunks_per_sample = (s.C + cb - 1) / cb;
            } else {
                // runs of tile rows inside one plane
                const uint32_t step = unit / gcd_u32(unit, band);
                uint32_t cb = max_elems / band / step * step;
                if (cb == 0) continue;
                if (cb > s.Hb) cb = s.Hb;
                pl.mode = 0;
                pl.cb = cb;
                pl.cpp = (s.Hb + cb - 1) / cb;
                pl.chunk_elems = cb * band;
                pl.chunks_per_sample = pl.cpp * s.C;
            }
            const uint64_t total_chunks = (uint64_t)pl.chunks_per_sample * s.N;
            if (total_chunks >= (1ull << 31)) return DIV_ERR_PARAM;
            pl.stage_bytes = (pl.chunk_elems * elem_bytes + 127u) & ~127u;
            pl.smem_bytes = (int32_t)(stages * pl.stage_bytes + table_bytes);
            uint64_t grid = (uint64_t)di.sms * ctas_per_sm;
            if (grid > total_chunks) grid = total_chunks;
            pl.grid = (int32_t)grid;
            // a CTA may hold at most `lag` + 1 chunks of one sample before it waits for that sample
            if ((pl.chunks_per_sample + grid - 1) / grid > lag) continue;
            *out = pl;
            return DIV_OK;
        }
    }
    return DIV_ERR_PARAM;
}

template <typename XT, typename LT, int Q, int P2>
inline div_status launch_fused(const FusedParams& prm, cudaStream_t st) {
    auto kern = fused_compress_kernel<XT, LT, Q, P2>;
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

template <typename XT, typename LT, int Q>
inline div_status launch_fused_p2(const FusedParams& prm, cudaStream_t st) {
    switch (prm.pl.p2) {
        case 4: return launch_fused<XT, LT, Q, 4>(prm, st);
        case 8: return launch_fused<XT, LT, Q, 8>(prm, st);
        case 16: return launch_fused<XT, LT, Q, 16>(prm, st);
        case 32: return launch_fused<XT, LT, Q, 32>(prm, st);
    }
    return DIV_ERR_PARAM;
}

inline div_status compress_fused(const div_desc* d, const Shape& s, const div_layout& lo, const FusedPlan& pl,
                                 const void* x, uint8_t* blob, uint32_t* ws, uint64_t seed, cudaStream_t st,
                                 uint32_t expected_arrivals = 0, uint64_t timeout_ns = 0) {
    FusedParams prm;
    prm.s = s;
    prm.pl = pl;
    prm.by_S = host_fastdiv(pl.chunks_per_sample);
    prm.by_cpp = host_fastdiv(pl.cpp ? pl.cpp : 1u);
    prm.by_tpp = host_fastdiv(s.TPP);
    prm.x = x;
    prm.lfc = blob + lo.lfc_off;
    prm.packed = reinterpret_cast<uint32_t*>(blob + lo.packed_off);
    prm.stats = reinterpret_cast<float*>(blob + lo.stats_off);
    prm.ws = ws;
    prm.seed = seed;
    prm.total_chunks = (uint64_t)pl.chunks_per_sample * s.N;
    prm.expected_arrivals = expected_arrivals ? expected_arrivals : pl.chunks_per_sample;
    prm.timeout_ns = timeout_ns ? timeout_ns : 2000000000ull;   // 2 s
    typedef __nv_bfloat16 bf16;
#define DIVK_Q_SWITCH(XT, LT)                                         \
    switch (d->qbits) {                                               \
        case 1: return launch_fused_p2<XT, LT, 1>(prm, st);           \
        case 2: return launch_fused_p2<XT, LT, 2>(prm, st);           \
        case 4: return launch_fused_p2<XT, LT, 4>(prm, st);           \
        case 8: return launch_fused_p2<XT, LT, 8>(prm, st);           \
    }                                                                 \
    return DIV_ERR_PARAM;
    if (d->x_dtype == DIV_F32) {
        if (d->lfc_dtype == DIV_F32) { DIVK_Q_SWITCH(float, float) }
        DIVK_Q_SWITCH(float, bf16)
    }
    if (d->lfc_dtype == DIV_F32) { DIVK_Q_SWITCH(bf16, float) }
    DIVK_Q_SWITCH(bf16, bf16)
#undef DIVK_Q_SWITCH
}

}  // namespace divk
