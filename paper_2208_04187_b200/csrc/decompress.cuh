// Decompress kernels (DIVISION Sec. 4.2, Eq. 10; Algorithm 1, backward loop):
//   x_hat = UpSampling(H^L) + (Delta * V^H + delta), rounded to the activation dtype.
// One fused pass: unpack, dequantise, add the nearest-upsampled low-frequency value, store.
#pragma once

#include "common.cuh"
#include "twopass.cuh"   // Shape

namespace divk {

// ---------------------------------------------------------------------------------------------
// general kernel: one thread per packed word, any shape
// ---------------------------------------------------------------------------------------------
template <typename XT, typename LT, int Q>
__global__ void __launch_bounds__(256)
decompress_general_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                          const float* __restrict__ stats, XT* __restrict__ xhat, Shape s, uint64_t nwords) {
    constexpr uint32_t PER = 32 / Q;
    constexpr uint32_t MASK = (Q == 32) ? 0xFFFFFFFFu : ((1u << Q) - 1u);
    const uint64_t word = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (word >= nwords) return;
    uint64_t i = word * PER;
    uint32_t n = (uint32_t)(i / s.CHW);
    uint32_t e = (uint32_t)(i - (uint64_t)n * s.CHW);
    uint32_t plane = e / s.HW;
    uint32_t rem = e - plane * s.HW;
    uint32_t h = rem / s.W, w = rem - h * s.W;
    const uint32_t bits = packed[word];
    uint32_t cur_n = 0xFFFFFFFFu;
    float delta = 0.f, step = 0.f;
    for (uint32_t j = 0; j < PER && i < s.total; ++j, ++i) {
        if (n != cur_n) {
            delta = stats[2 * (size_t)n];
            step = stats[2 * (size_t)n + 1];
            cur_n = n;
        }
        const size_t lidx = ((size_t)n * s.C + plane) * s.TPP + (h / s.B) * s.Wb + (w / s.B);
        const float l = Elem<LT>::load(lfc + lidx);
        Elem<XT>::store(xhat + i, reconstruct((bits >> (j * Q)) & MASK, step, delta, l));
        if (++w == s.W) {
            w = 0;
            if (++h == s.H) {
                h = 0;
                if (++plane == s.C) {
                    plane = 0;
                    ++n;
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// vector kernel: W % 4 == 0, B a power of two >= 4 (so that 4 consecutive elements share a tile, and so do
// the 4 rows of an aligned row group).  One thread produces 4 quads (4 elements each, one 16-byte or 8-byte
// store): the same 4 columns of 4 consecutive rows, which share one low-frequency value and one set of index
// arithmetic.  Threads of a warp take consecutive quads of a row group, so every store instruction of a warp
// writes contiguous spans.
// grid = (ceil(C * ceil(H/4) * (W/4) / 256), N)
// ---------------------------------------------------------------------------------------------
struct DecFast {
    uint32_t qps;        // quads per sample = CHW / 4
    uint32_t C, TPP, Wb;
    uint32_t log2B;
    uint32_t H;
    uint32_t hwq, wq;    // quads per plane and per row
    uint32_t ipp;        // work items per plane = ceil(H/4) * (W/4)
    uint32_t hq_count;   // ceil(H/4): SPREAD items take the rows hq, hq + hq_count, hq + 2 hq_count, hq + 3 hq_count
    uint32_t items;      // work items per sample = C * ipp
    FastDiv by_ipp;      // / ipp
    FastDiv by_wq;       // / (W/4)
};

template <typename XT> struct Quad;
template <> struct Quad<float> {
    static __device__ __forceinline__ void store(float* p, float a, float b, float c, float d) {
        __stcs(reinterpret_cast<float4*>(p), make_float4(a, b, c, d));
    }
};
template <> struct Quad<__nv_bfloat16> {
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float a, float b, float c, float d) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
        uint2 v;
        v.x = *reinterpret_cast<uint32_t*>(&lo);
        v.y = *reinterpret_cast<uint32_t*>(&hi);
        __stcs(reinterpret_cast<uint2*>(p), v);
    }
};

// Dequantisation through a table (Sec. 4.2: H^H_hat = Delta * V^H + delta).  A sample has only 2^Q
// different values of fl(fl(Delta * code) + delta), so a CTA (which works inside one sample) builds them
// once in shared memory, indexed by the packed bits of several codes at a time:
//   Q = 1: 4 codes (a nibble)  -> 16 entries of 4 values      Q = 2: 4 codes (a byte) -> 256 entries of 4 values
//   Q = 4: 2 codes (a byte)    -> 256 entries of 2 values     Q = 8: 1 code           -> 256 entries of 1 value
template <int Q> struct DeqTable;
template <> struct DeqTable<1> {
    float4 t[16];
    __device__ __forceinline__ void build(float step, float delta) {
        if (threadIdx.x < 16) {
            const uint32_t i = threadIdx.x;
            t[i] = make_float4(dequantise(i & 1u, step, delta), dequantise((i >> 1) & 1u, step, delta),
                               dequantise((i >> 2) & 1u, step, delta), dequantise((i >> 3) & 1u, step, delta));
        }
    }
    __device__ __forceinline__ float4 quad(uint32_t bits) const { return t[bits & 15u]; }
};
template <> struct DeqTable<2> {
    float4 t[256];
    __device__ __forceinline__ void build(float step, float delta) {
        const uint32_t i = threadIdx.x;
        if (i < 256)
            t[i] = make_float4(dequantise(i & 3u, step, delta), dequantise((i >> 2) & 3u, step, delta),
                               dequantise((i >> 4) & 3u, step, delta), dequantise((i >> 6) & 3u, step, delta));
    }
    __device__ __forceinline__ float4 quad(uint32_t bits) const { return t[bits & 255u]; }
};
template <> struct DeqTable<4> {
    float2 t[256];
    __device__ __forceinline__ void build(float step, float delta) {
        const uint32_t i = threadIdx.x;
        if (i < 256) t[i] = make_float2(dequantise(i & 15u, step, delta), dequantise((i >> 4) & 15u, step, delta));
    }
    __device__ __forceinline__ float4 quad(uint32_t bits) const {
        const float2 a = t[bits & 255u], b = t[(bits >> 8) & 255u];
        return make_float4(a.x, a.y, b.x, b.y);
    }
};
template <> struct DeqTable<8> {
    float t[256];
    __device__ __forceinline__ void build(float step, float delta) {
        const uint32_t i = threadIdx.x;
        if (i < 256) t[i] = dequantise(i, step, delta);
    }
    __device__ __forceinline__ float4 quad(uint32_t bits) const {
        return make_float4(t[bits & 255u], t[(bits >> 8) & 255u], t[(bits >> 16) & 255u], t[bits >> 24]);
    }
};

// the packed bits of quad number `quad` (global numbering) of the code stream
template <int Q>
__device__ __forceinline__ uint32_t quad_bits(const uint32_t* __restrict__ packed, uint64_t quad) {
    if (Q == 2) return __ldg(reinterpret_cast<const uint8_t*>(packed) + quad);
    if (Q == 4) return __ldg(reinterpret_cast<const uint16_t*>(packed) + quad);
    if (Q == 8) return __ldg(packed + quad);
    return (__ldg(reinterpret_cast<const uint8_t*>(packed) + (quad >> 1)) >> (4u * (uint32_t)(quad & 1u))) & 15u;
}

// SPREAD: where a row is not a whole number of 32-byte sectors (28 fp32 columns: 112 bytes) the 4 rows of a work
// item are taken hq_count rows apart instead of next to each other, so that the lanes of a warp write consecutive
// rows with one store instruction (whole sectors) instead of pieces 4 rows apart; the rows of an item then lie in
// different tiles, each with its own low-frequency value.
template <typename XT, typename LT, int Q, int QPT, bool SPREAD>
__global__ void __launch_bounds__(256)
decompress_quad_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                       const float* __restrict__ stats, XT* __restrict__ xhat, DecFast d) {
    static_assert(QPT == 4, "a work item is 4 rows high");
    __shared__ DeqTable<Q> table;
    const uint32_t n = blockIdx.y;
    table.build(__ldg(stats + 2 * (size_t)n + 1), __ldg(stats + 2 * (size_t)n));
    __syncthreads();
    const uint32_t item = blockIdx.x * 256u + threadIdx.x;
    if (item >= d.items) return;
    const uint32_t plane = fdiv(item, d.by_ipp);
    const uint32_t rem = item - plane * d.ipp;
    const uint32_t hq = fdiv(rem, d.by_wq);
    const uint32_t wq = rem - hq * d.wq;
    const uint32_t h0 = SPREAD ? hq : hq * 4u;
    const uint32_t hstep = SPREAD ? d.hq_count : 1u;
    const LT* lfc_p = lfc + ((size_t)n * d.C + plane) * d.TPP + ((wq * 4u) >> d.log2B);
    const uint64_t quad0 = (uint64_t)n * d.qps + plane * d.hwq + h0 * d.wq + wq;      // first row's quad
    const uint32_t qstep = hstep * d.wq;
    float lf[4];
    uint32_t bits[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const uint32_t h = h0 + (uint32_t)r * hstep;
        bits[r] = 0u;
        lf[r] = 0.f;
        if (h < d.H) {
            bits[r] = quad_bits<Q>(packed, quad0 + (uint32_t)r * qstep);
            if (SPREAD || r == 0) lf[r] = Elem<LT>::load(lfc_p + (h >> d.log2B) * d.Wb);
        }
        if (!SPREAD && r > 0) lf[r] = lf[0];              // 4 neighbouring rows from a multiple of 4 on share a tile
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        if (h0 + (uint32_t)r * hstep < d.H) {
            const float4 hq4 = table.quad(bits[r]);
            Quad<XT>::store(xhat + (quad0 + (uint32_t)r * qstep) * 4u, __fadd_rn(lf[r], hq4.x), __fadd_rn(lf[r], hq4.y),
                            __fadd_rn(lf[r], hq4.z), __fadd_rn(lf[r], hq4.w));
        }
    }
}

// ---------------------------------------------------------------------------------------------
// line kernel: 1-D maps (H == 1), W % 4 == 0, B a power of two >= 4.  One thread produces QPT quads, 256 quads
// apart; a quad's block is (position in the row) / B.
// grid = (ceil(quads_per_sample / (256*QPT)), N)
// ---------------------------------------------------------------------------------------------
struct DecLine {
    uint32_t qps;        // quads per sample = C * W / 4
    uint32_t C, Wb;
    uint32_t qpr;        // quads per row
    uint32_t log2lpt;    // log2(B / 4)
    FastDiv by_qpr;
};
template <typename XT, typename LT, int Q, int QPT>
__global__ void __launch_bounds__(256)
decompress_line_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                       const float* __restrict__ stats, XT* __restrict__ xhat, DecLine d) {
    __shared__ DeqTable<Q> table;
    const uint32_t n = blockIdx.y;
    table.build(__ldg(stats + 2 * (size_t)n + 1), __ldg(stats + 2 * (size_t)n));
    __syncthreads();
    const uint64_t sample_quad0 = (uint64_t)n * d.qps;
    const LT* lfc_n = lfc + (size_t)n * d.C * d.Wb;
    const uint32_t q0 = blockIdx.x * (256u * QPT) + threadIdx.x;
    uint32_t bits[QPT];
    float lf[QPT];
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < d.qps) {
            bits[k] = quad_bits<Q>(packed, sample_quad0 + q);
            const uint32_t row = fdiv(q, d.by_qpr);
            lf[k] = Elem<LT>::load(lfc_n + (row * d.Wb + ((q - row * d.qpr) >> d.log2lpt)));
        }
    }
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < d.qps) {
            const float4 hq = table.quad(bits[k]);
            Quad<XT>::store(xhat + (sample_quad0 + q) * 4u, __fadd_rn(lf[k], hq.x), __fadd_rn(lf[k], hq.y),
                            __fadd_rn(lf[k], hq.z), __fadd_rn(lf[k], hq.w));
        }
    }
}

// ---------------------------------------------------------------------------------------------
// flat kernel: any W and B, sample size a multiple of 4 elements, planes of at most FLAT_MAX_HW
// elements.  One thread produces QPT quads of 4 consecutive elements (global flat order), which may
// lie in different tiles, rows or planes.  Where the 4 low-frequency values of a quad sit repeats every
// lcm(HW, 4) elements, so a table in shared memory (built once per CTA) holds, for every quad of one such
// period, the 4 offsets (plane inside the period * tiles per plane + tile inside the plane) as 16-bit numbers:
// one 8-byte load per quad instead of a walk over positions.  The low-frequency values of the planes a CTA
// touches are staged in shared memory too.
// grid = (ceil(quads_per_sample / (256*QPT)), N), dynamic shared memory = flat_smem_bytes()
// ---------------------------------------------------------------------------------------------
constexpr uint32_t FLAT_MAX_HW = 8192;

struct DecFlat {
    uint32_t qps;        // quads per sample = CHW / 4
    uint32_t C, TPP, Wb, HW, W, B;
    uint32_t table_words;    // 32-bit words the quad table takes in shared memory
    uint32_t planes_per_cta; // upper bound of the planes one CTA touches
    uint32_t period;         // quads after which the quad table repeats
    uint32_t period_planes;  // planes one period covers (1, 2 or 4)
    FastDiv by_hw, by_w, by_b, by_period;
};
// planes a run of `elems` consecutive elements can touch, and the dynamic shared memory of the flat kernels
inline uint32_t flat_planes_per_cta(uint32_t elems, uint32_t hw) { return (elems + hw - 1) / hw + 1; }
inline uint32_t flat_table_words(uint32_t hw) { return (hw + 1) / 2; }            // a 16-bit tile number per position of a plane
inline uint32_t quad_period(uint32_t hw) { return hw / ((hw & 3u) == 0 ? 4u : (hw & 1u) == 0 ? 2u : 1u); }
inline uint32_t quad_period_planes(uint32_t hw) { return (hw & 3u) == 0 ? 1u : (hw & 1u) == 0 ? 2u : 4u; }
inline uint32_t quad_table_words(uint32_t hw) { return 2u * quad_period(hw); }    // 4 16-bit offsets per quad of a period
inline size_t flat_smem_bytes(uint32_t elems, uint32_t hw, uint32_t tpp) {
    return 4ull * quad_table_words(hw) + 4ull * flat_planes_per_cta(elems, hw) * tpp;
}

// entry idx of the quad table: for each of the elements 4 idx .. 4 idx + 3 of a run of planes that starts on a
// plane boundary, (plane inside the run) * TPP + tile inside the plane (fits 16 bits: at most 4 planes of at most
// FLAT_MAX_HW tiles)
__device__ __forceinline__ uint2 quad_table_entry(uint32_t idx, uint32_t HW, uint32_t W, uint32_t Wb, uint32_t TPP,
                                                  const FastDiv& by_hw, const FastDiv& by_w, const FastDiv& by_b) {
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t e = 4u * idx + (uint32_t)i;
        const uint32_t dp = fdiv(e, by_hw), pos = e - dp * HW;
        const uint32_t h = fdiv(pos, by_w), w = pos - h * W;
        o[i] = dp * TPP + fdiv(h, by_b) * Wb + fdiv(w, by_b);
    }
    return make_uint2(o[0] | (o[1] << 16), o[2] | (o[3] << 16));
}

template <typename XT, typename LT, int Q, int QPT>
__global__ void __launch_bounds__(256)
decompress_flat_kernel(const LT* __restrict__ lfc, const uint32_t* __restrict__ packed,
                       const float* __restrict__ stats, XT* __restrict__ xhat, DecFlat d) {
    extern __shared__ __align__(16) uint32_t flat_smem[];
    uint2* quad_of = reinterpret_cast<uint2*>(flat_smem);            // quad inside a period -> where its 4 low-frequency values sit
    float* lfc_s = reinterpret_cast<float*>(flat_smem + d.table_words);   // low-frequency values of this CTA's planes
    __shared__ DeqTable<Q> table;
    const uint32_t n = blockIdx.y;
    // the codes of this thread's quads are asked for first: their trip to memory overlaps the set-up below
    const uint64_t sample_quad0 = (uint64_t)n * d.qps;
    const uint32_t q0 = blockIdx.x * (256u * QPT) + threadIdx.x;
    uint32_t bits[QPT];
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        bits[k] = q < d.qps ? quad_bits<Q>(packed, sample_quad0 + q) : 0u;
    }
    table.build(__ldg(stats + 2 * (size_t)n + 1), __ldg(stats + 2 * (size_t)n));
    for (uint32_t idx = threadIdx.x; idx < d.period; idx += 256u)
        quad_of[idx] = quad_table_entry(idx, d.HW, d.W, d.Wb, d.TPP, d.by_hw, d.by_w, d.by_b);
    const uint32_t e_first = blockIdx.x * (1024u * QPT);
    const uint32_t plane0 = fdiv(e_first, d.by_hw);
    const uint32_t nplanes = min(d.planes_per_cta, d.C - plane0);
    const LT* lfc_n = lfc + ((size_t)n * d.C + plane0) * d.TPP;
    for (uint32_t idx = threadIdx.x; idx < nplanes * d.TPP; idx += 256u) lfc_s[idx] = Elem<LT>::load(lfc_n + idx);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < QPT; ++k) {
        const uint32_t q = q0 + k * 256u;
        if (q < d.qps) {
            const float4 hq = table.quad(bits[k]);
            const float hv[4] = {hq.x, hq.y, hq.z, hq.w};
            const uint32_t grp = fdiv(q, d.by_period);
            const uint2 ent = quad_of[q - grp * d.period];
            // the period may start before the first plane staged here; the elements of this CTA do not
            const int base = ((int)(grp * d.period_planes) - (int)plane0) * (int)d.TPP;
            float v[4];
            v[0] = __fadd_rn(lfc_s[base + (int)(ent.x & 0xFFFFu)], hv[0]);
            v[1] = __fadd_rn(lfc_s[base + (int)(ent.x >> 16)], hv[1]);
            v[2] = __fadd_rn(lfc_s[base + (int)(ent.y & 0xFFFFu)], hv[2]);
            v[3] = __fadd_rn(lfc_s[base + (int)(ent.y >> 16)], hv[3]);
            Quad<XT>::store(xhat + (sample_quad0 + q) * 4u, v[0], v[1], v[2], v[3]);
        }
    }
}

}  // namespace divk
