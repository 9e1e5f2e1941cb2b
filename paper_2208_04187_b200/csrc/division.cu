// Host side of the C ABI declared in include/division.h: argument checks, byte-layout arithmetic,
// kernel selection and launches.  Nothing here allocates device memory; the only device memory the library
// owns is the fixed scratch array of div_compress_static.
#include "../../include/division.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "common.cuh"
#include "decompress.cuh"
#include "fused.cuh"
#include "fused_v.cuh"
#include "lagged.cuh"
#include "lines.cuh"
#include "masks.cuh"
#include "planegroup.cuh"
#include "planes.cuh"
#include "staged.cuh"
#include "twopass.cuh"
#include "volume.cuh"

namespace {

using namespace divk;
typedef __nv_bfloat16 bf16;

constexpr uint64_t SECTION_ALIGN = 128;
constexpr uint32_t DIV_FLAG_ALL = DIV_FLAG_FORCE_TWO_PASS | DIV_FLAG_NO_STRIP_KERNEL | DIV_FLAG_NO_LAGGED_KERNEL |
                                  DIV_FLAG_NO_PLANE_KERNELS | DIV_FLAG_NO_LINE_KERNELS | DIV_FLAG_NO_STAGED_KERNEL |
                                  DIV_FLAG_TWO_LAUNCH_PLANES;

inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }
inline uint32_t dtype_bytes(int32_t dt) { return dt == DIV_F32 ? 4u : 2u; }

div_status check_desc(const div_desc* d) {
    if (!d) return DIV_ERR_NULL;
    if (d->n < 1 || d->c < 1 || d->h < 1 || d->w < 1) return DIV_ERR_SHAPE;
    if (d->n >= (1ll << 31) || d->c >= (1ll << 32) || d->h >= (1ll << 32) || d->w >= (1ll << 32)) return DIV_ERR_SHAPE;
    // c*h*w < 2^32 (width of the random-number counter), checked without overflow
    const unsigned __int128 chw = (unsigned __int128)d->c * (unsigned __int128)d->h * (unsigned __int128)d->w;
    if (chw >= ((unsigned __int128)1 << 32)) return DIV_ERR_SHAPE;
    if (d->block < 1) return DIV_ERR_PARAM;
    if (!(d->qbits == 1 || d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return DIV_ERR_PARAM;
    if (!(d->x_dtype == DIV_F32 || d->x_dtype == DIV_BF16)) return DIV_ERR_PARAM;
    if (!(d->lfc_dtype == DIV_F32 || d->lfc_dtype == DIV_BF16)) return DIV_ERR_PARAM;
    return DIV_OK;
}

Shape make_shape(const div_desc* d) {
    Shape s;
    s.N = (uint32_t)d->n;
    s.C = (uint32_t)d->c;
    s.H = (uint32_t)d->h;
    s.W = (uint32_t)d->w;
    // a block larger than both sides behaves like a block equal to the larger side
    const uint32_t big = s.H > s.W ? s.H : s.W;
    s.B = (uint32_t)d->block > big ? big : (uint32_t)d->block;
    s.Hb = (s.H + s.B - 1) / s.B;
    s.Wb = (s.W + s.B - 1) / s.B;
    s.P2 = 1;
    while (s.P2 < s.B) s.P2 <<= 1;
    s.HW = s.H * s.W;
    s.CHW = s.C * s.HW;
    s.TPP = s.Hb * s.Wb;
    s.total = (uint64_t)s.N * s.CHW;
    s.tiles = (uint64_t)s.N * s.C * s.TPP;
    return s;
}

void make_layout(const div_desc* d, const Shape& s, div_layout* out) {
    out->lfc_off = 0;
    out->lfc_bytes = s.tiles * dtype_bytes(d->lfc_dtype);
    out->packed_off = align_up(out->lfc_bytes, SECTION_ALIGN);
    // ceil(total*Q/32) words; total*Q < 2^31 * 2^32 * 8 fits in 64 bits
    out->packed_bytes = ((s.total * (uint64_t)d->qbits + 31) / 32) * 4;
    out->stats_off = align_up(out->packed_off + out->packed_bytes, SECTION_ALIGN);
    out->stats_bytes = 8ull * s.N;
    out->total_bytes = out->stats_off + out->stats_bytes;
    out->closed_form_bytes = out->lfc_bytes + out->packed_bytes + out->stats_bytes;
    out->raw_bytes = s.total * dtype_bytes(d->x_dtype);
    out->workspace_bytes = align_up(4ull * (WS_HEADER_WORDS + (uint64_t)WS_SLOT_WORDS * s.N), 256);
}

// per-plane groups: the same sections, but the stats section holds one bfloat16 pair (4 bytes) per plane and
// no scratch is needed
void make_layout_pg(const div_desc* d, const Shape& s, div_layout* out) {
    make_layout(d, s, out);
    out->stats_bytes = 4ull * s.N * s.C;
    out->total_bytes = out->stats_off + out->stats_bytes;
    out->closed_form_bytes = out->lfc_bytes + out->packed_bytes + out->stats_bytes;
    out->workspace_bytes = 0;
}
inline bool pg_shape_ok(const Shape& s) { return (uint64_t)s.N * s.C < (1ull << 31); }
inline bool pg_decompress_flat_ok(const Shape& s) {
    return (s.total % 4 == 0) && s.HW <= FLAT_MAX_HW && s.TPP <= 65535 && s.total / 4096 < 0x7FFFFFFFull;
}

FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    f.d = d;
    uint32_t s = 0;
    while ((1ull << s) < d) ++s;
    f.shift = 31 + s;
    f.mul = (uint32_t)((((1ull << f.shift) - 1) / d) + 1);
    return f;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ------------------------------------------------------------------------------------------
// dispatch helpers: runtime (dtype, dtype, Q) -> template instance
// ------------------------------------------------------------------------------------------
template <typename F>
div_status dispatch_q(int qbits, F&& f) {
    switch (qbits) {
        case 1: return f(std::integral_constant<int, 1>());
        case 2: return f(std::integral_constant<int, 2>());
        case 4: return f(std::integral_constant<int, 4>());
        case 8: return f(std::integral_constant<int, 8>());
    }
    return DIV_ERR_PARAM;
}
template <typename F>
div_status dispatch_types(int x_dtype, int lfc_dtype, F&& f) {
    if (x_dtype == DIV_F32) {
        if (lfc_dtype == DIV_F32) return f((float*)nullptr, (float*)nullptr);
        return f((float*)nullptr, (bf16*)nullptr);
    }
    if (lfc_dtype == DIV_F32) return f((bf16*)nullptr, (float*)nullptr);
    return f((bf16*)nullptr, (bf16*)nullptr);
}

inline div_status launch_status() { return cudaGetLastError() == cudaSuccess ? DIV_OK : DIV_ERR_CUDA; }

// ------------------------------------------------------------------------------------------
// two-pass compress
// ------------------------------------------------------------------------------------------
div_status compress_two_pass(const div_desc* d, const Shape& s, const div_layout& lo, const void* x, uint8_t* blob,
                             uint32_t* ws, uint64_t seed, cudaStream_t st) {
    const uint64_t nwords = lo.packed_bytes / 4;
    const uint64_t g1 = (s.tiles + 255) / 256, g2 = (nwords + 255) / 256;
    if (g1 > 0x7FFFFFFFull || g2 > 0x7FFFFFFFull) return DIV_ERR_SHAPE;
    return dispatch_types(d->x_dtype, d->lfc_dtype, [&](auto* xt, auto* lt) -> div_status {
        typedef std::remove_pointer_t<decltype(xt)> XT;
        typedef std::remove_pointer_t<decltype(lt)> LT;
        lfc_stats_kernel<XT, LT><<<(unsigned)g1, 256, 0, st>>>((const XT*)x, (LT*)(blob + lo.lfc_off), ws, s);
        if (launch_status() != DIV_OK) return DIV_ERR_CUDA;
        return dispatch_q(d->qbits, [&](auto q) -> div_status {
            quant_pack_kernel<XT, LT, decltype(q)::value><<<(unsigned)g2, 256, 0, st>>>(
                (const XT*)x, (const LT*)(blob + lo.lfc_off), ws, (uint32_t*)(blob + lo.packed_off),
                (float*)(blob + lo.stats_off), s, seed, nwords);
            return launch_status();
        });
    });
}

// ------------------------------------------------------------------------------------------
// decompress
// ------------------------------------------------------------------------------------------
constexpr int DEC_QPT = 4;
#ifndef DIVK_FLAT_QPT
#define DIVK_FLAT_QPT 8
#endif
constexpr int FLAT_QPT = DIVK_FLAT_QPT;       // quads per thread of the flat decompress kernel

// Which compress kernels run a descriptor.  Measured on the ResNet / WRN / DenseNet-shaped maps: from about
// 56 MB up with 8 x 8 blocks the staged kernel is fastest (both reads of x staged through shared memory by bulk
// copies), from about 20 MB up the lagged kernel (plain loads, several bands per lane, cheap for small strips),
// below that the strip ring kernel (shorter start-up); the general kernels take what those three cannot.
bool prefer_staged(const div_desc* d, const Shape& s) {
    return s.B == 8 && s.total * dtype_bytes(d->x_dtype) >= (56ull << 20);
}
// Maps whose planes are narrow enough for the fused small-plane kernel (W <= 32 for B = 8): measured faster than the
// strip ring and lagged kernels below 56 MiB (32 x 32 fp32, 34 MB: 19.5 against 25.8 us; 28 x 28, 58 MB: 29.7 against
// 37.0 us; 8 x 8 bf16, 10 MB: 15.2 against 20.4 us), except for bfloat16 maps from 32 MiB up (lagged 36 against 38 - 40 us).
bool prefer_planes(const div_desc* d, const Shape& s) {
    const uint64_t bytes = s.total * dtype_bytes(d->x_dtype);
    return bytes < (56ull << 20) && !(d->x_dtype == DIV_BF16 && bytes >= (32ull << 20));
}
bool prefer_lagged(const div_desc* d, const Shape& s) {
    return s.total * dtype_bytes(d->x_dtype) >= (20ull << 20);
}

struct Choice {
    int code;          // the value div_plan.fused reports
    LineGeom lg;
    SPlan sp;
    LPlan lp;
    VPlan vp;
    PlaneGeom pg;
    PlaneFusedPlan pf;
    LineFused lf;
    FusedPlan fp;
};

void choose_compress(const div_desc* d, const Shape& s, uint32_t flags, Choice* c) {
    const bool two_pass = (flags & DIV_FLAG_FORCE_TWO_PASS) != 0;
    c->code = 0;
    if (two_pass) return;
    if (!(flags & DIV_FLAG_NO_LINE_KERNELS) && plan_lines(d, s, &c->lg)) {
        c->code = (!(flags & DIV_FLAG_TWO_LAUNCH_PLANES) && line_fused_applies(d, s, c->lg, &c->lf)) ? 8 : 5;
        return;
    }
    const bool may_staged = !(flags & DIV_FLAG_NO_STAGED_KERNEL);
    const bool may_lag = !(flags & DIV_FLAG_NO_LAGGED_KERNEL);
    const bool may_strip = !(flags & DIV_FLAG_NO_STRIP_KERNEL);
    // (the preference holds only while no strip kernel is excluded: a flag set that leaves one of them in line gets it)
    if (may_staged && may_lag && may_strip && !(flags & (DIV_FLAG_NO_PLANE_KERNELS | DIV_FLAG_TWO_LAUNCH_PLANES)) &&
        prefer_planes(d, s) && plan_planes(d, s, &c->pg) && plane_fused_applies(d, s, c->pg, &c->pf)) {
        c->code = 7;
        return;
    }
    if (may_staged && prefer_staged(d, s) && plan_staged(d, s, &c->sp) == DIV_OK) {
        c->code = 6;
        return;
    }
    if (may_lag && prefer_lagged(d, s) && plan_lagged(d, s, &c->lp) == DIV_OK) {
        c->code = 3;
        return;
    }
    if (may_strip && plan_v(d, s, &c->vp) == DIV_OK) {
        c->code = 2;
        return;
    }
    if (may_lag && plan_lagged(d, s, &c->lp) == DIV_OK) {
        c->code = 3;
        return;
    }
    if (may_staged && plan_staged(d, s, &c->sp) == DIV_OK) {
        c->code = 6;
        return;
    }
    if (!(flags & DIV_FLAG_NO_PLANE_KERNELS) && plan_planes(d, s, &c->pg)) {
        c->code = (!(flags & DIV_FLAG_TWO_LAUNCH_PLANES) && plane_fused_applies(d, s, c->pg, &c->pf)) ? 7 : 4;
        return;
    }
    if (plan_fused(d, s, &c->fp) == DIV_OK) c->code = 1;
}

bool decompress_fast_ok(const Shape& s) {
    return (s.W % 4 == 0) && s.B >= 4 && (s.B & (s.B - 1)) == 0 && s.N <= 65535;
}
bool decompress_flat_ok(const Shape& s) {
    return (s.CHW % 4 == 0) && s.HW <= FLAT_MAX_HW && s.TPP <= 65535 && s.N <= 65535 && s.CHW < (1u << 31) &&
           flat_smem_bytes(4u * 256u * FLAT_QPT, s.HW, s.TPP) <= 40000;
}

}  // namespace

extern "C" {

const char* div_status_string(div_status s) {
    switch (s) {
        case DIV_OK: return "ok";
        case DIV_ERR_NULL: return "null pointer";
        case DIV_ERR_SHAPE: return "bad shape (need n,c,h,w >= 1, c*h*w < 2^32, n < 2^31)";
        case DIV_ERR_PARAM: return "bad parameter (block >= 1, qbits in {1,2,4,8}, dtype in {f32,bf16})";
        case DIV_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case DIV_ERR_CAPACITY: return "buffer too small";
        case DIV_ERR_CUDA: return "CUDA runtime error";
        case DIV_ERR_TIMEOUT: return "device-side bounded wait expired";
    }
    return "unknown status";
}

div_status div_compressed_bytes(const div_desc* desc, div_layout* out) {
    if (!desc || !out) return DIV_ERR_NULL;
    const div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    make_layout(desc, make_shape(desc), out);
    return DIV_OK;
}

div_status div_plan_query(const div_desc* desc, uint32_t flags, div_plan* out) {
    if (!desc || !out) return DIV_ERR_NULL;
    const div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    if (flags & ~DIV_FLAG_ALL) return DIV_ERR_PARAM;
    const Shape s = make_shape(desc);
    *out = div_plan();
    Choice ch;
    choose_compress(desc, s, flags, &ch);
    out->fused = ch.code;
    if (ch.code == 8) {
        out->grid = (int32_t)(ch.lf.ctas_per_sample * s.N);
        out->threads = 256;
        out->chunk_elems = (int64_t)ch.lf.rpc * s.W;
        out->chunks_per_sample = ch.lf.ctas_per_sample;
    } else if (ch.code == 5) {
        out->grid = (int32_t)((ch.lg.qps + 256 * LINE_QPT - 1) / (256 * LINE_QPT) * s.N);
        out->threads = 256;
        out->chunk_elems = 4 * LINE_QPT * 256;
    } else if (ch.code == 6) {
        out->grid = ch.sp.grid;
        out->threads = ch.sp.threads;
        out->stages = (int32_t)(ch.sp.kr + ch.sp.kq);
        out->lag = (int32_t)ch.sp.lag_steps;
        out->smem_bytes = ch.sp.smem_bytes;
        out->chunk_elems = ch.sp.chunk_elems;
        out->chunks_per_sample = ch.sp.chunks_per_sample;
    } else if (ch.code == 3) {
        out->grid = ch.lp.grid;
        out->threads = ch.lp.threads;
        out->stages = 0;
        out->lag = (int32_t)ch.lp.lag_units;
        out->smem_bytes = 0;
        out->chunk_elems = (int64_t)32 * ch.lp.bands_per_lane * 4 * s.B;       // elements of one full unit
        out->chunks_per_sample = ch.lp.units_per_sample;
    } else if (ch.code == 2) {
        out->grid = ch.vp.grid;
        out->threads = ch.vp.threads;
        out->stages = ch.vp.stages;
        out->lag = ch.vp.lag;
        out->smem_bytes = ch.vp.smem_bytes;
        out->chunk_elems = ch.vp.chunk_elems;
        out->chunks_per_sample = ch.vp.chunks_per_sample;
    } else if (ch.code == 7) {
        out->grid = (int32_t)(ch.pf.ctas_per_sample * s.N);
        out->threads = 256;
        out->smem_bytes = (int32_t)ch.pf.smem;
        out->chunk_elems = (int64_t)ch.pf.ppc * s.HW;
        out->chunks_per_sample = ch.pf.ctas_per_sample;
    } else if (ch.code == 4) {
        out->grid = (int32_t)((ch.pg.qps + 256 * PLANE_QPT - 1) / (256 * PLANE_QPT) * s.N);
        out->threads = 256;
        out->chunk_elems = 4 * PLANE_QPT * 256;
    } else if (ch.code == 1) {
        out->grid = ch.fp.grid;
        out->threads = ch.fp.threads;
        out->stages = ch.fp.stages;
        out->lag = ch.fp.lag;
        out->smem_bytes = ch.fp.smem_bytes;
        out->chunk_elems = ch.fp.chunk_elems;
        out->chunks_per_sample = ch.fp.chunks_per_sample;
    } else {
        out->grid = (int32_t)((s.tiles + 255) / 256);
        out->threads = 256;
    }
    out->decompress_fast = decompress_fast_ok(s) ? ((s.H == 1 && s.CHW < (1u << 31)) ? 3 : 1) : (decompress_flat_ok(s) ? 2 : 0);
    return DIV_OK;
}

div_status div_compress_ex(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                           void* workspace_dev, size_t workspace_bytes, uint64_t seed, void* cuda_stream,
                           uint32_t flags) {
    if (!desc || !x_dev || !comp_dev || !workspace_dev) return DIV_ERR_NULL;
    div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    if (flags & ~DIV_FLAG_ALL) return DIV_ERR_PARAM;
    if (!aligned16(x_dev) || !aligned16(comp_dev) || !aligned16(workspace_dev)) return DIV_ERR_ALIGN;
    const Shape s = make_shape(desc);
    div_layout lo;
    make_layout(desc, s, &lo);
    if (comp_capacity < lo.total_bytes || workspace_bytes < lo.workspace_bytes) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(workspace_dev, 0, lo.workspace_bytes, stream) != cudaSuccess) return DIV_ERR_CUDA;
    uint8_t* blob = (uint8_t*)comp_dev;
    uint32_t* ws = (uint32_t*)workspace_dev;
    // kernels that store bytes or half-words leave the unused top of a partial last word alone: it is zero by contract
    if ((s.total * (uint64_t)desc->qbits) % 32u != 0 &&
        cudaMemsetAsync(blob + lo.packed_off + lo.packed_bytes - 4, 0, 4, stream) != cudaSuccess)
        return DIV_ERR_CUDA;
    // The single-launch kernels need all their CTAs resident, so they are launched cooperatively; where the
    // device refuses such a launch (fewer SMs visible to the process than the device reports, for instance) the
    // next kernel in line takes the descriptor: nothing has been enqueued by the refused launch.
    for (uint32_t f = flags;;) {
        Choice ch;
        choose_compress(desc, s, f, &ch);
        div_status r = DIV_OK;
        uint32_t drop = 0;
        switch (ch.code) {
            case 8: return compress_lines(desc, s, lo, ch.lg, x_dev, blob, ws, seed, stream, true);
            case 5: return compress_lines(desc, s, lo, ch.lg, x_dev, blob, ws, seed, stream, false);
            case 6: r = compress_staged(desc, s, lo, ch.sp, x_dev, blob, ws, seed, stream); drop = DIV_FLAG_NO_STAGED_KERNEL; break;
            case 3: r = compress_lagged(desc, s, lo, ch.lp, x_dev, blob, ws, seed, stream); drop = DIV_FLAG_NO_LAGGED_KERNEL; break;
            case 2: r = compress_fused_v(desc, s, lo, ch.vp, x_dev, blob, ws, seed, stream); drop = DIV_FLAG_NO_STRIP_KERNEL; break;
            case 7: return compress_planes(desc, s, lo, ch.pg, x_dev, blob, ws, seed, stream, true);
            case 4: return compress_planes(desc, s, lo, ch.pg, x_dev, blob, ws, seed, stream, false);
            case 1: r = compress_fused(desc, s, lo, ch.fp, x_dev, blob, ws, seed, stream); drop = DIV_FLAG_FORCE_TWO_PASS; break;
            default: return compress_two_pass(desc, s, lo, x_dev, blob, ws, seed, stream);
        }
        if (r != DIV_ERR_CUDA) return r;
        f |= drop;
    }
    return compress_two_pass(desc, s, lo, x_dev, blob, ws, seed, stream);
}

div_status div_debug_compress_starved(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                                      void* workspace_dev, size_t workspace_bytes, uint64_t seed, void* cuda_stream,
                                      uint32_t flags, uint64_t timeout_ns) {
    if (!desc || !x_dev || !comp_dev || !workspace_dev) return DIV_ERR_NULL;
    div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    if ((flags & ~DIV_FLAG_ALL) || timeout_ns == 0 || timeout_ns > 100000000ull) return DIV_ERR_PARAM;
    if (!aligned16(x_dev) || !aligned16(comp_dev) || !aligned16(workspace_dev)) return DIV_ERR_ALIGN;
    const Shape s = make_shape(desc);
    div_layout lo;
    make_layout(desc, s, &lo);
    if (comp_capacity < lo.total_bytes || workspace_bytes < lo.workspace_bytes) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(workspace_dev, 0, lo.workspace_bytes, stream) != cudaSuccess) return DIV_ERR_CUDA;
    uint8_t* blob = (uint8_t*)comp_dev;
    uint32_t* ws = (uint32_t*)workspace_dev;
    const uint32_t never = 0xFFFFFFFFu;      // an arrival count no sample reaches
    if (!(flags & DIV_FLAG_NO_STRIP_KERNEL)) {
        VPlan vp;
        if (plan_v(desc, s, &vp) == DIV_OK) return compress_fused_v(desc, s, lo, vp, x_dev, blob, ws, seed, stream, never, timeout_ns);
    }
    if (!(flags & DIV_FLAG_NO_LAGGED_KERNEL)) {
        LPlan lp;
        if (plan_lagged(desc, s, &lp) == DIV_OK) return compress_lagged(desc, s, lo, lp, x_dev, blob, ws, seed, stream, never, timeout_ns);
    }
    if (!(flags & DIV_FLAG_NO_STAGED_KERNEL)) {
        SPlan sp;
        if (plan_staged(desc, s, &sp) == DIV_OK) return compress_staged(desc, s, lo, sp, x_dev, blob, ws, seed, stream, never, timeout_ns);
    }
    if (!(flags & (DIV_FLAG_NO_PLANE_KERNELS | DIV_FLAG_TWO_LAUNCH_PLANES))) {
        PlaneGeom pg;
        if (plan_planes(desc, s, &pg)) return compress_planes(desc, s, lo, pg, x_dev, blob, ws, seed, stream, true, never, timeout_ns);
    }
    return DIV_ERR_PARAM;
}

div_status div_compress(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                        void* workspace_dev, size_t workspace_bytes, uint64_t seed, void* cuda_stream) {
    return div_compress_ex(desc, x_dev, comp_dev, comp_capacity, workspace_dev, workspace_bytes, seed, cuda_stream, 0u);
}

div_status div_decompress(const div_desc* desc, const void* comp_dev, size_t comp_bytes, void* xhat_dev,
                          void* cuda_stream) {
    if (!desc || !comp_dev || !xhat_dev) return DIV_ERR_NULL;
    div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    if (!aligned16(comp_dev) || !aligned16(xhat_dev)) return DIV_ERR_ALIGN;
    const Shape s = make_shape(desc);
    div_layout lo;
    make_layout(desc, s, &lo);
    if (comp_bytes < lo.total_bytes) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const uint8_t* blob = (const uint8_t*)comp_dev;
    const uint64_t nwords = lo.packed_bytes / 4;
    return dispatch_types(desc->x_dtype, desc->lfc_dtype, [&](auto* xt, auto* lt) -> div_status {
        typedef std::remove_pointer_t<decltype(xt)> XT;
        typedef std::remove_pointer_t<decltype(lt)> LT;
        return dispatch_q(desc->qbits, [&](auto q) -> div_status {
            constexpr int Q = decltype(q)::value;
            const LT* lfc = (const LT*)(blob + lo.lfc_off);
            const uint32_t* packed = (const uint32_t*)(blob + lo.packed_off);
            const float* stats = (const float*)(blob + lo.stats_off);
            if (decompress_fast_ok(s) && s.H == 1 && s.CHW < (1u << 31)) {
                DecLine d;
                d.qps = s.CHW / 4;
                d.C = s.C;
                d.Wb = s.Wb;
                d.qpr = s.W / 4;
                d.log2lpt = 0;
                while ((4u << d.log2lpt) < s.B) ++d.log2lpt;
                d.by_qpr = make_fastdiv(d.qpr);
                const uint32_t per_block = 256u * DEC_QPT;
                dim3 grid((d.qps + per_block - 1) / per_block, s.N);
                decompress_line_kernel<XT, LT, Q, DEC_QPT><<<grid, 256, 0, stream>>>(lfc, packed, stats, (XT*)xhat_dev, d);
            } else if (decompress_fast_ok(s)) {
                DecFast d;
                d.qps = s.CHW / 4;
                d.C = s.C;
                d.TPP = s.TPP;
                d.Wb = s.Wb;
                d.log2B = 0;
                while ((1u << d.log2B) < s.B) ++d.log2B;
                d.H = s.H;
                d.hwq = s.HW / 4;
                d.wq = s.W / 4;
                d.hq_count = (s.H + 3u) / 4u;
                d.ipp = d.hq_count * d.wq;
                d.items = s.C * d.ipp;
                d.by_ipp = make_fastdiv(d.ipp);
                d.by_wq = make_fastdiv(d.wq);
                dim3 grid((d.items + 255u) / 256u, s.N);
                // rows that are not whole 32-byte sectors: the 4 rows of an item spread over the plane (see the kernel)
                if ((s.W * (uint32_t)sizeof(XT)) % 32u != 0 && s.H >= 8u)
                    decompress_quad_kernel<XT, LT, Q, DEC_QPT, true><<<grid, 256, 0, stream>>>(lfc, packed, stats, (XT*)xhat_dev, d);
                else
                    decompress_quad_kernel<XT, LT, Q, DEC_QPT, false><<<grid, 256, 0, stream>>>(lfc, packed, stats, (XT*)xhat_dev, d);
            } else if (decompress_flat_ok(s)) {
                DecFlat d;
                d.qps = s.CHW / 4;
                d.C = s.C;
                d.TPP = s.TPP;
                d.Wb = s.Wb;
                d.HW = s.HW;
                d.W = s.W;
                d.B = s.B;
                d.by_hw = make_fastdiv(s.HW);
                d.by_w = make_fastdiv(s.W);
                d.by_b = make_fastdiv(s.B);
                const uint32_t per_block = 256u * FLAT_QPT;
                d.table_words = quad_table_words(s.HW);
                d.period = quad_period(s.HW);
                d.period_planes = quad_period_planes(s.HW);
                d.by_period = make_fastdiv(d.period);
                d.planes_per_cta = flat_planes_per_cta(4u * per_block, s.HW);
                dim3 grid((d.qps + per_block - 1) / per_block, s.N);
                decompress_flat_kernel<XT, LT, Q, FLAT_QPT><<<grid, 256, flat_smem_bytes(4u * per_block, s.HW, s.TPP), stream>>>(
                    lfc, packed, stats, (XT*)xhat_dev, d);
            } else {
                const uint64_t g = (nwords + 255) / 256;
                if (g > 0x7FFFFFFFull) return DIV_ERR_SHAPE;
                decompress_general_kernel<XT, LT, Q><<<(unsigned)g, 256, 0, stream>>>(lfc, packed, stats, (XT*)xhat_dev, s, nwords);
            }
            return launch_status();
        });
    });
}

// ------------------------------------------------------------------------------------------------
// div_compress_static: compress with the scratch in a fixed array inside the library
// ------------------------------------------------------------------------------------------------
}  // extern "C"

namespace {

// Scratch of div_compress_static: header + one 128-byte slot per sample, for up to
// DIV_STATIC_MAX_SAMPLES samples.  It lives in every GPU that loads the library until the process ends.
constexpr size_t STATIC_WS_BYTES =
    (4ull * (divk::WS_HEADER_WORDS + (size_t)divk::WS_SLOT_WORDS * DIV_STATIC_MAX_SAMPLES) + 255ull) / 256ull * 256ull;
static __device__ __align__(256) unsigned char g_static_workspace[STATIC_WS_BYTES];

// Device address of g_static_workspace on the current device.  In host code the array's name is only a
// handle for the runtime, not an address a kernel could use, so the address is asked for (a host-side
// query, no allocation); asking on every call keeps the library free of cached pointers that a device reset
// would leave dangling.
div_status static_workspace_ptr(void** out) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || !ptr) {
        cudaGetLastError();
        return DIV_ERR_CUDA;
    }
    *out = ptr;
    return DIV_OK;
}

}  // namespace

extern "C" {

div_status div_compress_static(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                               uint64_t seed, void* cuda_stream) {
    if (!desc) return DIV_ERR_NULL;
    const div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    if (desc->n > DIV_STATIC_MAX_SAMPLES) return DIV_ERR_CAPACITY;      // the fixed scratch has no slot for more samples
    void* ws = nullptr;
    const div_status got = static_workspace_ptr(&ws);
    if (got != DIV_OK) return got;
    // same path as div_compress from here on (it clears the part of the scratch it uses on the stream)
    return div_compress_ex(desc, x_dev, comp_dev, comp_capacity, ws, STATIC_WS_BYTES, seed, cuda_stream, 0u);
}

div_status div_read_static_status(void* cuda_stream, int32_t* out_status) {
    if (!out_status) return DIV_ERR_NULL;
    void* ws = nullptr;
    const div_status got = static_workspace_ptr(&ws);
    if (got != DIV_OK) return got;
    return div_read_device_status(ws, cuda_stream, out_status);
}

// ------------------------------------------------------------------------------------------------
// per-plane quantisation groups
// ------------------------------------------------------------------------------------------------
div_status div_planegroup_bytes(const div_desc* desc, div_layout* out) {
    if (!desc || !out) return DIV_ERR_NULL;
    const div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    const Shape s = make_shape(desc);
    if (!pg_shape_ok(s)) return DIV_ERR_SHAPE;
    make_layout_pg(desc, s, out);
    return DIV_OK;
}

div_status div_planegroup_plan_query(const div_desc* desc, uint32_t flags, div_plan* out) {
    if (!desc || !out) return DIV_ERR_NULL;
    const div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    if (flags & ~DIV_FLAG_FORCE_TWO_PASS) return DIV_ERR_PARAM;
    const Shape s = make_shape(desc);
    if (!pg_shape_ok(s)) return DIV_ERR_SHAPE;
    *out = div_plan();
    PgPlan pl;
    if (!(flags & DIV_FLAG_FORCE_TWO_PASS) && plan_pg_strip(desc, s, &pl)) {
        out->fused = 1;
        out->grid = pl.grid;
        out->threads = (int32_t)pl.threads;
        out->chunk_elems = (int64_t)pl.G * s.HW;
        out->chunks_per_sample = (s.C + pl.G - 1) / pl.G;
    } else if (PgSmall g; !(flags & DIV_FLAG_FORCE_TWO_PASS) && plan_pg_small(desc, s, &g)) {
        out->fused = 2;
        out->grid = (int32_t)((g.planes + g.G - 1) / g.G);
        out->threads = 256;
        out->smem_bytes = (int32_t)pg_small_smem_bytes(g);
        out->chunk_elems = (int64_t)g.G * s.HW;
        out->chunks_per_sample = (s.C + g.G - 1) / g.G;
    } else {
        out->fused = 0;
        out->grid = (int32_t)(s.N * s.C);
        out->threads = 256;
        out->chunk_elems = s.HW;
        out->chunks_per_sample = s.C;
    }
    out->decompress_fast = decompress_fast_ok(s) ? 1 : (pg_decompress_flat_ok(s) ? 2 : 0);
    return DIV_OK;
}

div_status div_planegroup_compress(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                                   uint64_t seed, void* cuda_stream, uint32_t flags) {
    if (!desc || !x_dev || !comp_dev) return DIV_ERR_NULL;
    div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    if (flags & ~DIV_FLAG_FORCE_TWO_PASS) return DIV_ERR_PARAM;
    if (!aligned16(x_dev) || !aligned16(comp_dev)) return DIV_ERR_ALIGN;
    const Shape s = make_shape(desc);
    if (!pg_shape_ok(s)) return DIV_ERR_SHAPE;
    div_layout lo;
    make_layout_pg(desc, s, &lo);
    if (comp_capacity < lo.total_bytes) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    uint8_t* blob = (uint8_t*)comp_dev;
    // kernels that store bytes or half-words leave the unused top of a partial last word alone: it is zero by contract
    if ((s.total * (uint64_t)desc->qbits) % 32u != 0 &&
        cudaMemsetAsync(blob + lo.packed_off + lo.packed_bytes - 4, 0, 4, stream) != cudaSuccess)
        return DIV_ERR_CUDA;
    PgPlan pl;
    if (!(flags & DIV_FLAG_FORCE_TWO_PASS) && plan_pg_strip(desc, s, &pl))
        return compress_pg_strip(desc, s, lo, pl, x_dev, blob, seed, stream);
    if (PgSmall g; !(flags & DIV_FLAG_FORCE_TWO_PASS) && plan_pg_small(desc, s, &g))
        return compress_pg_small(desc, s, lo, g, x_dev, blob, seed, stream);
    // general kernel: words shared by two planes (and the zero-padded last word) are merged with atomic ORs
    // into a cleared buffer
    if (((uint64_t)s.HW * (uint64_t)desc->qbits) % 32u != 0 &&
        cudaMemsetAsync(blob + lo.packed_off, 0, lo.packed_bytes, stream) != cudaSuccess)
        return DIV_ERR_CUDA;
    return dispatch_types(desc->x_dtype, desc->lfc_dtype, [&](auto* xt, auto* lt) -> div_status {
        typedef std::remove_pointer_t<decltype(xt)> XT;
        typedef std::remove_pointer_t<decltype(lt)> LT;
        return dispatch_q(desc->qbits, [&](auto q) -> div_status {
            pg_general_kernel<XT, LT, decltype(q)::value><<<s.N * s.C, 256, 0, stream>>>(
                (const XT*)x_dev, (LT*)(blob + lo.lfc_off), (uint32_t*)(blob + lo.packed_off),
                (uint32_t*)(blob + lo.stats_off), s, seed);
            return launch_status();
        });
    });
}

div_status div_planegroup_decompress(const div_desc* desc, const void* comp_dev, size_t comp_bytes, void* xhat_dev,
                                     void* cuda_stream) {
    if (!desc || !comp_dev || !xhat_dev) return DIV_ERR_NULL;
    div_status st = check_desc(desc);
    if (st != DIV_OK) return st;
    if (!aligned16(comp_dev) || !aligned16(xhat_dev)) return DIV_ERR_ALIGN;
    const Shape s = make_shape(desc);
    if (!pg_shape_ok(s)) return DIV_ERR_SHAPE;
    div_layout lo;
    make_layout_pg(desc, s, &lo);
    if (comp_bytes < lo.total_bytes) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const uint8_t* blob = (const uint8_t*)comp_dev;
    const uint64_t nwords = lo.packed_bytes / 4;
    return dispatch_types(desc->x_dtype, desc->lfc_dtype, [&](auto* xt, auto* lt) -> div_status {
        typedef std::remove_pointer_t<decltype(xt)> XT;
        typedef std::remove_pointer_t<decltype(lt)> LT;
        return dispatch_q(desc->qbits, [&](auto q) -> div_status {
            constexpr int Q = decltype(q)::value;
            const LT* lfc = (const LT*)(blob + lo.lfc_off);
            const uint32_t* packed = (const uint32_t*)(blob + lo.packed_off);
            const uint32_t* stats = (const uint32_t*)(blob + lo.stats_off);
            if (decompress_fast_ok(s)) {
                DecFast d;
                d.qps = s.CHW / 4;
                d.C = s.C;
                d.TPP = s.TPP;
                d.Wb = s.Wb;
                d.log2B = 0;
                while ((1u << d.log2B) < s.B) ++d.log2B;
                d.H = s.H;
                d.hwq = s.HW / 4;
                d.wq = s.W / 4;
                d.hq_count = (s.H + 3u) / 4u;
                d.ipp = d.hq_count * d.wq;
                d.items = s.C * d.ipp;
                d.by_ipp = make_fastdiv(d.ipp);
                d.by_wq = make_fastdiv(d.wq);
                dim3 grid((d.items + 255u) / 256u, s.N);
                if ((s.W * (uint32_t)sizeof(XT)) % 32u != 0 && s.H >= 8u)
                    pg_decompress_quad_kernel<XT, LT, Q, DEC_QPT, true><<<grid, 256, 0, stream>>>(lfc, packed, stats, (XT*)xhat_dev, d);
                else
                    pg_decompress_quad_kernel<XT, LT, Q, DEC_QPT, false><<<grid, 256, 0, stream>>>(lfc, packed, stats, (XT*)xhat_dev, d);
            } else if (pg_decompress_flat_ok(s)) {
                PgDecFlat d;
                d.quads = s.total / 4;
                d.HW = s.HW;
                d.W = s.W;
                d.Wb = s.Wb;
                d.TPP = s.TPP;
                d.table_words = flat_table_words(s.HW);
                d.quads_same_plane = (s.HW % 4u == 0) ? 1u : 0u;
                d.by_hw = make_fastdiv(s.HW);
                d.by_w = make_fastdiv(s.W);
                d.by_b = make_fastdiv(s.B);
                const uint64_t g = (d.quads + 256u * DEC_QPT - 1) / (256u * DEC_QPT);
                pg_decompress_flat_kernel<XT, LT, Q, DEC_QPT><<<(unsigned)g, 256, 4u * d.table_words, stream>>>(
                    lfc, packed, stats, (XT*)xhat_dev, d);
            } else {
                const uint64_t g = (nwords + 255) / 256;
                if (g > 0x7FFFFFFFull) return DIV_ERR_SHAPE;
                pg_decompress_general_kernel<XT, LT, Q><<<(unsigned)g, 256, 0, stream>>>(lfc, packed, stats, (XT*)xhat_dev, s, nwords);
            }
            return launch_status();
        });
    });
}

// ------------------------------------------------------------------------------------------------
// 3-D activation maps
// ------------------------------------------------------------------------------------------------
}  // extern "C"

namespace {

div_status check_desc3(const div_desc3d* d) {
    if (!d) return DIV_ERR_NULL;
    if (d->n < 1 || d->c < 1 || d->d < 1 || d->h < 1 || d->w < 1) return DIV_ERR_SHAPE;
    if (d->n >= (1ll << 31) || d->c >= (1ll << 32) || d->d >= (1ll << 32) || d->h >= (1ll << 32) || d->w >= (1ll << 32))
        return DIV_ERR_SHAPE;
    const unsigned __int128 per = (unsigned __int128)d->c * (unsigned __int128)d->d * (unsigned __int128)d->h * (unsigned __int128)d->w;
    if (per >= ((unsigned __int128)1 << 32)) return DIV_ERR_SHAPE;
    if (d->block < 1) return DIV_ERR_PARAM;
    if (!(d->qbits == 1 || d->qbits == 2 || d->qbits == 4 || d->qbits == 8)) return DIV_ERR_PARAM;
    if (!(d->x_dtype == DIV_F32 || d->x_dtype == DIV_BF16)) return DIV_ERR_PARAM;
    if (!(d->lfc_dtype == DIV_F32 || d->lfc_dtype == DIV_BF16)) return DIV_ERR_PARAM;
    return DIV_OK;
}

Shape3 make_shape3(const div_desc3d* d) {
    Shape3 s;
    s.N = (uint32_t)d->n;
    s.C = (uint32_t)d->c;
    s.D = (uint32_t)d->d;
    s.H = (uint32_t)d->h;
    s.W = (uint32_t)d->w;
    uint32_t big = s.D > s.H ? s.D : s.H;
    if (s.W > big) big = s.W;
    s.B = (uint32_t)d->block > big ? big : (uint32_t)d->block;     // a block larger than every side is the largest side
    s.Db = (s.D + s.B - 1) / s.B;
    s.Hb = (s.H + s.B - 1) / s.B;
    s.Wb = (s.W + s.B - 1) / s.B;
    s.P2 = 1;
    while (s.P2 < s.B) s.P2 <<= 1;
    s.HW = s.H * s.W;
    s.DHW = s.D * s.HW;
    s.CDHW = s.C * s.DHW;
    s.TPV = s.Db * s.Hb * s.Wb;
    s.total = (uint64_t)s.N * s.CDHW;
    s.tiles = (uint64_t)s.N * s.C * s.TPV;
    return s;
}

// quad kernels of the 3-D form: 4 consecutive elements share a block
bool quad3_ok(const Shape3& s) { return s.W % 4 == 0 && s.B % 4 == 0 && s.CDHW < (1u << 31) && s.N <= 65535; }
Quad3 make_quad3(const Shape3& s) {
    Quad3 g;
    g.qps = s.CDHW / 4;
    g.C = s.C;
    g.Db = s.Db;
    g.Hb = s.Hb;
    g.Wb = s.Wb;
    g.B = s.B;
    g.qpr = s.W / 4;
    g.qpp = s.H * g.qpr;
    g.qpv = s.D * g.qpp;
    g.by_qpv = make_fastdiv(g.qpv);
    g.by_qpp = make_fastdiv(g.qpp);
    g.by_qpr = make_fastdiv(g.qpr);
    g.by_b = make_fastdiv(s.B);
    return g;
}

void make_layout3(const div_desc3d* d, const Shape3& s, div_layout* out) {
    out->lfc_off = 0;
    out->lfc_bytes = s.tiles * dtype_bytes(d->lfc_dtype);
    out->packed_off = align_up(out->lfc_bytes, SECTION_ALIGN);
    out->packed_bytes = ((s.total * (uint64_t)d->qbits + 31) / 32) * 4;
    out->stats_off = align_up(out->packed_off + out->packed_bytes, SECTION_ALIGN);
    out->stats_bytes = 8ull * s.N;
    out->total_bytes = out->stats_off + out->stats_bytes;
    out->closed_form_bytes = out->lfc_bytes + out->packed_bytes + out->stats_bytes;
    out->raw_bytes = s.total * dtype_bytes(d->x_dtype);
    out->workspace_bytes = align_up(4ull * (WS_HEADER_WORDS + (uint64_t)WS_SLOT_WORDS * s.N), 256);
}

}  // namespace

extern "C" {

div_status div_compressed_bytes_3d(const div_desc3d* desc, div_layout* out) {
    if (!desc || !out) return DIV_ERR_NULL;
    const div_status st = check_desc3(desc);
    if (st != DIV_OK) return st;
    make_layout3(desc, make_shape3(desc), out);
    return DIV_OK;
}

div_status div_compress_3d(const div_desc3d* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                           void* workspace_dev, size_t workspace_bytes, uint64_t seed, void* cuda_stream) {
    if (!desc || !x_dev || !comp_dev || !workspace_dev) return DIV_ERR_NULL;
    div_status st = check_desc3(desc);
    if (st != DIV_OK) return st;
    if (!aligned16(x_dev) || !aligned16(comp_dev) || !aligned16(workspace_dev)) return DIV_ERR_ALIGN;
    const Shape3 s = make_shape3(desc);
    div_layout lo;
    make_layout3(desc, s, &lo);
    if (comp_capacity < lo.total_bytes || workspace_bytes < lo.workspace_bytes) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(workspace_dev, 0, lo.workspace_bytes, stream) != cudaSuccess) return DIV_ERR_CUDA;
    uint8_t* blob = (uint8_t*)comp_dev;
    uint32_t* ws = (uint32_t*)workspace_dev;
    // kernels that store bytes or half-words leave the unused top of a partial last word alone: it is zero by contract
    if ((s.total * (uint64_t)desc->qbits) % 32u != 0 &&
        cudaMemsetAsync(blob + lo.packed_off + lo.packed_bytes - 4, 0, 4, stream) != cudaSuccess)
        return DIV_ERR_CUDA;
    const uint64_t nwords = lo.packed_bytes / 4;
    const uint64_t g1 = (s.tiles + 127) / 128, g2 = (nwords + 255) / 256;
    if (g1 > 0x7FFFFFFFull || g2 > 0x7FFFFFFFull) return DIV_ERR_SHAPE;
    return dispatch_types(desc->x_dtype, desc->lfc_dtype, [&](auto* xt, auto* lt) -> div_status {
        typedef std::remove_pointer_t<decltype(xt)> XT;
        typedef std::remove_pointer_t<decltype(lt)> LT;
        // blocks whose padded side fits a warp: a lane per block column (coalesced); else a thread per block
        const uint32_t bpw = s.P2 <= 32u ? 32u / s.P2 : 0u;
        const uint32_t gpr = bpw ? (s.Wb + bpw - 1u) / bpw : 0u;                       // warp groups per row of blocks
        const uint64_t groups = (uint64_t)s.N * s.C * s.Db * s.Hb * gpr;
        const uint64_t gw = (groups + 7u) / 8u;
        // W % 4 == 0 and B = 4 or 8: a lane per strip of 4 columns (16-byte loads)
        const uint64_t strip_slots = (uint64_t)s.N * s.C * s.Db * s.Hb * s.Wb * (s.B / 4u) * 2u;      // two lanes per strip
        const uint64_t gs = (strip_slots + 127u) / 128u;
        if (s.W % 4u == 0 && (s.B == 4u || s.B == 8u) && s.P2 == s.B && gs <= 0x7FFFFFFFull) {
            const XT* xs = (const XT*)x_dev;
            LT* lf = (LT*)(blob + lo.lfc_off);
            if (s.B == 8u) lfc_stats3d_strip_kernel<XT, LT, 8><<<(unsigned)gs, 128, 0, stream>>>(xs, lf, ws, s, strip_slots);
            else lfc_stats3d_strip_kernel<XT, LT, 4><<<(unsigned)gs, 128, 0, stream>>>(xs, lf, ws, s, strip_slots);
        } else if (bpw && gw <= 0x7FFFFFFFull) {
            const XT* xs = (const XT*)x_dev;
            LT* lf = (LT*)(blob + lo.lfc_off);
            switch (s.P2) {
                case 1: lfc_stats3d_warp_kernel<XT, LT, 1><<<(unsigned)gw, 256, 0, stream>>>(xs, lf, ws, s, gpr, groups); break;
                case 2: lfc_stats3d_warp_kernel<XT, LT, 2><<<(unsigned)gw, 256, 0, stream>>>(xs, lf, ws, s, gpr, groups); break;
                case 4: lfc_stats3d_warp_kernel<XT, LT, 4><<<(unsigned)gw, 256, 0, stream>>>(xs, lf, ws, s, gpr, groups); break;
                case 8: lfc_stats3d_warp_kernel<XT, LT, 8><<<(unsigned)gw, 256, 0, stream>>>(xs, lf, ws, s, gpr, groups); break;
                case 16: lfc_stats3d_warp_kernel<XT, LT, 16><<<(unsigned)gw, 256, 0, stream>>>(xs, lf, ws, s, gpr, groups); break;
                default: lfc_stats3d_warp_kernel<XT, LT, 32><<<(unsigned)gw, 256, 0, stream>>>(xs, lf, ws, s, gpr, groups); break;
            }
        } else {
            lfc_stats3d_kernel<XT, LT><<<(unsigned)g1, 128, 0, stream>>>((const XT*)x_dev, (LT*)(blob + lo.lfc_off), ws, s);
        }
        if (launch_status() != DIV_OK) return DIV_ERR_CUDA;
        if (s.W % 4u == 0 && (s.B == 4u || s.B == 8u) && s.P2 == s.B && gs <= 0x7FFFFFFFull && desc->qbits != 1) {
            void* packed = blob + lo.packed_off;
            float* stats = (float*)(blob + lo.stats_off);
            const XT* xs = (const XT*)x_dev;
            const LT* lf = (const LT*)(blob + lo.lfc_off);
#define DIVK_Q3(QQ, PP) quant3d_strip_kernel<XT, LT, QQ, PP><<<(unsigned)gs, 128, 0, stream>>>(xs, lf, ws, packed, stats, s, seed, strip_slots)
            if (s.B == 8u) {
                if (desc->qbits == 2) DIVK_Q3(2, 8); else if (desc->qbits == 4) DIVK_Q3(4, 8); else DIVK_Q3(8, 8);
            } else {
                if (desc->qbits == 2) DIVK_Q3(2, 4); else if (desc->qbits == 4) DIVK_Q3(4, 4); else DIVK_Q3(8, 4);
            }
#undef DIVK_Q3
            return launch_status();
        }
        if (quad3_ok(s) && desc->qbits != 1) {
            const Quad3 g = make_quad3(s);
            const dim3 grid((g.qps + 256u * DEC_QPT - 1) / (256u * DEC_QPT), s.N);
            void* packed = blob + lo.packed_off;
            float* stats = (float*)(blob + lo.stats_off);
            const XT* xs = (const XT*)x_dev;
            const LT* lf = (const LT*)(blob + lo.lfc_off);
            switch (desc->qbits) {
                case 2: quant3d_quad_kernel<XT, LT, 2, DEC_QPT><<<grid, 256, 0, stream>>>(xs, lf, ws, packed, stats, g, seed); break;
                case 4: quant3d_quad_kernel<XT, LT, 4, DEC_QPT><<<grid, 256, 0, stream>>>(xs, lf, ws, packed, stats, g, seed); break;
                default: quant3d_quad_kernel<XT, LT, 8, DEC_QPT><<<grid, 256, 0, stream>>>(xs, lf, ws, packed, stats, g, seed); break;
            }
            return launch_status();
        }
        return dispatch_q(desc->qbits, [&](auto q) -> div_status {
            quant_pack3d_kernel<XT, LT, decltype(q)::value><<<(unsigned)g2, 256, 0, stream>>>(
                (const XT*)x_dev, (const LT*)(blob + lo.lfc_off), ws, (uint32_t*)(blob + lo.packed_off),
                (float*)(blob + lo.stats_off), s, seed, nwords);
            return launch_status();
        });
    });
}

div_status div_decompress_3d(const div_desc3d* desc, const void* comp_dev, size_t comp_bytes, void* xhat_dev,
                             void* cuda_stream) {
    if (!desc || !comp_dev || !xhat_dev) return DIV_ERR_NULL;
    div_status st = check_desc3(desc);
    if (st != DIV_OK) return st;
    if (!aligned16(comp_dev) || !aligned16(xhat_dev)) return DIV_ERR_ALIGN;
    const Shape3 s = make_shape3(desc);
    div_layout lo;
    make_layout3(desc, s, &lo);
    if (comp_bytes < lo.total_bytes) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const uint8_t* blob = (const uint8_t*)comp_dev;
    const uint64_t nwords = lo.packed_bytes / 4;
    const uint64_t g = (nwords + 255) / 256;
    if (g > 0x7FFFFFFFull) return DIV_ERR_SHAPE;
    return dispatch_types(desc->x_dtype, desc->lfc_dtype, [&](auto* xt, auto* lt) -> div_status {
        typedef std::remove_pointer_t<decltype(xt)> XT;
        typedef std::remove_pointer_t<decltype(lt)> LT;
        // W % 4 == 0, B = 4 or 8, Q in {2,4,8}: a lane per half strip
        const uint64_t sps = (uint64_t)s.C * s.Db * s.Hb * s.Wb * (s.B / 4u) * 2u;
        if (s.W % 4u == 0 && (s.B == 4u || s.B == 8u) && s.P2 == s.B && desc->qbits != 1 && sps < (1ull << 31) && s.N <= 65535u) {
            const dim3 grid((unsigned)((sps + 255u) / 256u), s.N);
            const LT* lf = (const LT*)(blob + lo.lfc_off);
            const uint32_t* pk = (const uint32_t*)(blob + lo.packed_off);
            const float* stt = (const float*)(blob + lo.stats_off);
#define DIVK_D3(QQ, PP) decompress3d_strip_kernel<XT, LT, QQ, PP><<<grid, 256, 0, stream>>>(lf, pk, stt, (XT*)xhat_dev, s, (uint32_t)sps)
            if (s.B == 8u) {
                if (desc->qbits == 2) DIVK_D3(2, 8); else if (desc->qbits == 4) DIVK_D3(4, 8); else DIVK_D3(8, 8);
            } else {
                if (desc->qbits == 2) DIVK_D3(2, 4); else if (desc->qbits == 4) DIVK_D3(4, 4); else DIVK_D3(8, 4);
            }
#undef DIVK_D3
            return launch_status();
        }
        if (quad3_ok(s)) {
            const Quad3 g3 = make_quad3(s);
            const dim3 grid((g3.qps + 256u * DEC_QPT - 1) / (256u * DEC_QPT), s.N);
            return dispatch_q(desc->qbits, [&](auto q) -> div_status {
                decompress3d_quad_kernel<XT, LT, decltype(q)::value, DEC_QPT><<<grid, 256, 0, stream>>>(
                    (const LT*)(blob + lo.lfc_off), (const uint32_t*)(blob + lo.packed_off), (const float*)(blob + lo.stats_off),
                    (XT*)xhat_dev, g3);
                return launch_status();
            });
        }
        return dispatch_q(desc->qbits, [&](auto q) -> div_status {
            decompress3d_kernel<XT, LT, decltype(q)::value><<<(unsigned)g, 256, 0, stream>>>(
                (const LT*)(blob + lo.lfc_off), (const uint32_t*)(blob + lo.packed_off), (const float*)(blob + lo.stats_off),
                (XT*)xhat_dev, s, nwords);
            return launch_status();
        });
    });
}

// ------------------------------------------------------------------------------------------------
// ReLU / dropout operators with a packed 1-bit mask
// ------------------------------------------------------------------------------------------------
}  // extern "C"

namespace {
constexpr uint64_t MASK_MAX_TOTAL = 1ull << 40;
inline uint64_t mask_bytes_of(uint64_t total) { return (total + 31) / 32 * 4; }

div_status mask_forward(const void* x_dev, void* y_dev, void* mask_dev, size_t mask_capacity, uint64_t total,
                        int32_t dtype, bool dropout, uint64_t seed, uint32_t drop_threshold, void* cuda_stream) {
    if (!x_dev || !y_dev || !mask_dev) return DIV_ERR_NULL;
    if (total < 1 || total > MASK_MAX_TOTAL) return DIV_ERR_SHAPE;
    if (!(dtype == DIV_F32 || dtype == DIV_BF16) || drop_threshold > 65536u) return DIV_ERR_PARAM;
    if (!aligned16(x_dev) || !aligned16(y_dev) || !aligned16(mask_dev)) return DIV_ERR_ALIGN;
    if (mask_capacity < mask_bytes_of(total)) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    uint8_t* mask = (uint8_t*)mask_dev;
    // the kernels store one byte per 8 elements: the rest of a partial last word is zero by contract
    if (total % 32u != 0 && cudaMemsetAsync(mask + mask_bytes_of(total) - 4, 0, 4, stream) != cudaSuccess) return DIV_ERR_CUDA;
    const unsigned grid = (unsigned)((total + 2047) / 2048);
    const uint64_t base = rng_sample_base(seed, 0u);
    if (dtype == DIV_F32) {
        if (dropout) mask_forward_kernel<float, true><<<grid, 256, 0, stream>>>((const float*)x_dev, (float*)y_dev, mask, total, base, drop_threshold);
        else mask_forward_kernel<float, false><<<grid, 256, 0, stream>>>((const float*)x_dev, (float*)y_dev, mask, total, base, 0u);
    } else {
        if (dropout) mask_forward_kernel<bf16, true><<<grid, 256, 0, stream>>>((const bf16*)x_dev, (bf16*)y_dev, mask, total, base, drop_threshold);
        else mask_forward_kernel<bf16, false><<<grid, 256, 0, stream>>>((const bf16*)x_dev, (bf16*)y_dev, mask, total, base, 0u);
    }
    return launch_status();
}
}  // namespace

extern "C" {

div_status div_mask_bytes(uint64_t total, uint64_t* out_bytes) {
    if (!out_bytes) return DIV_ERR_NULL;
    if (total < 1 || total > MASK_MAX_TOTAL) return DIV_ERR_SHAPE;
    *out_bytes = mask_bytes_of(total);
    return DIV_OK;
}

div_status div_relu_forward(const void* x_dev, void* y_dev, void* mask_dev, size_t mask_capacity, uint64_t total,
                            int32_t dtype, void* cuda_stream) {
    return mask_forward(x_dev, y_dev, mask_dev, mask_capacity, total, dtype, false, 0, 0, cuda_stream);
}

div_status div_dropout_forward(const void* x_dev, void* y_dev, void* mask_dev, size_t mask_capacity, uint64_t total,
                               int32_t dtype, uint64_t seed, uint32_t drop_threshold, void* cuda_stream) {
    return mask_forward(x_dev, y_dev, mask_dev, mask_capacity, total, dtype, true, seed, drop_threshold, cuda_stream);
}

div_status div_mask_backward(const void* mask_dev, size_t mask_bytes, const void* grad_out_dev, void* grad_in_dev,
                             uint64_t total, int32_t dtype, void* cuda_stream) {
    if (!mask_dev || !grad_out_dev || !grad_in_dev) return DIV_ERR_NULL;
    if (total < 1 || total > MASK_MAX_TOTAL) return DIV_ERR_SHAPE;
    if (!(dtype == DIV_F32 || dtype == DIV_BF16)) return DIV_ERR_PARAM;
    if (!aligned16(mask_dev) || !aligned16(grad_out_dev) || !aligned16(grad_in_dev)) return DIV_ERR_ALIGN;
    if (mask_bytes < mask_bytes_of(total)) return DIV_ERR_CAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const unsigned grid = (unsigned)((total + 2047) / 2048);
    if (dtype == DIV_F32)
        mask_backward_kernel<float><<<grid, 256, 0, stream>>>((const uint8_t*)mask_dev, (const float*)grad_out_dev, (float*)grad_in_dev, total);
    else
        mask_backward_kernel<bf16><<<grid, 256, 0, stream>>>((const uint8_t*)mask_dev, (const bf16*)grad_out_dev, (bf16*)grad_in_dev, total);
    return launch_status();
}

div_status div_read_device_status(const void* workspace_dev, void* cuda_stream, int32_t* out_status) {
    if (!workspace_dev || !out_status) return DIV_ERR_NULL;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    int32_t v = 0;
    if (cudaMemcpyAsync(&v, workspace_dev, sizeof(v), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return DIV_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return DIV_ERR_CUDA;
    *out_status = v;
    return DIV_OK;
}

}  // extern "C"
