/*
 * division.h -- C ABI of the B200 DIVISION activation compress / decompress library.
 *
 * The operation is the per-layer pair of DIVISION ("Memory Efficient Training via Dual
 * Activation Precision"), Sec. 4.1 "Activation Map Compression" and Sec. 4.2 "Activation Map
 * Decompression" (Algorithm 1, forward and backward loops):
 *
 *   compress    H^L = AveragePooling(H), window = stride = B                    (Sec. 4.1)
 *               H^H = H - UpSampling(H^L), nearest interpolation                (Sec. 4.1)
 *               V^H = stochastic_round((H^H - delta) / Delta), Q bits           (Eq. 9)
 *               delta = min H^H,  Delta = (max H^H - delta) / (2^Q - 1)
 *   decompress  H_hat = UpSampling(H^L) + Delta * V^H + delta                   (Sec. 4.2, Eq. 10)
 *
 * for an activation map H of shape N x C x H x W (the paper's Minibatch x Channel x N x N),
 * contiguous NCHW, fp32 or bf16.  A 1-D map (Minibatch x Channel x N; the appendix "Compression of 1D and 3D
 * Activation Maps": pooling and up-sampling along the last axis) is described as N x C x 1 x W: a block then
 * covers B consecutive elements of a row.  3-D maps have entry points of their own (div_compress_3d).
 *
 * Conventions fixed by this library where the paper is silent (the same rules are written out in
 * the CPU checker, which was implemented separately):
 *   - one (delta, Delta) pair per SAMPLE, kept in fp32;
 *   - H or W not divisible by B: ceil grid, partial tiles average their in-bounds elements
 *     (a side shorter than B gives a 1 x 1 map, as the paper's footnote in Sec. 4.1 requires);
 *   - the residual is taken against the stored (rounded) low-frequency value;
 *   - rounding up happens with probability frac(t), t = (H^H - delta) * (2^Q - 1)/(max - min);
 *     the uniform number of element e of sample n is a pure function of (seed, n, e)
 *     ("DIVRNG-v1": one 64-bit mix per 4 elements, 16-bit uniforms);
 *   - all arithmetic is IEEE fp32, one rounding per operation, no fused multiply-add, and the
 *     block sum uses a fixed order (pairwise tree down the rows, then across the columns), so
 *     the output is a pure function of (descriptor, input bits, seed): independent of grid
 *     size, SM count and timing;
 *   - codes of 32/Q consecutive elements (global NCHW flat order) share one little-endian 32-bit
 *     word, first element in the lowest bits.
 *
 * Compressed buffer ("blob"), one caller-owned device allocation:
 *     [ lfc : N*C*ceil(H/B)*ceil(W/B) values of lfc_dtype | pad to 128 B |
 *       packed : ceil(N*C*H*W*Q/32) uint32 words          | pad to 128 B |
 *       stats  : N pairs (delta, Delta) fp32 ]
 *
 * Ownership and behaviour common to all entry points:
 *   - every pointer named *_dev is DEVICE memory owned by the caller, 16-byte aligned;
 *     descriptors and layouts are HOST memory;
 *   - the library allocates nothing and keeps no state between calls (one exception, documented there:
 *     div_compress_static works in a fixed array inside the library);
 *   - div_compress / div_decompress only enqueue work on the given CUDA stream (a cudaStream_t
 *     passed as void*; NULL is the default stream) and return; errors that can be seen on the
 *     host are returned at once and nothing is launched;
 *   - inputs must be finite.  x is never modified; outputs may not alias inputs.
 */
#ifndef DIVISION_H_
#define DIVISION_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum div_status {
    DIV_OK = 0,
    DIV_ERR_NULL = 1,      /* a required pointer is NULL                                   */
    DIV_ERR_SHAPE = 2,     /* n, c, h or w < 1, or c*h*w >= 2^32, or n >= 2^31             */
    DIV_ERR_PARAM = 3,     /* block < 1, qbits not in {1,2,4,8}, unknown dtype or flag     */
    DIV_ERR_ALIGN = 4,     /* a device pointer is not 16-byte aligned                      */
    DIV_ERR_CAPACITY = 5,  /* blob or workspace smaller than div_compressed_bytes reports  */
    DIV_ERR_CUDA = 6,      /* the CUDA runtime reported an error (launch, attribute, ...)  */
    DIV_ERR_TIMEOUT = 7    /* device side: a bounded wait inside the fused kernel ran out  */
} div_status;

typedef enum div_dtype { DIV_F32 = 0, DIV_BF16 = 1 } div_dtype;

/* Problem statement: tensor shape, block size B, bit width Q, dtypes (Sec. 4.1). */
typedef struct div_desc {
    int64_t n, c, h, w;   /* all >= 1; c*h*w < 2^32; n < 2^31                            */
    int32_t block;        /* B >= 1 (the paper uses 8; also 4, 12, 16, 18, 64)           */
    int32_t qbits;        /* Q in {1, 2, 4, 8} (the paper uses 2, 4, 8)                  */
    int32_t x_dtype;      /* div_dtype of x and of x_hat                                 */
    int32_t lfc_dtype;    /* div_dtype the low-frequency map is stored in                */
} div_desc;

/* Byte layout of the blob and of the scratch workspace; all offsets from the blob start. */
typedef struct div_layout {
    uint64_t lfc_off, lfc_bytes;
    uint64_t packed_off, packed_bytes;
    uint64_t stats_off, stats_bytes;
    uint64_t total_bytes;        /* blob size to allocate (includes alignment padding)          */
    uint64_t closed_form_bytes;  /* lfc_bytes + packed_bytes + stats_bytes (what the ratio uses) */
    uint64_t raw_bytes;          /* n*c*h*w*sizeof(x_dtype)                                      */
    uint64_t workspace_bytes;    /* scratch div_compress needs (per-sample min/max/arrival slots) */
} div_layout;

/* How div_compress will run a descriptor (introspection for tests and benchmarks). */
typedef struct div_plan {
    int32_t fused;          /* for W%4==0, B in {4,8}, Q in {2,4,8}, one launch:
                               6: x read from HBM once and re-read from L2 a little later, both reads staged through
                                  shared-memory rings by bulk copies (staged kernel; first choice from 56 MB up
                                  with B = 8);
                               3: as 6, with plain global loads (lagged kernel; first choice from 20 MB up);
                               2: chunks wait in a shared-memory ring (strip ring kernel; first choice below 20 MB);
                               7: small planes of any width (tile side 4, 8 or 16 after padding, at most 32 lanes per
                                  plane row, Q in {2,4,8}) in one launch: a CTA owns a run of planes of one sample,
                                  joins the sample's other CTAs through an arrival count and quantises the same
                                  planes (second read from L1 / L2); taken when all its CTAs can be resident; also the
                                  first choice for maps of such planes with W%4==0 below 56 MiB (bfloat16: below
                                  32 MiB), as long as the flags exclude none of the kernels 2, 3, 6;
                               4: the same in two launches;
                               1: one launch, shared-memory ring, general kernel;  0: two-pass general kernels;
                               8: 1-D maps (h == 1; the appendix on 1D and 3D activation maps), W%4==0, B a power of two
                                  in [4,128], Q in {2,4,8}, in one launch: a CTA owns a run of rows of one sample, joins
                                  the sample's other CTAs through an arrival count and quantises the same rows (second
                                  read from L1 / L2); taken when all its CTAs can be resident;
                               5: the same in two launches */
    int32_t grid;           /* CTAs of the (first) compress kernel                            */
    int32_t threads;        /* threads per CTA                                                */
    int32_t stages;         /* shared-memory ring depth (ring kernels only)                   */
    int32_t lag;            /* chunks (ring kernels) or units (3) between the reduce and the quantise
                               half of the same data                                           */
    int32_t smem_bytes;     /* dynamic shared memory per CTA                                  */
    int64_t chunk_elems;    /* elements per full chunk (ring kernels) or per unit (3)         */
    int64_t chunks_per_sample;
    int32_t decompress_fast;/* 1: quad kernel (W%4==0, B a power of two >= 4); 3: the same conditions on a 1-D map
                               (h == 1): line kernel; 2: flat kernel with a tile table (sample size a multiple of 4,
                               planes up to 8192 elements); 0: general */
    int32_t reserved;
} div_plan;

/* flags of div_compress_ex */
#define DIV_FLAG_FORCE_TWO_PASS 1u   /* never take a fused kernel                          */
#define DIV_FLAG_NO_STRIP_KERNEL 2u  /* never take the strip variant of the ring kernel    */
#define DIV_FLAG_NO_LAGGED_KERNEL 4u /* never take the lagged (L2 re-read) kernel          */
#define DIV_FLAG_NO_PLANE_KERNELS 8u /* never take the small-plane pair of kernels          */
#define DIV_FLAG_NO_LINE_KERNELS 16u /* never take the pair of kernels for 1-D maps          */
#define DIV_FLAG_NO_STAGED_KERNEL 32u/* never take the staged (bulk-copy rings) kernel       */
#define DIV_FLAG_TWO_LAUNCH_PLANES 64u /* small planes and 1-D maps: the pair of kernels, not the fused one */

/*
 * Sizes of the cached tuple (H^L, V^H, Delta, delta) of Sec. 4.1 in the blob layout above:
 *   closed form = N*C*ceil(H/B)*ceil(W/B)*sizeof(lfc) + ceil(N*C*H*W*Q/32)*4 + 8*N.
 * Host only, pure integer arithmetic, never touches a device.
 * desc, out: host pointers.  Returns DIV_ERR_NULL / DIV_ERR_SHAPE / DIV_ERR_PARAM on bad input.
 */
div_status div_compressed_bytes(const div_desc* desc, div_layout* out);

/*
 * Compress one activation map (Sec. 4.1; Algorithm 1, forward loop).
 *   desc           host; the problem statement
 *   x_dev          device; N*C*H*W values of x_dtype, contiguous NCHW; read only
 *   comp_dev       device; receives the blob; at least layout.total_bytes
 *   comp_capacity  bytes available at comp_dev
 *   workspace_dev  device scratch of at least layout.workspace_bytes; contents on entry are
 *                  irrelevant (the call clears it on the stream); after the call its first word
 *                  holds a device-side status (see div_read_device_status)
 *   workspace_bytes bytes available at workspace_dev
 *   seed           seed of the stochastic rounding
 *   cuda_stream    cudaStream_t as void*
 * Two calls that overlap on the GPU must not share a workspace.
 */
div_status div_compress(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                        void* workspace_dev, size_t workspace_bytes, uint64_t seed, void* cuda_stream);

/* Same as div_compress with DIV_FLAG_* bits (0 = default behaviour). */
div_status div_compress_ex(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                           void* workspace_dev, size_t workspace_bytes, uint64_t seed, void* cuda_stream,
                           uint32_t flags);

/*
 * Compress without a caller-supplied workspace.  (The paper has no counterpart: this is a convenience of
 * this library.)
 *
 * Who needs it: code that may not allocate device memory at the point where it compresses.  Examples are
 * a host callback or a plug-in running inside somebody else's framework whose memory pool it must not
 * touch, a process whose device memory budget is fully handed out at start-up, or a latency-critical loop
 * in which a cudaMalloc (which synchronises the device) is not acceptable.  Such a caller still owns x and
 * the blob, but cannot produce the few kilobytes of scratch div_compress asks for.
 *
 * Here the scratch is a fixed array inside the library (128 bytes per sample, for at most
 * DIV_STATIC_MAX_SAMPLES samples, about 128 KB).  Every GPU that loads the library holds that array until
 * the process exits, whether or not this entry point is used.  The call allocates and frees nothing.
 *
 *   desc, x_dev, comp_dev, comp_capacity, seed, cuda_stream   exactly as for div_compress
 *
 * Returns what div_compress returns, and additionally
 *   DIV_ERR_CAPACITY  when desc->n > DIV_STATIC_MAX_SAMPLES (the fixed scratch is too small; use div_compress),
 *   DIV_ERR_CUDA      when the address of the array cannot be obtained on the current device.
 *
 * Things to know:
 *   - every call asks the CUDA runtime for the device address of the array (a host-side query with the
 *     current device; the first one on a device may make the runtime load the library's code onto it): make
 *     the first call on each device outside any stream capture;
 *   - all calls on one device share the one array.  Each call clears the part it uses before its kernel
 *     runs (on the given stream), so earlier contents do not matter, but two calls whose work overlaps on
 *     the GPU (different streams, or different host threads without ordering between their streams) race
 *     on it and produce wrong output.  Keep calls on a device ordered one after the other;
 *   - the output is byte-for-byte what div_compress writes for the same arguments;
 *   - the device-side status word (a bounded wait that ran out, see div_read_device_status) lives in the
 *     array: read it with div_read_static_status before the next call on that device overwrites it.
 */
#define DIV_STATIC_MAX_SAMPLES 1024
div_status div_compress_static(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                               uint64_t seed, void* cuda_stream);

/*
 * Device-side status of the last div_compress_static on the current device (no counterpart in the paper):
 * what div_read_device_status reports for a caller-owned workspace, read from the library's fixed array.
 * Synchronises the stream, copies one word back; allocates nothing.  *out_status is DIV_OK or
 * DIV_ERR_TIMEOUT (the blob of that call is then unspecified: compress again, e.g. with div_compress_ex and
 * DIV_FLAG_FORCE_TWO_PASS, whose kernels have no device-side waits).  Host-blocking.
 */
div_status div_read_static_status(void* cuda_stream, int32_t* out_status);

/*
 * Decompress (Sec. 4.2; Algorithm 1, backward loop): x_hat = UpSampling(H^L) + Delta*V^H + delta,
 * rounded to x_dtype.
 *   comp_dev    device; a blob written by div_compress with the SAME desc; read only
 *   comp_bytes  bytes valid at comp_dev (>= layout.total_bytes)
 *   xhat_dev    device; receives N*C*H*W values of x_dtype, contiguous NCHW
 */
div_status div_decompress(const div_desc* desc, const void* comp_dev, size_t comp_bytes,
                          void* xhat_dev, void* cuda_stream);

/*
 * Test hook for the bounded waits of the single-launch compress kernels (plan codes 2, 3, 6 and 7): runs the
 * kernel div_compress_ex would run, but tells it to wait for a number of arrivals per sample that is never
 * reached, with `timeout_ns` (at most 100 ms) as the limit of every wait.  The kernel must give up, record
 * DIV_ERR_TIMEOUT in the workspace status word (read it with div_read_device_status) and return; the blob's
 * contents are then unspecified.  The first of the strip ring, lagged, staged and fused small-plane
 * kernels that the flags allow and the descriptor fits is taken; DIV_ERR_PARAM when there is none.
 * Arguments as for div_compress_ex.  No counterpart in the paper.
 */
div_status div_debug_compress_starved(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                                      void* workspace_dev, size_t workspace_bytes, uint64_t seed, void* cuda_stream,
                                      uint32_t flags, uint64_t timeout_ns);

/*
 * Per-plane quantisation groups: the same pair of operations with one (delta, Delta) pair per
 * (sample, channel) plane, stored as two bfloat16 numbers.  This is the grouping behind the paper's count of
 * N^2*Q/8 + 4 bytes per channel for the high-frequency component (Sec. 4.1; proof of Theorem 3A), and
 * "Delta and delta are cached in bfloat16" (Sec. 4.1).  Differences from div_compress / div_decompress:
 *   - blob: same sections, but stats = N*C little-endian 32-bit words, low half delta_b, high half Delta_b
 *     (bfloat16 bit patterns); closed form = lfc + packed + 4*N*C bytes; layout.workspace_bytes = 0;
 *   - rounding of the pair, on which the paper is silent: delta_b = largest bfloat16 number <= min H^H,
 *     Delta_b = smallest bfloat16 number >= (max H^H - delta_b)/(2^Q - 1); both sides use the stored pair:
 *     t = (H^H - delta_b) * (1/Delta_b), H^H_hat = Delta_b * V^H + delta_b.  A plane whose Delta_b or
 *     1/Delta_b would be zero or not finite stores Delta_b = 0 and all codes 0;
 *   - a plane's extremes stay inside one CTA, so compress needs no scratch and no device-side waiting;
 *   - n*c < 2^31 (else DIV_ERR_SHAPE).
 * Everything else (pooling grid, residual against the stored value, stochastic rounding, random stream,
 * packing order, argument meaning, ownership, error codes) is as documented above.
 * flags: 0, or DIV_FLAG_FORCE_TWO_PASS to take the general kernel (one CTA per plane) even where the
 * register-resident strip kernel applies (W%4==0, B in {4,8}, Q in {2,4,8}, planes of at most 512 strips of
 * 4 columns x B rows).
 */
div_status div_planegroup_bytes(const div_desc* desc, div_layout* out);
div_status div_planegroup_compress(const div_desc* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                                   uint64_t seed, void* cuda_stream, uint32_t flags);
div_status div_planegroup_decompress(const div_desc* desc, const void* comp_dev, size_t comp_bytes,
                                     void* xhat_dev, void* cuda_stream);
/* plan.fused: 1 strip kernel, 2 small-plane kernel (tile row of at most 32 padded columns, B up to 16, Q in
   {2,4,8}, sample size a multiple of 4), 0 general kernel; plan.decompress_fast: 1 quad kernel, 2 flat kernel
   (total size a multiple of 4, planes up to 8192 elements), 0 general. */
div_status div_planegroup_plan_query(const div_desc* desc, uint32_t flags, div_plan* out);

/*
 * 3-D activation maps (the appendix "Compression of 1D and 3D Activation Maps": Minibatch x Channel x N x N x N;
 * average pooling and nearest up-sampling over B x B x B blocks, Eq. 9 and its inverse unchanged).  x is
 * contiguous N x C x D x H x W.  Conventions as for 2-D maps: ceil grid on every axis, partial blocks average their
 * in-bounds elements, a block larger than every side is the largest side; the block sum is the balanced pairwise
 * tree along the depth axis, then down the rows, then across the columns; in-sample index
 * e = ((c*D + d)*H + h)*W + w; one fp32 (delta, Delta) pair per sample; blob = [lfc: N*C*ceil(D/B)*ceil(H/B)*
 * ceil(W/B) values | packed | stats] with the same padding, workspace as for div_compress.  c*d*h*w < 2^32.
 * Any shape, block size and Q; faster kernels where the padded block side is at most 32 (block means) and where
 * W%4==0 and B%4==0 (quantise, decompress).
 * Arguments, ownership and error codes as for div_compressed_bytes / div_compress / div_decompress.
 */
typedef struct div_desc3d {
    int64_t n, c, d, h, w;
    int32_t block, qbits, x_dtype, lfc_dtype;
} div_desc3d;
div_status div_compressed_bytes_3d(const div_desc3d* desc, div_layout* out);
div_status div_compress_3d(const div_desc3d* desc, const void* x_dev, void* comp_dev, size_t comp_capacity,
                           void* workspace_dev, size_t workspace_bytes, uint64_t seed, void* cuda_stream);
div_status div_decompress_3d(const div_desc3d* desc, const void* comp_dev, size_t comp_bytes, void* xhat_dev,
                             void* cuda_stream);

/*
 * ReLU and dropout operators with a packed 1-bit mask (the paper's appendix algorithms "Relu operator" and
 * "Dropout operator"; one bit per element, N^2/8 bytes per plane, in the byte count of Theorem 3A's proof):
 *   forward   V = mask,  H_out = V (.) H_in,  V packed and cached          backward  grad_in = V (.) grad_out
 * on flat arrays of `total` elements of `dtype` (1 <= total <= 2^40; DIV_ERR_SHAPE otherwise).
 *   - ReLU: V = [H_in > 0] (the paper's sgn read as the indicator of positivity; zeros and NaN give 0);
 *   - dropout: V = 1 (keep) with probability 1 - drop_threshold/65536: element i is dropped iff the 16-bit number of
 *     the random stream described above for (seed, sample 0, flat index i) is < drop_threshold (0 <= drop_threshold
 *     <= 65536, else DIV_ERR_PARAM); as in the paper's algorithm, kept values are not rescaled;
 *   - "(.)" is a select: masked positions become +0.0;
 *   - mask: bit (i mod 32) of little-endian 32-bit word i/32, ceil(total/32) words (div_mask_bytes), unused high
 *     bits of the last word zero;
 *   - x_dev / y_dev / grad_*_dev: device, `total` elements, 16-byte aligned; y_dev may be x_dev and grad_in_dev may
 *     be grad_out_dev (in place); mask_dev: device, 16-byte aligned, at least div_mask_bytes bytes
 *     (DIV_ERR_CAPACITY otherwise).  The calls enqueue one kernel on the stream and return.
 */
div_status div_mask_bytes(uint64_t total, uint64_t* out_bytes);
div_status div_relu_forward(const void* x_dev, void* y_dev, void* mask_dev, size_t mask_capacity, uint64_t total,
                            int32_t dtype, void* cuda_stream);
div_status div_dropout_forward(const void* x_dev, void* y_dev, void* mask_dev, size_t mask_capacity, uint64_t total,
                               int32_t dtype, uint64_t seed, uint32_t drop_threshold, void* cuda_stream);
div_status div_mask_backward(const void* mask_dev, size_t mask_bytes, const void* grad_out_dev, void* grad_in_dev,
                             uint64_t total, int32_t dtype, void* cuda_stream);

/* Which kernels a descriptor maps to on the current device.  desc, out: host. */
div_status div_plan_query(const div_desc* desc, uint32_t flags, div_plan* out);

/*
 * Device-side status of the last div_compress that used this workspace: synchronises the stream,
 * copies one word back.  *out_status is DIV_OK or DIV_ERR_TIMEOUT.  Host-blocking.
 */
div_status div_read_device_status(const void* workspace_dev, void* cuda_stream, int32_t* out_status);

/* Static, NUL-terminated description of a status code. */
const char* div_status_string(div_status s);

#ifdef __cplusplus
}
#endif
#endif /* DIVISION_H_ */
