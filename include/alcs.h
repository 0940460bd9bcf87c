/*
 * alcs.h -- C ABI of the SIMD-structured sparse convolution for NVIDIA B200: pointwise (1x1)
 * layers first, the general k x k case (alcs_spconv2d) further down.
 *
 *   Y[n, cout, h*w] = W_sparse[cout, cin] x X[n, cin, h*w] + bias   (optionally ReLU)
 *
 * W is pruned in blocks of g consecutive output channels that share one input-channel index
 * (paper, Section 3.2.1 "SIMD-structured pruning": the parameters at the same location of g
 * adjacent filters form one group and are kept or removed together; different groups of filters
 * may have different zero locations).  Block row r = output channels r*g .. r*g+g-1.
 *
 * General conventions
 *   - Every function returns an int status: ALCS_OK (0) or a negative alcs_status.  Nothing
 *     throws, aborts or prints.  alcs_strerror() names a status; alcs_last_cuda_error() gives
 *     the CUDA runtime's text for the calling thread's last ALCS_ERR_CUDA.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA global memory of the
 *     device the packed weights were uploaded to.  The caller owns every buffer it passes in;
 *     the library owns alcs_packed and alcs_stack objects until the matching free/destroy.
 *   - cuda_stream arguments are cudaStream_t values passed as void* (NULL = the default stream).
 *     Device work is enqueued asynchronously; no call synchronises unless stated.
 *   - Index type is int32.  Supported group sizes for packing: 1..64; for the GPU kernels:
 *     1, 2, 4, 8, 16 (others: ALCS_ERR_UNSUPPORTED).
 *   - There is no CPU implementation of the convolution in this library.  On a machine without a
 *     usable CUDA device every device entry point fails with ALCS_ERR_CUDA.
 */
#ifndef ALCS_H_
#define ALCS_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ALCS_API __attribute__((visibility("default")))
#else
#define ALCS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define ALCS_VERSION 2

typedef enum {
    ALCS_OK = 0,
    ALCS_ERR_INVALID_ARG = -1,  /* null pointer, negative size, misaligned or aliased buffer        */
    ALCS_ERR_SHAPE = -2,        /* sizes that do not fit together or overflow int32 indexing        */
    ALCS_ERR_UNSUPPORTED = -3,  /* valid request the kernels do not implement (g, dtype, ...)       */
    ALCS_ERR_ALLOC = -4,        /* host or device allocation failed                                 */
    ALCS_ERR_CUDA = -5,         /* a CUDA runtime call failed; see alcs_last_cuda_error()           */
    ALCS_ERR_CORRUPT = -6,      /* a serialized blob failed validation                              */
    ALCS_ERR_STATE = -7,        /* object not in the required state (e.g. weights not uploaded)     */
    ALCS_ERR_TOO_LARGE = -8     /* problem needs more than the fixed scratch of alcs_spconv1x1_noalloc */
} alcs_status;

typedef enum {
    ALCS_F32 = 0,               /* fp32 weights, activations and outputs, fp32 accumulation         */
    ALCS_F16 = 1,               /* IEEE binary16 weights and activations, fp32 accumulation         */
    ALCS_BF16 = 2               /* bfloat16 weights and activations, fp32 accumulation; by the paper's rule
                                   (Section 3.2.1: group size = register bits / element bits) a 16-bit type
                                   doubles the group size of fp32, as binary16 does.  CUDA-core kernels only. */
} alcs_dtype;

/* Bits of the `flags` argument of the convolution entry points. */
#define ALCS_RELU 1u            /* y = max(acc + bias, 0)                                           */
#define ALCS_Y_F32 2u           /* 16-bit weights only: write Y (and read a residual) as fp32 instead of the 16-bit type */

typedef struct alcs_packed alcs_packed;   /* opaque packed weight matrix, library-owned */
typedef struct alcs_stack alcs_stack;     /* opaque layer stack, library-owned          */

ALCS_API const char* alcs_strerror(int status);
ALCS_API const char* alcs_last_cuda_error(void);
ALCS_API int alcs_version(void);

/* ---------------------------------------------------------------------------------------------
 * Packing (host only).
 *
 * Storage format: paper, Section 3.2.2, paragraph "Storage format of SIMD-structured sparse
 * tensor" -- a grouped CSR that keeps, for each group of g filters, the number of non-zero
 * columns, one column offset per non-zero column (the number of columns before it in the
 * flattened kernel matrix, i.e. its absolute 0-based index) and the non-zero values, g per
 * column.  Here the three parts of all R = ceil(cout/g) groups are concatenated:
 *     row_ptr[R+1]   row_ptr[r+1]-row_ptr[r] = number of kept columns of group r
 *     col_idx[nb]    ascending inside a group
 *     vals[nb*g]     value j of kept block k at vals[k*g + j], j = channel inside the group
 * The mask decides what is kept, not the values: a kept block is stored even if all-zero and a
 * dropped block is dropped even if non-zero.  Values are copied bit for bit.  If cout is not a
 * multiple of g the last group is padded with +0 rows.
 * ------------------------------------------------------------------------------------------- */

/*
 * alcs_pack: w is row-major [cout][cin] of dtype dt (host); block_mask is [ceil(cout/g)][cin]
 * bytes (host), non-zero = keep.  On success *out receives a new packed matrix (free it with
 * alcs_packed_free).  Errors: INVALID_ARG (null, g outside 1..64), SHAPE (cout/cin <= 0 or
 * too many blocks for int32), ALLOC.
 */
ALCS_API int alcs_pack(const void* w, const uint8_t* block_mask, int cout, int cin, int g, alcs_dtype dt,
              alcs_packed** out);

/*
 * alcs_unpack: inverse of alcs_pack.  w_out [cout][cin] of the packed dtype receives the kept
 * values and +0 for dropped blocks; mask_out [ceil(cout/g)][cin] receives 0/1.  Either may be
 * NULL.  Host pointers.
 */
ALCS_API int alcs_unpack(const alcs_packed* p, void* w_out, uint8_t* mask_out);

/*
 * alcs_packed_view: borrow the packed arrays (host memory owned by p, valid until p is freed).
 * Any output pointer may be NULL.  *nb receives the number of kept blocks.
 */
ALCS_API int alcs_packed_view(const alcs_packed* p, int* cout, int* cin, int* g, alcs_dtype* dt, int* nb,
                     const int32_t** row_ptr, const int32_t** col_idx, const void** vals);

/*
 * Serialisation to a flat, position-independent little-endian byte blob
 * (header | row_ptr | col_idx | vals).  Call alcs_packed_serialize with buf == NULL to get the
 * size in *nbytes; with a buffer, *nbytes is its capacity on entry and the bytes written on
 * return.  alcs_packed_deserialize validates everything (magic, version, sizes, monotone row_ptr,
 * ascending in-range columns) and returns ALCS_ERR_CORRUPT otherwise.  Host pointers.
 */
ALCS_API int alcs_packed_serialize(const alcs_packed* p, void* buf, size_t* nbytes);
ALCS_API int alcs_packed_deserialize(const void* buf, size_t nbytes, alcs_packed** out);

/*
 * alcs_packed_upload: bind the packed matrix to CUDA device `device`.  The launch schedule (the
 * packed blocks re-ordered for one launch configuration) is built and copied to the device the
 * first time a convolution, alcs_spconv1x1_tune or alcs_stack_create needs it for a new shape; that
 * first call allocates device memory owned by p and waits for the copy, later calls do neither.
 * Uploading twice is an ALCS_ERR_STATE.  This is the "done in advance" re-organisation of the
 * paper's storage-format paragraph: it is not part of the timed path.
 */
ALCS_API int alcs_packed_upload(alcs_packed* p, int device, void* cuda_stream);

/*
 * alcs_packed_status: read the device error word of p (synchronises with the device).  *code is 0
 * unless a kernel gave up one of its bounded waits: 1 = a consumer warp waited too long for data,
 * 2 = the producer warp waited too long for a free pipeline stage.  A non-zero code means the
 * outputs of that launch are incomplete.
 */
ALCS_API int alcs_packed_status(const alcs_packed* p, int* code);

/* Free host and device memory of p (NULL is allowed). */
ALCS_API void alcs_packed_free(alcs_packed* p);

/* ---------------------------------------------------------------------------------------------
 * The convolution (device).
 *
 * Operation: paper, Section 3.2.2, the convolution formula
 *     O(n,h,w) = sum_c sum_r sum_s W(n,c,r,s) I(c,h+r,w+s)
 * at k_h = k_w = 1, stride 1, evaluated as in the paragraph "Efficient multiplication
 * computation": for every group, loop over its kept columns, multiply the column's g weights
 * with the input values addressed by the column offset and accumulate.  Bias and ReLU are a
 * fused epilogue.
 * ------------------------------------------------------------------------------------------- */

/*
 * Launch configuration override, for tuning and tests.  Zero in a field means "choose".
 *   pixels_per_lane   4 or 8: each warp covers 32*pixels_per_lane consecutive pixels
 *   rows_per_warp     block rows whose accumulators one warp holds at a time
 *   warps             consumer warps per thread block (one more warp only moves data)
 *   chunk_channels    input channels staged in shared memory per pipeline stage
 *   stages            pipeline depth (2..8)
 *   row_groups        how many work items share one pixel tile, each taking a subset of rows
 *   min_blocks        thread blocks per SM the kernel is compiled for (1 or 2)
 *   copy_mode         how X tiles reach shared memory: 1 = per-lane cp.async, 2 = bulk (TMA) copies
 *                     of whole pixel runs (needs 16-byte aligned rows; otherwise 1 is used).  Image rows
 *                     that are not a multiple of 16 bytes long are first repacked into a scratch tensor
 *                     with padded rows; 3 = per-lane cp.async of 8 bytes straight from X, without that
 *                     pass, for rows that are a multiple of 8 but not of 16 bytes long (16-bit elements,
 *                     14x14 images), stride 1 and X on an 8-byte boundary; elsewhere 3 acts like 1;
 *                     4 = X is first copied (one more kernel, into the same scratch) into a tile-major
 *                     layout [pixel tile][channel][tile pixels], so that the channel rows of a chunk lie one
 *                     after the other and a work item stages them with a few large bulk (TMA) copies: the
 *                     staging then costs the kernel next to no instructions, at the price of one more pass
 *                     over X where its rows would not have needed repacking.  Batches of more than 8 images
 *   producer_warps    warps of the thread block that only move data (1..4)
 *   math_mode         1 = fp32 FMA on the CUDA cores; 2 = tensor cores (fp16 weights and activations
 *                     only): 16 kept blocks of a block row times the 16 input rows they select is a
 *                     dense 16 x g by 16 x pixels contraction, run as warp-level MMA with fp32
 *                     accumulation; 3 = the small-problem kernel (fp32 only, meant for batch 1): no
 *                     staging of X, a thread block is one (block row, image, pixel tile) and its `warps`
 *                     (1..16) warps share the row's kept columns, reading the canonical storage format and
 *                     the input vectors straight from global memory; partial sums are added in a fixed
 *                     order.  Only pixels_per_lane (2, 4, 8; g * pixels_per_lane <= 32) and warps apply;
 *                     the device copy of the storage format is made on its first use with a packed matrix
 *   consumer_groups   1 = all consumer warps work on one work item at a time; 2 = two halves of the
 *                     consumer warps take the thread block's work items alternately (tensor-core
 *                     kernels only), so that one half multiplies while the other half stores
 *   split_rows        1 = the kernel flavour for skewed matrices: a block row far longer than the others of
 *                     its work item is split into parts that separate warps multiply, and the parts' partial
 *                     sums are added in a fixed order through shared memory before the row is stored (fp32
 *                     CUDA-core kernels, a subset of the shapes); 2 = rows are never split; 0 = choose
 */
typedef struct {
    int pixels_per_lane, rows_per_warp, warps, chunk_channels, stages, row_groups, min_blocks, copy_mode,
        producer_warps, math_mode, consumer_groups, split_rows;
} alcs_launch_cfg;

/*
 * alcs_schedule_selfcheck (host only, no CUDA): build the launch schedule of p for a CUDA-core kernel
 * with `warps` consumer warps of `slots` accumulator sets each (chunk_channels and row_groups as in
 * alcs_launch_cfg; row_groups is raised to what warps*slots block rows per work item require), walk
 * every (warp, set)'s segments chunk by chunk exactly as a consumer warp of the kernel does, and
 * compare what that walk multiplies with the canonical storage format (paper, Section 3.2.2): every
 * kept block exactly once, bit for bit, no other column touched, every block row bound to exactly
 * one (warp, set), or -- a row much longer than the others of its work item -- split into parts that
 * take one (warp, set) each, every kept block in exactly one part, one part storing the row and
 * reading each of the others' hand-over slots exactly once.  stats (may be NULL, else 8 entries)
 * receives {row groups; largest and smallest number of block slots (kept blocks plus padding) any of
 * the SM's four schedulers is given in a work item; pair records in total; kept blocks; largest and
 * smallest number of units a scheduler is given in a work item; secondary parts of split rows in
 * total}.  Returns ALCS_ERR_CORRUPT if the walk and the storage format disagree.
 */
ALCS_API int alcs_schedule_selfcheck(const alcs_packed* p, int chunk_channels, int row_groups, int warps, int slots,
                                     int64_t* stats);

/*
 * Introspection of the compiled kernel variants (host only): alcs_variant_count() entries, each a
 * (dtype, g, pixels_per_lane, rows_per_warp, warps, min_blocks, producer_warps) combination that
 * alcs_spconv1x1_cfg accepts; the other fields of *cfg are set to 0.
 */
ALCS_API int alcs_variant_count(void);
ALCS_API int alcs_variant_get(int index, alcs_dtype* dt, int* g, alcs_launch_cfg* cfg);

/*
 * alcs_spconv1x1: x device [n][cin][h*wd], y device [n][cout][h*wd], both contiguous NCHW of the
 * packed dtype (y fp32 if ALCS_Y_F32); bias device fp32 [cout] or NULL; flags = ALCS_RELU |
 * ALCS_Y_F32.  x and y must not overlap and must be aligned to their element size.  16-byte
 * aligned buffers with h*wd a multiple of 4 (fp32) or 8 (fp16) are used in place.  If the rows of
 * x are not a multiple of 16 bytes long (h*wd = 49, ...) x is first repacked, by a small kernel on
 * the same stream, into scratch memory owned by w (allocated or grown by the first call that
 * needs it; n*cin*round_up(h*wd)*element bytes) and y is stored element by element; results are
 * identical.  Because that scratch belongs to w, two such convolutions with the SAME w must not
 * run concurrently on different streams.  Enqueues one kernel on cuda_stream;
 * no allocation and no synchronisation once this shape has been seen (see alcs_packed_upload).  n == 0 or h*wd == 0 is a successful no-op.
 * Errors: INVALID_ARG, SHAPE (n*channels*pixels beyond int32 tiles), UNSUPPORTED (g), STATE (not
 * uploaded / wrong current device), CUDA.
 */
ALCS_API int alcs_spconv1x1(const alcs_packed* w, const void* x, void* y, int n, int h, int wd,
                   const float* bias, unsigned flags, void* cuda_stream);

/*
 * alcs_spconv1x1_ex: the pointwise convolution with a stride and a residual operand (paper, Section
 * 3.2.2, the convolution formula at k_h = k_w = 1 sampled every `stride` pixels -- the 1x1 projection
 * shortcuts of the ResNets evaluated in Section 4.1 -- and, for the last 1x1 convolution of a
 * bottleneck, the shortcut added before the activation):
 *     y[n][co][oh][ow] = act( sum_c W(co,c) * x[n][c][oh*stride][ow*stride] + bias[co] + residual[n][co][oh][ow] ),
 * oh < ceil(h/stride), ow < ceil(wd/stride).  x device [n][cin][h][wd]; y and residual device
 * [n][cout][oh*ow] of the same element type (the packed dtype, or fp32 with ALCS_Y_F32); residual may be
 * NULL; it must not overlap y.  stride = 1 with residual = NULL is alcs_spconv1x1_cfg.  With stride > 1
 * the pixels that are read are first gathered, by a small kernel on the same stream, into the scratch
 * memory owned by w (see alcs_spconv1x1); the residual is read straight from the caller's buffer in the
 * epilogue, added in fp32 before ReLU and before the single rounding of an fp16 output.  cfg may be
 * NULL.  Errors as alcs_spconv1x1, plus INVALID_ARG for stride < 1.
 */
ALCS_API int alcs_spconv1x1_ex(const alcs_packed* w, const void* x, void* y, int n, int h, int wd, int stride,
                               const float* bias, const void* residual, unsigned flags,
                               const alcs_launch_cfg* cfg, void* cuda_stream);

/* Same, with an explicit launch configuration (cfg == NULL behaves like alcs_spconv1x1). */
ALCS_API int alcs_spconv1x1_cfg(const alcs_packed* w, const void* x, void* y, int n, int h, int wd,
                       const float* bias, unsigned flags, const alcs_launch_cfg* cfg,
                       void* cuda_stream);

/*
 * alcs_spconv1x1_plan: report the launch configuration alcs_spconv1x1 would use for this shape
 * (host only, no device work).
 */
ALCS_API int alcs_spconv1x1_plan(const alcs_packed* w, int n, int h, int wd, unsigned flags,
                        alcs_launch_cfg* out);

/*
 * alcs_spconv1x1_tune: time the candidate launch configurations for this shape on the given
 * buffers (y is overwritten with the correct result each time), remember the fastest in w for
 * later alcs_spconv1x1 calls with the same (n, h, wd, flags), and write it to *best (may be
 * NULL).  Every launch is timed with cold caches (a buffer larger than L2 is rewritten before it):
 * each candidate three times, then the twelve best fifteen times more in turn, and the lowest median
 * wins.  Synchronises the stream; meant for set-up time, never for the timed path.
 */
ALCS_API int alcs_spconv1x1_tune(alcs_packed* w, const void* x, void* y, int n, int h, int wd,
                        const float* bias, unsigned flags, void* cuda_stream,
                        alcs_launch_cfg* best);

/*
 * alcs_spconv1x1_set_cfg: make later alcs_spconv1x1 / alcs_stack_create calls with this
 * (n, h, wd, flags) use the given configuration, e.g. one that alcs_spconv1x1_tune found in an
 * earlier process.  Fields left 0 are chosen by the library.  Host only; returns UNSUPPORTED if no
 * compiled kernel variant fits it.
 */
ALCS_API int alcs_spconv1x1_set_cfg(alcs_packed* w, int n, int h, int wd, unsigned flags,
                                    const alcs_launch_cfg* cfg);

/*
 * alcs_spconv1x1_host: the same operation on HOST buffers x_host / y_host / bias_host, staged
 * through a caller-provided device workspace of at least alcs_spconv1x1_host_workspace() bytes
 * (256-byte aligned).  Enqueues H2D copies, the kernel and the D2H copy on cuda_stream and
 * returns without synchronising; use pinned host memory for truly asynchronous copies.
 */
ALCS_API size_t alcs_spconv1x1_host_workspace(const alcs_packed* w, int n, int h, int wd, unsigned flags);
ALCS_API int alcs_spconv1x1_host(const alcs_packed* w, const void* x_host, void* y_host, int n, int h,
                        int wd, const float* bias_host, unsigned flags, void* workspace,
                        size_t workspace_bytes, void* cuda_stream);

/*
 * alcs_spconv1x1_noalloc: the same convolution for callers that must not allocate device memory.
 * (The paper has no counterpart to this entry point; it exists for the way this library is used.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a latency-critical serving
 * loop, after the process has handed all free device memory to another allocator, or in a plugin
 * whose host forbids allocation calls after initialisation.  alcs_spconv1x1 may allocate: the first
 * call for a shape uploads the launch schedule, and inputs whose rows are not a multiple of 16
 * bytes long (h*wd = 49, ...) are repacked into scratch that w allocates or grows on demand.  This
 * entry point never calls cudaMalloc, cudaFree or any other allocating routine:
 *   - the launch schedule for (n, h, wd, flags) must already be on the device, i.e. alcs_spconv1x1,
 *     alcs_spconv1x1_tune or alcs_stack_create has been called once for that shape during set-up;
 *     otherwise the call fails with ALCS_ERR_STATE and launches nothing;
 *   - the repacked copy of x goes into one fixed array of ALCS_NOALLOC_SCRATCH_BYTES bytes that is
 *     part of the library image (every GPU that loads the library holds it until the process exits).
 *     A problem that needs more, n*cin*round_up(h*wd to 16 bytes)*element size, is rejected with
 *     ALCS_ERR_TOO_LARGE; inputs with 16-byte-multiple rows need no scratch and have no size limit.
 * The address of that array is looked up per device at set-up time, by alcs_packed_upload (which
 * runs with that device current); loading the library's device code on a GPU -- which is when the
 * driver backs the array there -- therefore also happens during set-up, not inside the phase that
 * may not allocate.  Should that look-up have failed, the first alcs_spconv1x1_noalloc call on the
 * device repeats it; make that first call before any stream capture begins.  All calls share the one array and it keeps
 * what the previous call left there: every call rewrites the part it uses, padding included, but two
 * calls that overlap on the GPU (different streams) race on it -- keep them on one stream or order
 * them with events.  Arguments, results and error codes are otherwise those of alcs_spconv1x1.
 */
#define ALCS_NOALLOC_SCRATCH_BYTES (16u << 20)
ALCS_API int alcs_spconv1x1_noalloc(const alcs_packed* w, const void* x, void* y, int n, int h, int wd,
                                    const float* bias, unsigned flags, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Measurement probes (device).  The paper has no counterpart: they exist so that the roofline the
 * kernels are judged against is measured on the GPU at hand instead of taken from a data sheet, and
 * so that the ceiling of the hot loop of Section 3.2.2's "efficient multiplication computation" can be
 * re-measured by anyone.  Each call launches one thread block per SM on cuda_stream, times it with
 * CUDA events (best of three after a warm-up), allocates and frees a few hundred KB of device
 * memory, and synchronises the stream: set-up / benchmarking use only.
 *
 * alcs_probe_fma_peak: dependent-chain-free fp32 FMAs on register operands, 16 warps per SM;
 *   packed = 0 scalar fma.rn.f32, 1 the two-wide fma.rn.f32x2 the kernels use.
 * alcs_probe_lds: cycles of the SM's load/store pipe one warp-wide shared-memory load instruction
 *   costs when 16 warps do nothing else: bytes_per_lane 4, 8 or 16; uniform = 0 every lane its own
 *   (conflict-free) address, 1 all lanes the same address.
 * alcs_probe_segment_loop: the pointwise kernel's segment loop, compiled as in the kernel, on
 *   synthetic segments of pairs_per_segment pair records that are resident in shared memory together
 *   with a 64-channel X tile (no staging, no barriers, no stores): `warps` warps per SM, each with
 *   rows_per_warp accumulator sets of g x pixels_per_lane; deep = 1 the flavour that keeps the next
 *   pair's X vectors in a second register set.  Only a fixed list of shapes is compiled
 *   (ALCS_ERR_UNSUPPORTED otherwise): g = 4 with (pixels, rows, warps, deep) in {(8,2,16,0), (8,2,16,1),
 *   (8,2,12,0), (8,2,12,1), (8,2,8,1), (8,1,16,0), (16,1,16,0), (16,1,12,1), (4,4,16,0)}, and
 *   (g, pixels, rows, warps, deep) in {(1,8,2,16,0), (8,4,2,16,0), (16,4,1,16,0)}.
 * frac_of_fp32_peak is relative to SMs x 128 lanes x 2 x the device's maximum SM clock.
 * Errors: INVALID_ARG, UNSUPPORTED, SHAPE, CUDA.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    double ms;                  /* duration of one launch                                          */
    double tflops;              /* fp32 FLOP/s reached, in units of 1e12                           */
    double frac_of_fp32_peak;   /* the same as a fraction of SMs x 128 x 2 x max SM clock          */
    int registers;              /* registers per thread of the probe kernel                        */
    int spill_bytes;            /* local-memory bytes per thread (0 = no spills)                   */
} alcs_probe_result;

ALCS_API int alcs_probe_fma_peak(int packed, alcs_probe_result* out, void* cuda_stream);
ALCS_API int alcs_probe_lds(int bytes_per_lane, int uniform, double* cycles_per_instruction, void* cuda_stream);
ALCS_API int alcs_probe_segment_loop(int g, int pixels_per_lane, int rows_per_warp, int warps, int deep,
                                     int pairs_per_segment, alcs_probe_result* out, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * General k_h x k_w convolution (device), fp32.
 *
 * Operation: paper, Section 3.2.2, the convolution formula with all three sums,
 *     O(co, oh, ow) = sum_c sum_r sum_s W(co, c, r, s) * I(c, oh*stride - pad + r, ow*stride - pad + s),
 * I read as zero outside the image (the paper writes the stride-1, unpadded case), evaluated as
 * W* x I* without materialising I*: W* stacks the flattened filters, so the packed matrix has
 * cin*kh*kw columns and column (c*kh + r)*kw + s holds tap (r, s) of input channel c.  The pruning
 * pattern is that of Section 3.2.1 for a general kernel: the parameters at one location (c, r, s)
 * of g adjacent filters are kept or removed together.  Pack the weights with
 *     alcs_pack(w [cout][cin*kh*kw], block_mask [ceil(cout/g)][cin*kh*kw], cout, cin*kh*kw, g, ALCS_F32, ...).
 *
 * alcs_spconv2d: x device [n][cin][h][wd], y device [n][cout][oh][ow] with
 * oh = (h + 2*pad - kh)/stride + 1 (ow likewise), contiguous NCHW fp32, 4-byte aligned, not
 * overlapping; bias device fp32 [cout] or NULL; flags = ALCS_RELU or 0.  Enqueues one kernel on
 * cuda_stream.  The first call for a new geometry builds that geometry's launch schedule, allocates
 * device memory owned by w for it and waits for its upload; later calls with the same geometry do
 * neither.  n == 0 is a successful no-op.
 * Errors: INVALID_ARG (null or misaligned or overlapping buffers, non-positive sizes, unknown
 * flags), SHAPE (cin*kh*kw is not the packed column count, kernel larger than the padded image,
 * more than 2^31-1 elements), UNSUPPORTED (fp16 weights, g outside {1,2,4,8,16}, stride > 2,
 * kernels wider than 8*stride+1, or so many input channels that not even a one-row strip of all of
 * them fits in shared memory), STATE, ALLOC, CUDA.
 *
 * alcs_spconv2d_plan reports the launch configuration alcs_spconv2d would use (host only).
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int positions_per_lane;     /* output positions per lane (2, 4 or 8)                           */
    int strip_rows;             /* output rows per work item                                        */
    int row_groups;             /* work items that share one strip, each taking a subset of rows    */
    int position_tiles;         /* tiles of 32*positions_per_lane positions per strip               */
    int warps_per_tile;         /* warps that share one position tile and split its block rows      */
    int smem_bytes;             /* dynamic shared memory per thread block                           */
    int chunk_channels;         /* input channels staged at a time (cin: all at once)               */
    int images_per_item;        /* whole images per work item (1, 2 or 4; > 1 only for small images) */
} alcs_conv2d_cfg;

ALCS_API int alcs_spconv2d(const alcs_packed* w, const void* x, void* y, int n, int cin, int h, int wd,
                           int kh, int kw, int stride, int pad, const float* bias, unsigned flags,
                           void* cuda_stream);
/* Same, with parts of the launch configuration fixed (tests, tuning): non-zero positions_per_lane,
 * strip_rows, chunk_channels, images_per_item and row_groups of *cfg are taken as given (row_groups only when all
 * channels are staged at once), the rest is chosen; UNSUPPORTED if nothing fits.  cfg == NULL
 * behaves like alcs_spconv2d. */
ALCS_API int alcs_spconv2d_cfg(const alcs_packed* w, const void* x, void* y, int n, int cin, int h, int wd,
                               int kh, int kw, int stride, int pad, const float* bias, unsigned flags,
                               const alcs_conv2d_cfg* cfg, void* cuda_stream);
ALCS_API int alcs_spconv2d_plan(const alcs_packed* w, int n, int cin, int h, int wd, int kh, int kw,
                                int stride, int pad, alcs_conv2d_cfg* out);

/* ---------------------------------------------------------------------------------------------
 * Latency model and projection with bisection.
 *
 * Latency model: paper, Section 3.3.  The run time of layer l is a function of its number of
 * non-zero parameters, T^(l)(W^(l)) = T^(||W^(l)||_0), approximated by linear interpolation over
 * measured pairs (k_i, t_i), 0 = k_1 < ... < k_n = N^(l) (the paper measures 11 of them, at
 * 0, 0.1 N, ..., N):  T^(s) = t_1 + sum_i delta_i alpha_i min(k_{i+1} - k_i, s - k_i) with
 * delta_i = [s >= k_i] and alpha_i = (t_{i+1} - t_i) / (k_{i+1} - k_i); the network's run time is
 * T(W) = tau + sum_l T^(l)(W^(l)).  Host only; all pointers are host memory.
 * Errors: INVALID_ARG (null pointers, fewer than 2 knots, knots not strictly ascending).
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int n_knots;                /* number of measured points, >= 2                               */
    const int64_t* k;           /* [n_knots] non-zero parameter counts, strictly ascending        */
    const double* t;            /* [n_knots] measured run time at each count (any unit)           */
} alcs_latency_table;

ALCS_API int alcs_layer_latency(const alcs_latency_table* tab, int64_t s, double* out);
ALCS_API int alcs_network_latency(double tau, const alcs_latency_table* tabs, int n_layers, const int64_t* s,
                                  double* out);

/*
 * alcs_project_bisection: paper, Section 3.4, Algorithm 1 ("Projection operation with bisection").
 * The variable to project is given layer by layer: u_tilde[l] is a DEVICE pointer to a row-major
 * fp32 matrix [cout[l]][cols[l]] (cols = cin*kh*kw, the flattened filters); the arrays u_tilde,
 * cout, cols, tabs themselves are host memory.  What is computed: the groups are the g adjacent
 * filters at one location (Section 3.2.1): group (r, c) of a layer = elements (r*g .. r*g+g-1, c).
 * All groups of all layers are ranked together by L2 norm, largest first -- the ranking key is the
 * squared norm accumulated in fp32 in ascending filter order with separately rounded multiplies and
 * adds, equal keys keep (layer, r, c) order.  The result keeps a prefix of that ranking; its length N
 * is searched by halving a bracket [n0, n1] (initially 0 and the number of groups): the model
 * latency of "the N best-ranked groups kept" uses ||W^(l)||_0 = g * (kept groups of layer l) in the
 * latency model above, the half whose end latency is below t_budget (strictly) is discarded from
 * below, the other from above, until the latencies of the two ends differ by at most eps or the
 * bracket has width 1 (a case the paper leaves open); N = (n0 + n1) / 2, rounded down.
 * Outputs: mask_out, DEVICE, one byte per group, the layers one after the other, each
 * [ceil(cout/g)][cols] -- the block_mask layout of alcs_pack; u_out (may be NULL), a host array of
 * DEVICE pointers, u_out[l] (may be NULL) receives u_tilde[l] with the dropped groups set to +0;
 * kept_per_layer (host, may be NULL) the number of kept groups per layer; *result (host, may be
 * NULL).  The call takes temporary device memory (about 18 bytes per group plus the sort's
 * workspace) from the device's stream-ordered memory pool and returns it there, copies 2 bytes per
 * group to the host for the search, and synchronises cuda_stream.
 * Errors: INVALID_ARG, SHAPE (2^31 or more groups), UNSUPPORTED (more than 4096 layers), ALLOC, CUDA.
 */
typedef struct {
    int64_t n_keep;             /* groups kept = (n0 + n1) / 2                                     */
    int64_t n0, n1;             /* final bracket                                                   */
    int64_t n_groups;           /* groups in total                                                 */
    int iters;                  /* bisection steps taken                                           */
    double latency;             /* model latency of the result                                     */
} alcs_projection_result;

ALCS_API int alcs_project_bisection(const float* const* u_tilde, const int* cout, const int* cols, int n_layers, int g,
                                    const alcs_latency_table* tabs, double tau, double t_budget, double eps,
                                    uint8_t* mask_out, float* const* u_out, int64_t* kept_per_layer,
                                    alcs_projection_result* result, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Layer stack: a network's pointwise layers run back to back on one stream (paper, Section 3.3,
 * T(W) = tau + sum_l T_l(W_l): the network's run time is the sum over its layers).
 * ------------------------------------------------------------------------------------------- */

typedef struct {
    const alcs_packed* w;       /* uploaded packed weights                     */
    const void* x;              /* device [n][cin][h*wd]                       */
    void* y;                    /* device [n][cout][h*wd]                      */
    int n, h, wd;
    const float* bias;          /* device fp32 [cout] or NULL                  */
    unsigned flags;             /* ALCS_RELU | ALCS_Y_F32                      */
    const void* residual;       /* device, shape and type of y, or NULL (see alcs_spconv1x1_ex) */
    int stride;                 /* 0 or 1: none; > 1: y is [n][cout][ceil(h/stride)*ceil(wd/stride)] */
} alcs_layer;

#define ALCS_STACK_GRAPH 1u     /* replay the launches as one CUDA graph       */

/*
 * alcs_stack_create copies the layer descriptions (the buffers stay the caller's and must outlive
 * the stack) and fixes each layer's launch configuration.  With ALCS_STACK_GRAPH the first
 * alcs_stack_run captures the launches into a CUDA graph on that stream and later runs replay it.
 * alcs_stack_run enqueues all layers in order on cuda_stream without synchronising.
 * Layers whose input rows are not a multiple of 16 bytes long are repacked into scratch memory that
 * the STACK owns (allocated by alcs_stack_create with the layers' device current, sized for its
 * largest such layer, released by alcs_stack_destroy): nothing a captured graph refers to is freed
 * or moved by later alcs_spconv1x1 calls with the same packed matrices, at any batch size.  Two runs
 * of the same stack must not overlap on the GPU (they share that scratch and the outputs).
 */
ALCS_API int alcs_stack_create(const alcs_layer* layers, int n_layers, unsigned stack_flags,
                      alcs_stack** out);
ALCS_API int alcs_stack_run(alcs_stack* s, void* cuda_stream);
ALCS_API int alcs_stack_destroy(alcs_stack* s);

/*
 * alcs_stack_tune: choose the layers' launch configurations IN CONTEXT.  alcs_spconv1x1_tune times a layer
 * alone, with cold caches and nothing before it on the stream; inside a stack a layer starts while its
 * predecessor drains (programmatic dependent launch), finds whatever the earlier layers left in L2, and, at
 * batch 1, costs little more than its launch, so the configuration that wins alone is not always the one
 * that wins there.  For every layer in turn this call tries the candidates (the best twelve of the last
 * alcs_spconv1x1_tune for the layer's shape if there was one, else the cost model's best eight; for batches
 * of at most 8 images also every shape of the small-problem kernel that applies), each time timing the WHOLE stack the way alcs_stack_run
 * runs it (a graph stack is captured again), and keeps a candidate only if the stack gets faster by more
 * than 0.4 %; `passes` sweeps over the layers (0 = 2), stopping early when a sweep changes nothing.  The
 * chosen configurations are also remembered in the packed matrices for later calls with the same shape.
 * us_before / us_after (may be NULL): microseconds per pass over the stack before and after.  The layers'
 * outputs are overwritten many times with the same correct values.  Synchronises the stream; set-up time
 * only.  alcs_stack_layer_cfg reports the configuration layer `layer` (0-based) of the stack uses now (all
 * zero for an empty layer).
 */
ALCS_API int alcs_stack_tune(alcs_stack* s, int passes, void* cuda_stream, double* us_before, double* us_after);
ALCS_API int alcs_stack_layer_cfg(const alcs_stack* s, int layer, alcs_launch_cfg* out);

#ifdef __cplusplus
}
#endif
#endif /* ALCS_H_ */
