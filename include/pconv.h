/*
 * pconv.h -- C ABI of the B200 pattern-sparse 3x3 convolution library (PCONV forward pass).
 *
 * The operation is the paper's Eq. 1 (cross-correlation, no kernel flip) applied per layer,
 *
 *     y[n,o,i,j] = act( b[o] + sum_c sum_{u,v<3} xpad[n,c,i*s+u-1,j*s+v-1] * W[o,c,u,v] ),
 *
 * for weights that carry the two sparsities of the paper's "Sparse Convolution Pattern" section:
 * every surviving (filter o, input channel c) kernel has its non-zeros inside one 3x3 binary
 * pattern of a small set (pattern pruning: 4 of 9 taps, the "2.25x" of the pattern-count tables),
 * and whole kernels are removed (connectivity pruning).  The library skips every pruned kernel and
 * every tap outside the pattern; the result equals the dense convolution up to summation order.
 * Zero padding 1, stride 1 or 2, dilation 1, groups 1, optional bias and fused ReLU are fixed by
 * this build (the paper does not state them).
 *
 * General rules
 *  - Every call returns a pconv_status; nothing throws, aborts or prints.  Out-parameters are
 *    written only on PCONV_OK unless stated otherwise.
 *  - "host" pointers are ordinary CPU memory; "dev" pointers are CUDA device memory of the current
 *    device.  `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *  - Tensors are dense and contiguous: activations NCHW, weights OIHW ([C_out][C_in][3][3]).
 *  - Pattern masks are 9-bit integers: bit (3*u + v) set <=> tap (row u, column v) may be
 *    non-zero; bit 4 is the centre.
 *  - Storage type PCONV_F32: x, y and packed weights are fp32.  PCONV_F16: x, y and packed
 *    weights are IEEE fp16 (weights rounded to nearest even at pack time); bias and every
 *    accumulation stay fp32, and the output is rounded once at the store.
 */
#ifndef PCONV_H_
#define PCONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pconv_handle pconv_handle; /* one packed layer; opaque, library-owned */
typedef struct pconv_stack pconv_stack;   /* a chain of packed layers with its activations */

typedef enum {
  PCONV_OK = 0,
  PCONV_ERR_NULL = 1,              /* a required pointer is NULL */
  PCONV_ERR_SHAPE = 2,             /* non-positive or inconsistent sizes, bad stride */
  PCONV_ERR_PATTERN_SET = 3,       /* a mask without exactly 4 of 9 bits, duplicates, bad count */
  PCONV_ERR_KERNEL_NOT_IN_SET = 4, /* a kernel's non-zeros fit no pattern (or not 0/4 when strict) */
  PCONV_ERR_RANGE = 5,             /* NaN/Inf weight, or overflow when rounding to fp16 */
  PCONV_ERR_UNSUPPORTED = 6,       /* unknown storage type or flag */
  PCONV_ERR_ALIGN = 7,             /* a device pointer is not aligned as required */
  PCONV_ERR_ALLOC = 8,             /* host or device allocation failed */
  PCONV_ERR_CUDA = 9,              /* a CUDA runtime call or a kernel launch failed */
  PCONV_ERR_DEVICE_TIMEOUT = 10,   /* a kernel's bounded wait ran out (see pconv_device_status) */
  PCONV_ERR_WORKSPACE = 11         /* the shape needs more scratch than the entry point can offer */
} pconv_status;

enum { PCONV_F32 = 0, PCONV_F16 = 1 };

enum {
  PCONV_RELU = 1u,    /* forward: y = max(0, .) after the bias */
  PCONV_STRICT4 = 2u, /* pack: every kernel must have exactly 0 or 4 non-zeros */
  PCONV_POOL2X2 = 4u, /* forward: a 2x2 / stride-2 max-pool is applied to the activated output in
                         the same kernel (tiled kernels only); y then holds
                         [n][c_out][h_out/2][w_out/2] */
  /* Kernel selection (forward).  Default: the library picks per shape.  These bits exist so that
   * tests and benchmarks can pin one implementation; they never change the result beyond
   * summation order. */
  PCONV_REPRODUCIBLE = 8u, /* forward: the same call gives bit-identical outputs every time: the
                              warps that share a tile take their chunks in a fixed order and the
                              channel range is not split across thread blocks (a workspace, if
                              given, is left untouched).  Without it the grouping of the fp32 partial
                              sums -- not the result beyond rounding -- may vary from run to run. */
  PCONV_CHAIN = 0x10u,     /* stacks: consecutive layers whose launch plans are single waves of CTAs
                              (batch-1 inference) run as ONE persistent kernel: Tensor Memory,
                              barriers and the CTAs stay, a CTA fetches the next layer's weight
                              blocks while others finish, and layers are crossed on a grid-wide
                              count with a bounded wait.  Off by default: on this hardware a launch
                              with programmatic stream serialisation crosses a layer boundary
                              faster (19 us per 512-filter 14x14 layer against 24 us chained). */
  PCONV_KERNEL_SIMPLE = 0x100u, /* one thread per output, walks the per-filter kernel list */
  PCONV_KERNEL_TILED = 0x200u,  /* shared-memory halo tiles, packed FMAs, one straight-line body per
                                   pattern mask (any set of 4-of-9 masks); the default */
  PCONV_KERNEL_GENERIC_TAPS = 0x400u, /* tiled path that tests the 9 mask bits at run time; slower,
                                         kept as a cross-check of the per-mask bodies */
  PCONV_ROWS4 = 0x1000u, /* tiled kernel with one-byte codes (canonical pattern sets): pins the */
  PCONV_ROWS8 = 0x2000u, /* output rows a lane owns per sub-tile.  4: sixteen consumer warps, a
                            decoded kernel runs 16 packed FMAs; 8: eight consumer warps with twice
                            the Tensor Memory columns each, 32 packed FMAs per decoded kernel (less
                            decoding per multiply-add, for layers with many pixels).  Default: the
                            planner picks per shape.  PCONV_ROWS8 with another pattern set or with
                            PCONV_KERNEL_GENERIC_TAPS: PCONV_ERR_UNSUPPORTED. */
  PCONV_CLUSTER = 0x4000u, /* channel split of the tiled kernel (a workspace must be given, as for any
                              split): the thread blocks that share an output tile form a thread-block
                              cluster -- when they are at most 16 and the device can hold all the
                              launch's clusters at once, otherwise the bit changes nothing -- and add
                              their partial sums up through distributed shared memory in rank
                              order; no atomics, no tickets, the workspace stays untouched.  Off by
                              default: measured equal to the workspace form on single layers
                              (49 us on the 512-filter 28x28 layer either way) and 3 % slower on
                              the VGG stack at batch 1 (0.396 against 0.384 ms), where a cluster
                              must find its SMs free inside one GPC while the previous layer drains. */
  PCONV_STAGE_BULK = 0x8000u, /* tiled kernel, fp32 storage: input chunks are fetched by the copy engine
                                 (cp.async.bulk: a sub-tile's rows where the image is wider than a
                                 sub-tile and its width a multiple of 4, one span of the plane per
                                 channel where the sub-tile is as wide as the image and the plane a
                                 multiple of 4 elements; other shapes are unaffected) into a raw ring
                                 that the producer warps rebuild into the kernel's tile layout,
                                 instead of by 4-byte cp.async straight into that layout.  Off by
                                 default: measured slower on every VGG layer at batch 1 (a bulk copy
                                 takes ~2 us to land here and the raw ring is two deep: the first
                                 chunk is ready after 8.7-15 us against 4.3-5.6 us; 0.57 against
                                 0.38 ms for the stack). */
  PCONV_KERNEL_TENSOR = 0x800u /* fp16 storage, stride 1 only: the layer as a dense implicit GEMM over
                                  the zero-inserted weights on the tensor cores (tcgen05.mma, fp32
                                  accumulators in Tensor Memory).  It multiplies the pruned zeros too
                                  -- 9 / (4 x keep rate) times the surviving multiply-adds -- and is
                                  still several times faster for fp16 at the benchmark's keep rates,
                                  so the library picks it by default when the batch gives it enough
                                  tiles; fp16 products are exact in fp32, so the result differs from
                                  the sparse kernels by summation order only.  No fused max-pool. */
};

#define PCONV_MAX_PATTERNS 16

typedef struct {
  int c_out, c_in, stride, storage, n_patterns;
  long long kept_kernels;                       /* surviving (o,c) kernels */
  long long per_pattern[PCONV_MAX_PATTERNS];    /* kernels per pattern id; sums to kept_kernels */
  int min_per_filter, max_per_filter;           /* surviving kernels per filter */
  int n_groups, group_size;                     /* filter groups of the tiled layout */
  long long max_group_kernels, min_group_kernels; /* load balance of the grouping */
  long long packed_bytes;                       /* device bytes held by the handle */
  int canonical_patterns;                       /* 1 if every pattern is one of the canonical eight (one-byte codes) */
} pconv_stats_t;

/*
 * pconv_pack -- host-side packer: layerwise information extraction, filter/kernel reorder and
 * compressed weight storage (paper, "Compiler-assisted DNN Inference Framework": steps (i) and
 * (ii), and the index-free storage that pattern regularity allows).
 *
 *  w_oihw_host  [c_out][c_in][3][3] fp32, HOST; read during the call only (caller keeps it).
 *  patterns     n_patterns masks, HOST; each must have exactly 4 of 9 bits, all distinct,
 *               1 <= n_patterns <= PCONV_MAX_PATTERNS.
 *  stride       1 or 2.   storage  PCONV_F32 or PCONV_F16.   flags  0 or PCONV_STRICT4.
 *  stream       stream used for the upload; the call synchronises it before returning.
 *  out          receives the handle (owns its device buffers until pconv_free).
 *  bad_o,bad_c  optional; on PCONV_ERR_KERNEL_NOT_IN_SET / PCONV_ERR_RANGE they receive the first
 *               offending kernel (written on those errors only).
 *
 * A kernel's support is the set of its non-zero taps (-0.0 counts as zero).  Empty support =
 * pruned.  Otherwise it is assigned the lowest pattern id whose mask contains the support; zeros
 * inside the mask are stored as zeros.  A filter with no surviving kernel is legal.
 * Filters are permuted into groups of 16 balanced by surviving-kernel count; outputs are always
 * written at the original filter index.
 */
pconv_status pconv_pack(const float* w_oihw_host, int c_out, int c_in, const uint16_t* patterns,
                        int n_patterns, int stride, int storage, unsigned flags, void* stream,
                        pconv_handle** out, int* bad_o, int* bad_c);

/*
 * pconv_forward -- the hot path (Eq. 1 over surviving taps only: per-pattern 4-tap multiply-add,
 * the paper's "load redundancy elimination" -- only inputs under non-zero taps are touched --
 * with bias and ReLU fused).
 *
 *  x_dev     [n][c_in][h_in][w_in], DEVICE, storage type of the handle, 16-byte aligned.
 *  bias_dev  [c_out] fp32, DEVICE, or NULL for no bias.
 *  y_dev     [n][c_out][h_out][w_out], DEVICE, same storage type, 16-byte aligned, must not
 *            overlap x.  h_out = (h_in - 1) / stride + 1, likewise w_out.
 *  flags     PCONV_RELU, PCONV_POOL2X2, PCONV_REPRODUCIBLE and/or one PCONV_KERNEL_* bit.  With PCONV_POOL2X2 the
 *            layer's output is max-pooled before it is stored (the VGG stacks of the evaluation
 *            pool after conv2/4/7/10): y_dev is [n][c_out][h_out/2][w_out/2] (odd trailing row
 *            and column dropped, as pconv_maxpool2x2 does), h_out and w_out must be >= 2, and the
 *            call is refused with PCONV_ERR_UNSUPPORTED when no tiled kernel takes the shape or
 *            PCONV_KERNEL_SIMPLE is asked for.
 *
 * Asynchronous on `stream`; allocates nothing and never synchronises.  PCONV_ERR_CUDA reports
 * launch-time errors only.  A handle is immutable: concurrent forwards on several streams are
 * allowed.  n == 0 is a no-op.
 * The tiled kernels are launched with programmatic stream serialisation: a launch may begin its
 * own set-up while the previous kernel of the stream is still running, and waits for that kernel
 * to finish before it reads x or writes y, so stream order holds for every buffer named here.
 */
pconv_status pconv_forward(const pconv_handle* h, const void* x_dev, const float* bias_dev,
                           void* y_dev, int n, int h_in, int w_in, unsigned flags, void* stream);

/*
 * pconv_workspace_bytes / pconv_forward_ws -- the same operation as pconv_forward, with a
 * caller-provided scratch buffer that lets the library split the input-channel range of a layer
 * over several thread blocks when the batch offers too few output tiles to fill the GPU (batch-1
 * layers).  Partial sums are accumulated in the workspace with fp32 atomics (so the summation
 * order, not the result beyond rounding, varies from run to run) and the last warp to finish a
 * part of an output tile applies bias / ReLU and writes that part of y.  A forward that ends with
 * PCONV_ERR_DEVICE_TIMEOUT (pconv_device_status) may leave the workspace non-zero: clear it before
 * it is used again.  The paper has no counterpart; this is how the
 * build recovers parallelism that the paper's one-image-at-a-time mobile setting never needed.
 *
 *  bytes       receives the workspace size for this handle and input shape (0 = never split).
 *  ws_dev      DEVICE buffer of at least that size, 256-byte aligned, or NULL (= no split).
 *              It must be all zero before its first use; every forward leaves it all zero again.
 *              Forwards that share a workspace must not overlap in time.
 */
pconv_status pconv_workspace_bytes(const pconv_handle* h, int n, int h_in, int w_in, size_t* bytes);
pconv_status pconv_forward_ws(const pconv_handle* h, const void* x_dev, const float* bias_dev,
                              void* y_dev, int n, int h_in, int w_in, unsigned flags, void* ws_dev,
                              size_t ws_bytes, void* stream);

/*
 * pconv_forward_static_ws -- pconv_forward_ws for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for integration, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is forbidden or unavailable -- inside another
 * framework's memory plan that hands out no scratch, in a process whose allocator is owned by
 * someone else, or on a latency path that must never reach the driver's allocator.  Such callers
 * still own x, y and the bias, but have nowhere to put the channel-split workspace.  Here the
 * workspace is a fixed array inside the library's device image, PCONV_STATIC_WS_BYTES long; every
 * GPU that loads the library holds that much memory until the process exits.
 *
 *  - Same arguments and result as pconv_forward_ws without the workspace pair.
 *  - A shape whose workspace (pconv_workspace_bytes) exceeds PCONV_STATIC_WS_BYTES is refused
 *    with PCONV_ERR_WORKSPACE and nothing is launched; shapes that need no workspace always pass.
 *  - The call allocates nothing: no cudaMalloc / cudaFree, no allocating library routine.  The
 *    first call on each device looks up the array's device address (cudaGetSymbolAddress) and
 *    caches it; make that first call before starting any stream capture.
 *  - Every call uses the same array.  It is cleared on `stream` (cudaMemsetAsync over the part the
 *    shape needs) before the kernel runs, so an earlier call's leftovers never leak in -- but two
 *    calls that overlap on the GPU (different streams, or concurrent handles) race on it and give
 *    wrong results.  Serialise them, or use pconv_forward_ws with separate buffers.
 */
#define PCONV_STATIC_WS_BYTES (8u << 20)
pconv_status pconv_forward_static_ws(const pconv_handle* h, const void* x_dev,
                                     const float* bias_dev, void* y_dev, int n, int h_in, int w_in,
                                     unsigned flags, void* stream);

/* Releases the handle and its device buffers.  NULL is allowed. */
void pconv_free(pconv_handle* h);

/*
 * pconv_maxpool2x2 -- the plain 2x2 / stride-2 max-pool that separates the VGG blocks
 * (y[n,c,i,j] = max of x[n,c,2i..2i+1,2j..2j+1]; odd trailing rows/columns are dropped).
 * x_dev [n][c][h][w] and y_dev [n][c][h/2][w/2] are DEVICE pointers of `storage` type.
 */
pconv_status pconv_maxpool2x2(const void* x_dev, void* y_dev, int n, int c, int h, int w,
                              int storage, void* stream);

/* ---- test and inspection aids --------------------------------------------------------------- */

/* Decodes the DEVICE copy of the packed layer back to dense OIHW fp32 on the HOST
 * (w_out: c_out*c_in*9 floats).  fp16 handles return the rounded values.  Synchronous. */
pconv_status pconv_unpack(const pconv_handle* h, float* w_oihw_host_out);

/* How the tiled kernel would run one forward (the paper has no counterpart: its tuning step picks
 * tile sizes off line; here the library picks them per call from the shape). */
typedef struct pconv_plan_t {
  int generic_taps;      /* 1 = run-time masks (asked for with PCONV_KERNEL_GENERIC_TAPS) */
  int rows_per_lane;     /* output rows a lane owns per sub-tile: 4 or 8 (see PCONV_ROWS4 / PCONV_ROWS8) */
  int warps_per_unit;    /* consumer warps that share one (pixels, filter group) and split each chunk's
                            channels among themselves: 1, 2 or 4 */
  int channel_splits;    /* CTAs that share one output tile through the workspace (1 = none) */
  int groups_per_cta;    /* filter groups (of 16) per CTA */
  int pixel_sets;        /* independent sets of 64 x rows_per_lane pixels per CTA */
  int tile_width;        /* output columns of a sub-tile (2..32) */
  int stages;            /* depth of the staging ring */
  int smem_bytes;        /* dynamic shared memory the geometry needs */
  long long ctas;        /* CTAs launched */
  int staging;           /* how input chunks reach shared memory: 0 = element-wise (cp.async for fp32,
                            loads for fp16), 1 = fp16 pairs by cp.async into a raw ring, 2 / 3 = fp32 rows /
                            plane spans by bulk copies (cp.async.bulk) into a raw ring; the raw ring is
                            rebuilt into the kernel's tile layout by the producer warps */
  int tensor_path;       /* 1 = a default forward of this shape (no kernel-selection flag, no fused
                            pool) runs the dense tensor-core kernel instead of the tiled one; the
                            fields above still describe the tiled kernel */
} pconv_plan_t;

/* Test / tuning aid: fills *plan with the geometry a tiled forward of this shape would use;
 * with_workspace != 0 asks for the plan of pconv_forward_ws with a large enough workspace.
 * flags: 0, PCONV_KERNEL_GENERIC_TAPS, PCONV_ROWS4 or PCONV_ROWS8.  Launches nothing.  PCONV_ERR_UNSUPPORTED if the tiled
 * kernel cannot take the shape. */
pconv_status pconv_plan(const pconv_handle* h, int n, int h_in, int w_in, unsigned flags,
                        int with_workspace, pconv_plan_t* plan);

/* The same without a handle (host arithmetic only, needs no device): the plan for a layer of the
 * given shape with `kept_kernels` surviving kernels; canonical_patterns != 0 = the pattern set lies
 * inside the canonical eight. */
pconv_status pconv_plan_shape(int c_out, int c_in, long long kept_kernels, int stride, int storage,
                              int canonical_patterns, int n, int h_in, int w_in, unsigned flags,
                              int with_workspace, pconv_plan_t* plan);

/* Fills *out with the layer's structure counts. */
pconv_status pconv_stats(const pconv_handle* h, pconv_stats_t* out);

/* Copies the filter permutation to the HOST: perm_out[slot] = original filter index or -1 for a
 * padding slot; perm_out has n_groups*group_size entries. */
pconv_status pconv_filter_order(const pconv_handle* h, int* perm_out);

/* Synchronises the device and returns PCONV_ERR_DEVICE_TIMEOUT if any forward on this handle
 * abandoned a bounded wait since the handle was created (then *where, if given, receives the
 * internal wait id), else PCONV_OK. */
pconv_status pconv_device_status(const pconv_handle* h, int* where);

/* Constant, NUL-terminated description of a status. */
const char* pconv_status_str(pconv_status s);

/* ---- producing PCONV weights from dense ones --------------------------------------------------- */

/*
 * pconv_project -- projection of dense 3x3 kernels onto the PCONV constraint set: the step of the
 * ADMM-based training framework (accuracy-analysis section) that picks one pattern per kernel and
 * removes whole kernels.  Its formulas are in a supplement that is not available, so the Euclidean
 * projection is this build's reading.  Not part of the forward pass.
 *
 * For each kernel the pattern that retains the largest sum of squares is chosen (lowest pattern id
 * on ties); the k = round(keep * n_kernels) kernels with the largest retained sum survive,
 * together with every kernel that ties with the k-th; everything else becomes zero.  The sums are
 * formed in fp32, tap after tap in ascending tap order, multiply and add separately; where two
 * candidates differ by less than that rounding, the choice may differ from an exact evaluation.
 *
 *  w_dev           [n_kernels][9] fp32, DEVICE (an OIHW tensor with n_kernels = c_out * c_in).
 *  patterns        n_patterns masks, HOST, as for pconv_pack.
 *  keep            fraction of kernels to keep, 0..1.
 *  w_out_dev       [n_kernels][9] fp32, DEVICE; may be w_dev (in place).
 *  pattern_id_dev  [n_kernels] int8, DEVICE: the chosen pattern, -1 for pruned kernels.
 *  ws_dev          DEVICE scratch of pconv_project_workspace_bytes(n_kernels) bytes, 256-byte
 *                  aligned; contents irrelevant before and after.
 * Asynchronous on `stream`; allocates nothing.  PCONV_ERR_WORKSPACE if ws_bytes is too small.
 */
pconv_status pconv_project_workspace_bytes(long long n_kernels, size_t* bytes);
pconv_status pconv_project(const float* w_dev, long long n_kernels, const uint16_t* patterns,
                           int n_patterns, double keep, float* w_out_dev,
                           signed char* pattern_id_dev, void* ws_dev, size_t ws_bytes, void* stream);

/* ---- layer stacks ---------------------------------------------------------------------------- */

/*
 * pconv_stack_create -- chains layers: x -> conv(layers[0]) [-> maxpool] -> conv(layers[1]) ...
 * for a fixed input shape (n, h, w), as in the VGG-16 stacks of the evaluation.  The stack
 * allocates its two ping-pong activation buffers and the channel-split workspace of its layers on
 * the device here (never during forward), and
 * borrows the handles and bias pointers, which must outlive it.
 *  layers      n_layers handles (HOST array), same storage type, c_in of layer k+1 = c_out of k.
 *  bias_dev    n_layers DEVICE pointers (HOST array; entries may be NULL), or NULL.
 *  pool_after  n_layers bytes (HOST), non-zero = a 2x2 max-pool follows that layer; or NULL.
 *  flags       applied to every layer's forward (PCONV_RELU, kernel selection).
 */
pconv_status pconv_stack_create(const pconv_handle* const* layers, const float* const* bias_dev,
                                const unsigned char* pool_after, int n_layers, int n, int h, int w,
                                unsigned flags, pconv_stack** out);

/* Kernel launches one forward of the stack makes: a run of layers executed by one persistent
 * kernel counts once, a max-pool that is not fused into its layer counts as one more. */
pconv_status pconv_stack_launches(const pconv_stack* s, int* launches);

/* Shape of the stack's result: [n][c][h][w] (any pointer may be NULL). */
pconv_status pconv_stack_out_shape(const pconv_stack* s, int* n, int* c, int* h, int* w);

/* Runs the chain with DEVICE input and output; asynchronous on `stream`, allocates nothing.
 * Two forwards of the same stack must not overlap (they share the activation buffers). */
pconv_status pconv_stack_forward(pconv_stack* s, const void* x_dev, void* y_dev, void* stream);

/* The same with HOST input and output: copies x to the device, runs the chain, copies the result
 * back and synchronises `stream` before returning.  Pinned host memory makes the copies
 * asynchronous; pageable memory also works.  Uses two extra device buffers owned by the stack.
 * Returns PCONV_ERR_DEVICE_TIMEOUT (y_host then holds no valid result) if a kernel of this forward
 * abandoned a bounded wait; pconv_stack_status gives the wait id and makes the stack usable again. */
pconv_status pconv_stack_forward_host(pconv_stack* s, const void* x_host, void* y_host,
                                      void* stream);

/* Captures one forward from x_dev to y_dev into a CUDA graph kept by the stack (replacing an
 * earlier one), on a stream that allows capture (not the legacy default stream:
 * PCONV_ERR_UNSUPPORTED); the launches keep their programmatic dependencies inside the graph.
 * pconv_stack_replay launches it; x_dev and y_dev must then still be the same buffers.
 * pconv_stack_forward_host captures and replays on its own buffers where it can. */
pconv_status pconv_stack_capture(pconv_stack* s, const void* x_dev, void* y_dev, void* stream);
pconv_status pconv_stack_replay(pconv_stack* s, void* stream);

/* Synchronises the device and returns PCONV_ERR_DEVICE_TIMEOUT if a kernel launched by this stack
 * abandoned a bounded wait since the stack was created or since the last call of this function
 * (then *where, if given, receives the internal wait id, and the stack's output of that forward is
 * not valid), else PCONV_OK.  The call clears the record and zeroes the stack's channel-split
 * workspace again, so the stack can be used afterwards. */
pconv_status pconv_stack_status(pconv_stack* s, int* where);

/* Releases the stack (not the handles).  NULL is allowed. */
void pconv_stack_free(pconv_stack* s);


#ifdef __cplusplus
}
#endif
#endif /* PCONV_H_ */
