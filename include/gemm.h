/*
 * b200 GEMM -- C ABI of the dense matrix-multiply hot path for NVIDIA B200 (sm_100a).
 *
 *     D = act( alpha * op(A) * op(B) + beta * C + bias )
 *
 * This is the GEMM kernel family of the paper's case study (Section 5.4; the
 * strategy census of Table 1: tensor cores, tiling, vectorised and asynchronous
 * copies, swizzled layouts, multi-stage pipelines, thread-block swizzle),
 * re-designed for Blackwell: TMA-fed mbarrier pipelines, tcgen05.mma with the
 * accumulator in tensor memory, optional 2-CTA tiles, a persistent swizzled tile
 * scheduler, a TMEM -> shared -> TMA-store epilogue and a stream-K path for
 * skinny memory-bound shapes.  Plan-time selection of the path follows the
 * roofline classification of Section 4.3 (memory-bound / compute-bound by
 * arithmetic intensity against the machine ridge).
 *
 * Conventions
 *   Storage is ROW-MAJOR.  transa = GEMM_OP_N: A is stored M x K (lda >= K);
 *   GEMM_OP_T: A is stored K x M (lda >= M).  transb = GEMM_OP_N: B is stored
 *   K x N (ldb >= N); GEMM_OP_T: B is stored N x K (ldb >= K), i.e. "B
 *   column-major" / an nn.Linear weight.  C and D share one buffer: M x N,
 *   ldc >= N, read only when beta != 0 and then overwritten.  A and B have one
 *   16-bit dtype (bf16 or fp16); products are accumulated in fp32; C/D is fp32,
 *   bf16 or fp16 (round to nearest even, no saturation).  bias is fp32[N], added
 *   per output column and not scaled by alpha.  With batch_count > 1, matrix b
 *   starts b * stride_{a,b,c} elements into its buffer.
 *
 * Pointers named "device" must be device memory of the current CUDA device;
 * the caller owns every buffer (A, B, C, bias, workspace) and keeps it alive
 * until the stream work has completed.  The library owns the plan object and a
 * small device status word per plan.  No call synchronises the device except
 * gemm_plan_status() (gemm_plan_status_stream() waits for one stream only,
 * gemm_plan_status_async() for nothing).  Nothing throws; every failure is a
 * gemm_status_t, and an argument error launches nothing.
 */
#ifndef B200_GEMM_H_
#define B200_GEMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gemm_plan_s* gemm_plan_t; /* opaque, host memory */
typedef void* gemm_stream_t;             /* a cudaStream_t (NULL = default stream) */

typedef enum {
  GEMM_OK = 0,
  GEMM_ERR_NULL = 1,        /* a required pointer is NULL */
  GEMM_ERR_INVALID_ARG = 2, /* bad extent, leading dimension, enum value or struct_size */
  GEMM_ERR_UNSUPPORTED = 3, /* valid request the library does not implement */
  GEMM_ERR_ALIGNMENT = 4,   /* pointer, leading dimension or stride not 16-byte aligned */
  GEMM_ERR_WORKSPACE = 5,   /* workspace NULL or smaller than gemm_workspace_bytes() */
  GEMM_ERR_ARCH = 6,        /* no CUDA device, or the device is not sm_100 */
  GEMM_ERR_CUDA = 7,        /* a CUDA runtime / driver call failed */
  GEMM_ERR_TIMEOUT = 8      /* a bounded device-side wait expired (see gemm_plan_status) */
} gemm_status_t;

typedef enum {
  GEMM_BF16 = 0,
  GEMM_F16 = 1,
  GEMM_F32 = 2,
  GEMM_FP8_E4M3 = 3, /* 8-bit float, 4 exponent / 3 mantissa bits, no infinities (largest finite 448); operands only */
  GEMM_FP8_E5M2 = 4  /* 8-bit float, 5 exponent / 2 mantissa bits, IEEE-like; operands only */
} gemm_dtype_t;
typedef enum { GEMM_OP_N = 0, GEMM_OP_T = 1 } gemm_op_t;
typedef enum {
  GEMM_EPI_NONE = 0,
  GEMM_EPI_BIAS = 1,
  GEMM_EPI_RELU = 2,
  GEMM_EPI_BIAS_RELU = 3,
  GEMM_EPI_GELU_ERF = 4,     /* x * Phi(x) with the exact error function */
  GEMM_EPI_BIAS_GELU_ERF = 5,
  GEMM_EPI_GELU_TANH = 6,    /* 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))) */
  GEMM_EPI_BIAS_GELU_TANH = 7,
  GEMM_EPI_SILU = 8,         /* x / (1 + e^-x) */
  GEMM_EPI_BIAS_SILU = 9     /* odd values: the bias is added before the activation */
} gemm_epilogue_t;

/* Roofline class of a problem (Section 4.3 of the paper, applied at plan time). */
typedef enum { GEMM_REGIME_MEMORY = 0, GEMM_REGIME_MIDDLE = 1, GEMM_REGIME_COMPUTE = 2 } gemm_regime_t;
/* Kernel family a plan selected. */
typedef enum {
  GEMM_VARIANT_DENSE_1CTA = 1,      /* 128 x N tile per CTA, accumulator double buffered */
  GEMM_VARIANT_DENSE_2CTA = 2,      /* CTA pair, 256 x N pair tile, accumulator double buffered */
  GEMM_VARIANT_SKINNY_STREAMK = 3,  /* M <= 64 or N <= 64 (transa = N, transb = T, no batch): stream-K over the long operand */
  GEMM_VARIANT_DENSE_2CTA_WIDE = 4  /* CTA pair, 512 x 256 pair tile: least operand traffic per FLOP (N * output element size a
                                       multiple of 16 bytes; bias per column, ReLU and erf GELU only; no structure flags) */
} gemm_variant_t;

/* gemm_desc_t.flags: 0 = the plain problem, every choice left to the plan.  The first group are tuning fields (they
 * never change the result; gemm_tune chooses them by measurement), the second group changes what is computed or how
 * it is launched. */
#define GEMM_FLAG_VARIANT_SHIFT 4          /* bits 4-7: force a gemm_variant_t (0 = automatic) */
#define GEMM_FLAG_VARIANT_MASK 0xF0u
#define GEMM_FLAG_TILE_N_SHIFT 8           /* bits 8-12: force tile N (0 = automatic): 1 ... 16 = N / 16 (the 1-CTA and pair
                                              variants take multiples of 64 up to 256), 17 ... 20 = 320, 384, 448, 512
                                              (tiles of two MMAs side by side with a single accumulator buffer; B stored
                                              N x K only) */
#define GEMM_FLAG_TILE_N_MASK 0x1F00u
#define GEMM_FLAG_TAIL_SPLIT 0x2000u       /* when the last wave of a 1-CTA or pair plan would fill at most half of the SMs, cut
                                              its tiles into K slices, one per CTA or pair (the plan then wants a workspace for
                                              the flag words and raw accumulators of the further slices).  Without the flag this happens only
                                              for a handful of tiles with a very long K (three or more slices each); otherwise
                                              it is left to the caller and to gemm_tune: under the power cap idle SMs lend
                                              their budget to the busy ones, so it pays only on small problems (measured:
                                              -10 % at 1024 x 1024 x 4096, nothing at 4096^3) */
#define GEMM_FLAG_RASTER_SHIFT 16          /* bits 16-22: force the raster group height in tiles (0 = automatic) */
#define GEMM_FLAG_RASTER_MASK 0x7F0000u
#define GEMM_FLAG_STAGES_SHIFT 24          /* bits 24-27: force the pipeline depth (0 = automatic) */
#define GEMM_FLAG_STAGES_MASK 0xF000000u
#define GEMM_FLAG_KSLICES_SHIFT 28         /* bits 28-29: force the number of 128-byte K slices (64 elements of 16 bits, 128 of 8)
                                              per pipeline stage: 1 or 2, stream-K also 3 (0 = automatic) */
#define GEMM_FLAG_KSLICES_MASK 0x30000000u
#define GEMM_FLAG_NO_K_SERPENTINE 0x8u      /* walk K forwards in every tile (default: alternate tiles walk it backwards,
                                              which re-uses the operand lines L2 touched last) */
/* Structure of op(A) (M x K), a promise by the caller, not a mask: with A_LOWER every element with k > i IS zero in
 * memory, with A_UPPER every element with k < i.  The result is that of the plain GEMM; the library skips the K
 * ranges that can only contribute zeros (about half the work for a square A).  Dense variants only; at most one
 * of the two.  (The paper lists symmetric and triangular operands among its operator cases, Section 5.1.) */
#define GEMM_FLAG_A_LOWER 0x2u
#define GEMM_FLAG_A_UPPER 0x800000u
/* Symmetric results (D = A * A^T and the like; the paper's symmetric operator case, Section 5.1): only one triangle
 * of D is wanted.  With D_LOWER the elements with row >= column are computed, with D_UPPER those with row <= column;
 * output tiles that lie wholly in the other triangle are neither computed nor written (nor read, when beta != 0).
 * The tiles the diagonal crosses are computed in full, so an element outside the wanted triangle is either left
 * untouched or holds its value of the plain GEMM.  About half the work for a square D.  1-CTA and pair variants
 * only (not the wide pair tile, not stream-K); at most one of the two; combines with A_LOWER / A_UPPER and batches. */
#define GEMM_FLAG_D_LOWER 0x4000u
#define GEMM_FLAG_D_UPPER 0x8000u
/* gemm_desc_t.structure -- structure of op(B) (K x N), a promise like A_LOWER / A_UPPER: with B_LOWER every element
 * with k < j IS zero in memory, with B_UPPER every element with k > j.  The K ranges that can only contribute zeros
 * are skipped per output tile; together with A_UPPER and D_UPPER (or the three LOWER ones) this is the product of two
 * triangular matrices, itself triangular, at about a sixth of the dense work.  Dense 1-CTA and pair variants only; at
 * most one of the two. */
#define GEMM_STRUCT_B_LOWER 0x1u
#define GEMM_STRUCT_B_UPPER 0x2u
/* With GEMM_FLAG_D_LOWER or D_UPPER and M == N: after the product, the wanted triangle is copied into the other one, so
 * that D comes out symmetric (every element beyond the diagonal holds the bits of its mirror image; the diagonal and
 * the wanted triangle are those of the product).  A second, bandwidth-bound kernel on the same stream, per batch. */
#define GEMM_STRUCT_D_MIRROR 0x4u
/* gemm_desc_t.options.  GEMM_OPT_STREAMK_WORKSPACE: a stream-K plan hands its partial tiles over through the workspace
 * even where the CTAs of each output tile could be launched as a thread-block cluster and add them up in shared memory
 * (the default wherever all clusters fit on the device at once; it needs no workspace and is several microseconds
 * faster on mid-sized problems).  Results are bit-identical either way.  For callers that want no cluster launches,
 * and for tests. */
#define GEMM_OPT_STREAMK_WORKSPACE 0x1u
#define GEMM_FLAG_BIAS_PER_ROW 0x1u         /* the bias is fp32[M], one value per output row (default: fp32[N], one per
                                              column); not a tuning knob: it changes what is computed */
#define GEMM_FLAG_NO_EARLY_LAUNCH 0x4u       /* launch without programmatic dependent launch (default: the kernel may be
                                              scheduled while the previous kernel of the stream is finishing and does
                                              its set-up then; it waits for that kernel to complete before it reads or
                                              writes global memory) */
#define GEMM_FLAG_L2_HINTS 0x40000000u     /* load A with evict-last and B with evict-first L2 priority (default: normal) */
#define GEMM_FLAG_DEBUG_STALL 0x80000000u  /* test hook: in the plan's first run one producer arrival is withheld so that
                                              a bounded wait expires and GEMM_ERR_TIMEOUT is reported; later runs are normal */

typedef struct {
  uint32_t struct_size;  /* = sizeof(gemm_desc_t) */
  uint32_t flags;        /* GEMM_FLAG_* */
  int64_t M, N, K;       /* op(A) is M x K, op(B) is K x N, C/D is M x N; all >= 1 */
  int32_t transa, transb;     /* gemm_op_t */
  int32_t ab_dtype;           /* gemm_dtype_t: GEMM_BF16, GEMM_F16, or an 8-bit float (then transa = N and transb = T), for both A
                                 and B */
  int32_t c_dtype;            /* gemm_dtype_t of C/D */
  int64_t lda, ldb, ldc;      /* leading dimensions in elements */
  int32_t batch_count;        /* >= 1 */
  int32_t epilogue;           /* gemm_epilogue_t */
  int64_t stride_a, stride_b, stride_c; /* elements between consecutive matrices; ignored when batch_count == 1 */
  uint32_t structure;         /* GEMM_STRUCT_*: further structure promises (flags has no bit left); 0 = none */
  uint32_t options;           /* GEMM_OPT_*: 0 = none; unknown bits are an error */
} gemm_desc_t;

typedef struct {
  uint32_t struct_size;  /* = sizeof(gemm_info_t), set by the caller */
  int32_t variant;       /* gemm_variant_t */
  int32_t regime;        /* gemm_regime_t */
  int32_t tile_m, tile_n, tile_k; /* output tile of one CTA (1-CTA) or CTA pair (2-CTA); skinny: tile over the long extent, padded short extent, K */
  int32_t stages;        /* depth of the shared-memory ring */
  int32_t cluster_size;  /* 1 or 2 */
  int32_t grid;          /* CTAs launched */
  int32_t raster_group;  /* tile rows swept together by the scheduler */
  int32_t split;         /* skinny: maximum number of CTAs contributing to one output tile; dense: 1 */
  int32_t smem_bytes;    /* dynamic shared memory per CTA */
  int64_t num_tiles;     /* output tiles (dense) or k-block work units (skinny) */
  double flops;          /* 2 * M * N * K * batch */
  double min_bytes;      /* compulsory HBM traffic */
  double intensity;      /* flops / min_bytes */
  size_t workspace_bytes;
} gemm_info_t;

/*
 * gemm_plan -- validate `desc` (host pointer), classify the problem on the
 * roofline (Section 4.3), choose the kernel variant, tile shape, pipeline depth,
 * cluster size, raster order and stream-K split, and return a plan (host
 * memory).  If a CUDA device is current, also allocates the plan's 16-byte
 * device status word and reads the SM count; without a device the plan is still
 * created (148 SMs assumed) so that planning can be inspected, and gemm_run
 * reports GEMM_ERR_ARCH.  Errors: NULL -> GEMM_ERR_NULL; extents < 1, leading
 * dimension smaller than the row length, unknown enum, wrong struct_size ->
 * GEMM_ERR_INVALID_ARG; lda/ldb/ldc or batch strides whose byte size is not a
 * multiple of 16 -> GEMM_ERR_ALIGNMENT; fp32 A/B or an impossible forced
 * variant -> GEMM_ERR_UNSUPPORTED.
 */
gemm_status_t gemm_plan(const gemm_desc_t* desc, gemm_plan_t* out_plan);

/* Bytes of device workspace gemm_run needs for this plan: 0 for the plain dense variants; for stream-K the arrival
 * words of the output tiles followed by the partial tiles, for a dense plan with a tail split the flag words followed
 * by the partial accumulators.  The workspace needs no initialisation and may hold anything.  0 on a NULL plan. */
size_t gemm_workspace_bytes(gemm_plan_t plan);

/*
 * gemm_run -- enqueue D = act(alpha*op(A)*op(B) + beta*C + bias) on `stream`
 * (asynchronous; the hot path of Section 5.4).  A, B, C: device pointers, 16-byte
 * aligned, laid out as `desc` said.  bias: device fp32[N] (fp32[M] with
 * GEMM_FLAG_BIAS_PER_ROW), shared by all batches, required iff the epilogue
 * has a bias.  C is read only when beta != 0, and only the M x N elements of D (per batch) are written: row padding
 * (ldc > N) and gaps between batches keep their contents, so D may be a column block of a wider matrix.  workspace: device
 * memory of at least gemm_workspace_bytes(plan) bytes, 16-byte aligned (may be NULL when
 * that is 0), with any contents: the hand-shake words at its head carry a 48-bit tag that is new with every run and
 * spread pseudo-randomly over its bits, so whatever the memory held before reads as "nothing yet" (a stale 64-bit word
 * passes for this run's only if 48 of its bits equal that one value; a caller who wants certainty zeroes the workspace
 * once after allocating it).  Runs of one plan may overlap on the GPU (several streams, several host
 * threads) as long as runs that overlap use DIFFERENT workspaces; they share only the status word, which then reports
 * a timeout of any of them.  Runs that share a workspace must be ordered (one stream, or events).  One kind of plan
 * wants the SMs it was planned for: a dense plan that cuts tiles along K (a dense variant with gemm_workspace_bytes > 0)
 * has one CTA per tile wait, within the plan's time limit, for the other slices of that tile, which are CTAs of the same
 * launch; if other work on the device keeps those from becoming resident the wait can run out (GEMM_ERR_TIMEOUT, never a
 * hang).  Stream-K plans never wait for another CTA, inside clusters only at the hardware's cluster barrier.  alpha and beta are
 * host scalars.  The call only fetches or encodes tensor maps on the host (a plan remembers the maps of the operand
 * addresses it has seen, so a repeated address costs no encoding) and launches: once a plan has run once (which sets
 * kernel attributes), further runs may be recorded by stream capture into a CUDA graph (tested).  A captured run replays
 * with the tag it was captured with, which is safe because every run leaves its hand-shake words at zero; only after a
 * GEMM_ERR_TIMEOUT must a captured graph of a plan with a workspace be captured again (or the first
 * gemm_workspace_bytes bytes of that workspace be zeroed) before it is replayed.  Errors are returned before anything is launched:
 * GEMM_ERR_NULL, GEMM_ERR_ALIGNMENT, GEMM_ERR_WORKSPACE, GEMM_ERR_ARCH,
 * GEMM_ERR_INVALID_ARG (the current CUDA device is not the one the plan was
 * made on), GEMM_ERR_CUDA (tensor-map encoding or launch failure).
 */
gemm_status_t gemm_run(gemm_plan_t plan, const void* A, const void* B, void* C, const float* bias, float alpha,
                       float beta, void* workspace, size_t workspace_bytes, gemm_stream_t stream);

/*
 * The plan's status word: GEMM_OK, or GEMM_ERR_TIMEOUT if a bounded device-side wait of an earlier run expired (the
 * kernel then returned early and its output is undefined; until the word has been taken, later runs of the plan may
 * give up early as well, and a stream-K plan does not finish split tiles).  Taking the word clears it and puts the
 * plan back in order.  (The bounded waits are this library's; the paper's kernels have no counterpart.)  Three forms:
 *
 * gemm_plan_status_async -- enqueue on `stream` a one-thread kernel that takes the word into page-locked host
 *   memory owned by the plan; returns at once and synchronises nothing (the first call on a plan allocates that
 *   host word: make it outside stream capture).  gemm_plan_status_result then reports the word that was taken
 *   last; the caller must first have waited, by any means (event, stream synchronise, graph completion), for the
 *   stream to get past the enqueued kernel.  Without an earlier _async call it returns GEMM_OK.
 * gemm_plan_status_stream -- the two together around cudaStreamSynchronize(stream): waits for that one stream only.
 *   This is the form to use after runs on `stream`.
 * gemm_plan_status -- the same after cudaDeviceSynchronize(): for callers that do not know which streams ran the
 *   plan.  It stalls every stream of the device and must not be used while a stream capture is under way.
 * Errors: GEMM_ERR_NULL; GEMM_ERR_ARCH (plan made without a device); GEMM_ERR_INVALID_ARG (the current device is not
 * the plan's); GEMM_ERR_CUDA.
 */
gemm_status_t gemm_plan_status_async(gemm_plan_t plan, gemm_stream_t stream);
gemm_status_t gemm_plan_status_result(gemm_plan_t plan);
gemm_status_t gemm_plan_status_stream(gemm_plan_t plan, gemm_stream_t stream);
gemm_status_t gemm_plan_status(gemm_plan_t plan);

/* Override the device-side wait limit of this plan (default 2000 ms; minimum 1 ms). */
gemm_status_t gemm_plan_set_timeout_ms(gemm_plan_t plan, uint32_t ms);

/* Copy the plan's decisions into *out (out->struct_size must be sizeof(gemm_info_t)). */
gemm_status_t gemm_plan_info(gemm_plan_t plan, gemm_info_t* out);

/*
 * gemm_plan_schedule -- list the work items of a plan in the order its CTAs execute them: which CTA (for the pair
 * variants: which CTA pair) computes which output tile over which part of K.  This is the persistent tile scheduler
 * with its swizzled (grouped) raster order -- the "thread-block swizzle" strategy of the paper's Table 1 -- the
 * schedule dealt ahead of time for structured problems, the tail split and the stream-K decomposition, walked on the
 * host by the same functions the kernels run; it needs no device.  Meant for inspection and for tests (every wanted
 * tile exactly once, every K stage of a split tile exactly once).
 *   items: host array of `capacity` entries (may be NULL when capacity is 0); *count receives the number of items
 *   the plan has, which may exceed capacity (only the first `capacity` are written).
 * Errors: GEMM_ERR_NULL.
 */
typedef struct {
  int32_t cta;       /* CTA (pair variants: cluster) that executes the item; items of one CTA appear in execution order */
  int32_t batch;     /* matrix of the batch */
  int32_t tile_row;  /* output tile, in units of gemm_info_t.tile_m rows ... */
  int32_t tile_col;  /* ... and tile_n columns (stream-K: the 128-wide tile along the long extent, the other index 0) */
  int32_t k_begin;   /* ring stages [k_begin, k_end) of gemm_info_t.tile_k elements of K each */
  int32_t k_end;
  int32_t slice;     /* -1: the item computes its tile alone; >= 0: one of several K slices of the tile (0 finishes it
                        in a tail split; stream-K: position among the tile's contributors, the last arrival finishes) */
  int32_t reserved;
} gemm_work_item_t;
gemm_status_t gemm_plan_schedule(gemm_plan_t plan, gemm_work_item_t* items, size_t capacity, size_t* count);

/* Free the plan and its status word.  NULL is accepted. */
gemm_status_t gemm_destroy(gemm_plan_t plan);

/*
 * gemm_skinny_run_noalloc -- the paper has no counterpart; this is a library convenience.  It runs the
 * skinny stream-K path (transa = N, transb = T, batch_count = 1, M <= 64) WITHOUT a plan and WITHOUT a
 * caller workspace, for callers that may not allocate device memory while they run: a process that gave
 * the whole GPU to its own memory pool at start-up, a latency-critical loop that cannot take the
 * device-wide synchronisation of cudaMalloc, or code under a "no allocator calls after initialisation"
 * rule.  The call makes no cudaMalloc / cudaFree and uses no allocating library routine; the plan is built
 * on the stack and the kernel's scratch (status word, arrival counters, partial tiles) is a fixed 4 MiB
 * array inside the library, present on every GPU that loads the library until the process exits.
 *   desc, A, B, C, bias, alpha, beta, stream: as for gemm_plan / gemm_run.  The tuning fields of desc->flags are
 *   ignored; a flag or structure bit that changes what is computed (GEMM_FLAG_A_*, GEMM_FLAG_D_*,
 *   GEMM_FLAG_BIAS_PER_ROW, any GEMM_STRUCT_*) is refused with GEMM_ERR_UNSUPPORTED, as the stream-K plans refuse it.
 *   sync_and_check: 0 = asynchronous, only launch-time errors are reported; non-zero = wait for `stream`
 *   and return GEMM_ERR_TIMEOUT if a bounded device-side wait expired.
 * Limits and rules: problems whose scratch need exceeds the array (with 148 SMs: M > 16) are rejected
 * with GEMM_ERR_WORKSPACE and nothing is launched (gemm_last_cuda_error() gives the sizes).  The first
 * call on each device resolves the array's device address and sets a kernel attribute; under CUDA's lazy
 * module loading it is also the moment the driver loads the library's module (the kernel image and the
 * 4 MiB array), which takes device memory once and can fail on a GPU that has none left.  So make that
 * first call during initialisation -- before the GPU's memory is handed to the caller's own pool and before
 * any stream capture begins; every later call on the device allocates nothing.  All calls on a device share the one array: it keeps the
 * previous call's contents (the call clears what must start at zero), and two calls whose kernels overlap
 * on the GPU (different streams, or several host threads) race on it -- serialise them.
 */
gemm_status_t gemm_skinny_run_noalloc(const gemm_desc_t* desc, const void* A, const void* B, void* C, const float* bias,
                                      float alpha, float beta, gemm_stream_t stream, int sync_and_check);

/*
 * Measured plan selection.  The paper's search (Section 4.3: the roofline class of a kernel steers which
 * optimisations are tried, and candidates are kept by measured time) has one part that needs no language
 * model: among the handful of kernel families, tile widths, ring shapes and raster heights this library
 * has, try the ones the problem's roofline class makes plausible, time them on the caller's buffers, keep
 * the fastest and remember it for the shape.
 *
 * GEMM_TUNE_MAX_CANDIDATES bounds the report arrays.
 */
#define GEMM_TUNE_MAX_CANDIDATES 32
typedef struct {
  uint32_t struct_size;         /* = sizeof(gemm_tune_report_t) */
  int32_t candidates_tried;     /* plans that ran and were timed (entries of tried_*) */
  int32_t candidates_skipped;   /* refused by gemm_plan for this problem, or needing more workspace than given */
  uint32_t best_flags;          /* gemm_desc_t.flags of the winner (tuning fields filled in) */
  float best_ms;                /* its mean device time per launch */
  float auto_ms;                /* the same for the untuned automatic plan, for comparison */
  uint32_t tried_flags[GEMM_TUNE_MAX_CANDIDATES];
  float tried_ms[GEMM_TUNE_MAX_CANDIDATES];
} gemm_tune_report_t;

/* Workspace that lets gemm_tune try every candidate of this problem (0 if none needs any). */
size_t gemm_tune_workspace_bytes(const gemm_desc_t* desc);

/*
 * gemm_tune -- plan `desc` by measurement.  A, B, C, bias, alpha, beta, workspace, stream: as for gemm_run;
 * every candidate is RUN on them (2 warm-up launches, then `iterations` timed launches between CUDA events
 * on `stream`; iterations < 1 means 10), so C is overwritten again and again (and, with beta != 0, keeps
 * accumulating): pass scratch data.  The call synchronises `stream` several times.  Tuning fields of
 * desc->flags (variant, tile, raster, stages, K slices) are ignored; the other flags are kept.
 * On success *out_plan is the winner, ready for gemm_run, and the winner's flags are remembered for this
 * device and shape: later gemm_plan calls with the same shape and no tuning fields set use them.
 * report may be NULL.  Errors: as gemm_plan and gemm_run; GEMM_ERR_TIMEOUT if a candidate's device-side
 * wait expired (nothing is remembered then); GEMM_ERR_UNSUPPORTED if no candidate could run.
 */
gemm_status_t gemm_tune(const gemm_desc_t* desc, const void* A, const void* B, void* C, const float* bias, float alpha,
                        float beta, void* workspace, size_t workspace_bytes, gemm_stream_t stream, int iterations,
                        gemm_plan_t* out_plan, gemm_tune_report_t* report);

/* Forget every remembered tuning result (all devices). */
void gemm_tune_cache_clear(void);

/*
 * Keep tuning results across processes (the paper's search runs once per operator and hardware, Section 4; this is the
 * memory of that search).  gemm_tune_cache_save writes what was remembered for the CURRENT device to a text file
 * (overwriting it); gemm_tune_cache_load adds the file's results to the current device's, after which gemm_plan picks
 * them up like results of gemm_tune in this process.  path: host string.  *entries (may be NULL): results written /
 * read.  Errors: GEMM_ERR_NULL; GEMM_ERR_ARCH without a CUDA device; GEMM_ERR_INVALID_ARG when the file cannot be
 * opened or is malformed (nothing is loaded then); GEMM_ERR_UNSUPPORTED when the file was written on another GPU
 * model or SM count.  A remembered choice that this version of the library cannot plan is ignored by gemm_plan.
 */
gemm_status_t gemm_tune_cache_save(const char* path, int* entries);
gemm_status_t gemm_tune_cache_load(const char* path, int* entries);

/*
 * GEMM on HOST-resident operands (the end-to-end path of a caller whose matrices live in host memory; the
 * paper's measurements start with the data on the GPU, so this has no counterpart there).  The output rows are cut
 * into `panels` row panels; panel p's slice of A is copied in while panel p-1 is multiplied and panel p-2's result is
 * copied out, on three streams owned by the handle, so the whole call costs little more than the longer of the two
 * copy directions.  B (and the bias) go to the device once per run.
 *
 * gemm_host_create: desc as for gemm_plan, with transa = N and batch_count = 1 (row panels of A and C must be
 * contiguous row ranges); panels = 0 picks a count (about 8, fewer for small M).  Allocates the device staging
 * buffers (B, two A panels, two C panels, a workspace if the panel plan wants one), the streams and the events, on
 * the current device.  Errors: as gemm_plan; GEMM_ERR_UNSUPPORTED for transa = T, a batch, a triangular op(A) or a wanted triangle of D; GEMM_ERR_CUDA if an
 * allocation fails (nothing is leaked).
 * gemm_host_run: hA, hB, hC (and hbias, iff the epilogue has a bias): HOST pointers laid out as desc says; page-locked
 * memory is what makes the copies overlap (pageable memory works, without overlap).  hC is read only when beta != 0
 * and receives D.  Blocks until D is complete in hC.  Returns GEMM_ERR_TIMEOUT if a device-side wait expired.
 * One run at a time per handle.  gemm_host_destroy frees everything; NULL is accepted.
 */
typedef struct gemm_host_s* gemm_host_t;
gemm_status_t gemm_host_create(const gemm_desc_t* desc, int panels, gemm_host_t* out);
gemm_status_t gemm_host_run(gemm_host_t h, const void* hA, const void* hB, void* hC, const float* hbias, float alpha, float beta);
/* Row panels the handle uses (0 on NULL). */
int gemm_host_panels(gemm_host_t h);
gemm_status_t gemm_host_destroy(gemm_host_t h);

/* Static string for a status code. */
const char* gemm_status_string(gemm_status_t s);

/* Detail of the last GEMM_ERR_CUDA on this thread (CUDA error name), or "". */
const char* gemm_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* B200_GEMM_H_ */
