/*
 * exo_gemm.h -- C ABI of the B200 (sm_100a) tensor-core GEMM library.
 *
 * Operation.  C = alpha * A * B + beta * C with 16-bit floating-point operands
 * (bf16 or fp16) and fp32 accumulation: the matrix-multiply-accumulate the
 * paper's kernels implement ("D += matmul(A, B)", Section 2.2 listings; the
 * GEMM kernels of Section 6, "Evaluation", measured against BLAS Sgemm, whose
 * alpha/beta/layout/leading-dimension conventions this interface follows).
 *
 * Every compute step runs in hand-written CUDA kernels on the device; there is
 * no CPU path and no fallback: on a device that is not compute capability 10.x
 * exo_gemm_create fails with EXO_GEMM_ERR_ARCH.
 *
 * Plain C.  Callers need no CUDA headers: the stream is passed as void*.
 */
#ifndef EXO_GEMM_H_
#define EXO_GEMM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct exo_gemm_plan* exo_gemm_handle_t; /* opaque; owned by the library */

typedef enum {
  EXO_GEMM_OK = 0,
  EXO_GEMM_ERR_NULL = 1,           /* a required pointer argument is NULL                         */
  EXO_GEMM_ERR_INVALID_ARG = 2,    /* negative or oversized dimension, ld below extent, bad enum   */
  EXO_GEMM_ERR_UNSUPPORTED = 3,    /* legal BLAS call outside the supported set (see below)       */
  EXO_GEMM_ERR_ALIGNMENT = 4,      /* a matrix base pointer is not 16-byte aligned (run)          */
  EXO_GEMM_ERR_ARCH = 5,           /* device is not compute capability 10.x                        */
  EXO_GEMM_ERR_CUDA = 6,           /* a CUDA runtime/driver call failed                            */
  EXO_GEMM_ERR_DEVICE_TIMEOUT = 7  /* a bounded device-side wait gave up in an earlier launch      */
} exo_gemm_status_t;

typedef enum { EXO_GEMM_BF16 = 0, EXO_GEMM_FP16 = 1, EXO_GEMM_FP32 = 2 } exo_gemm_dtype_t;
typedef enum { EXO_GEMM_ROW_MAJOR = 0, EXO_GEMM_COL_MAJOR = 1 } exo_gemm_layout_t;

/*
 * Tuning overrides, OR-ed into exo_gemm_desc_t.flags.  0 = let the library choose.
 *   bits 0..1   cta_group: 1 = one SM per tile, 2 = a pair of SMs (2-CTA cluster) per tile
 *   bits 2..5   tile N / 64 (1, 2 or 4  =>  64, 128 or 256 columns per tile)
 *   bits 6..9   raster band width in tiles (1..15)
 *   bit  10     raster direction: 0 = library choice, set = bands along M instead of N
 *   bit  11     the parts of a cut tail tile meet in C by TMA reduce-add (see EXO_GEMM_FLAG_SPLIT_REDUCE_ADD)
 *   bits 12..19 grid limit: launch at most this many CTAs (multiple of cta_group), 0 = all SMs
 *   bits 20..21 k sub-blocks (of 64 elements) per pipeline stage: 1 or 2
 *   bits 22..23 staging buffers per epilogue warp: 1 or 2 (also keeps the staged epilogue -- registers ->
 *               swizzled shared memory -> TMA store -- in runs that could store C straight from registers)
 *   bits 24..27 upper limit on the pipeline depth (2..8)
 *   bits 28..31 K-slices per tile of the partial last wave: 1 = never cut, 2..8 = at most this many on average
 */
#define EXO_GEMM_FLAG_CTA_GROUP(g)  ((uint32_t)(g) & 3u)
#define EXO_GEMM_FLAG_TILE_N(n)     ((((uint32_t)(n) / 64u) & 15u) << 2)
#define EXO_GEMM_FLAG_BAND(b)       (((uint32_t)(b) & 15u) << 6)
#define EXO_GEMM_FLAG_BANDS_ALONG_M (1u << 10)
/*
 * The unordered form of the K split, as in the paper's Section 6 split-K kernels (TMA reduce-add of fp32
 * partial sums): every part of a cut tile adds alpha * (its partial sum) onto C with
 * cp.reduce.async.bulk.tensor instead of handing it to the owning part through a workspace.  No
 * workspace, no waiting; the order of the additions is the memory system's, so results are not
 * bitwise reproducible from run to run.  fp32 C only (ERR_UNSUPPORTED from validate otherwise), plain
 * tiles only (ERR_INVALID_ARG together with SHARE_ALWAYS / SHARE_SUBSTITUTED or CTA_ROWS(256));
 * exo_gemm_run then accepts beta == 1 (C is accumulated onto) and beta == 0 (the run first clears C
 * with a memset on the same stream) and returns ERR_UNSUPPORTED for any other beta.  Off by default:
 * the ordered workspace reduction measured level or faster and is deterministic.
 */
#define EXO_GEMM_FLAG_SPLIT_REDUCE_ADD (1u << 11)
#define EXO_GEMM_FLAG_GRID_LIMIT(c) (((uint32_t)(c) & 255u) << 12)
#define EXO_GEMM_FLAG_K_SUBBLOCKS(k) (((uint32_t)(k) & 3u) << 20)
#define EXO_GEMM_FLAG_EPI_BUFFERS(b) (((uint32_t)(b) & 3u) << 22)
#define EXO_GEMM_FLAG_MAX_STAGES(s) (((uint32_t)(s) & 15u) << 24)
#define EXO_GEMM_FLAG_SPLIT_K(f) (((uint32_t)(f) & 15u) << 28)

/*
 * flags2, bits 0-1: clusters of two CTA pairs (4 SMs) that compute neighbouring 256 x 256
 * tiles of the same rows of C and share the loads of A -- each of the two CTAs that need a
 * 128-row block fetches half of it and the TMA copy is multicast to both (the paper's
 * Section 6 kernels multicast the operand their cluster has in common in the same way).
 * The grid is cut into slots of four CTAs; the launch prefers 4-CTA clusters and lets the
 * device substitute two plain pairs for a slot where no four SMs of one GPC are free (those
 * pairs compute the same two tiles, each loading all of its A rows), so every SM is used.
 * 0 = the library decides, 1 = never, 2 = always (ERR_UNSUPPORTED from create /
 * run_static / plan_preview if the loaded library was built without the variant, see
 * exo_gemm_has_shared_operand_clusters; ERR_INVALID_ARG together with a CTA_GROUP(1),
 * a TILE_N other than 256 or a GRID_LIMIT that is not a multiple of 4), 3 = as 2 but every
 * slot is launched as two plain pairs (a test aid for the substitute path).
 */
#define EXO_GEMM_FLAG2_SHARE_AUTO 0u
#define EXO_GEMM_FLAG2_SHARE_NEVER 1u
#define EXO_GEMM_FLAG2_SHARE_ALWAYS 2u
#define EXO_GEMM_FLAG2_SHARE_SUBSTITUTED 3u

/*
 * flags2, bits 2-3: rows of C per CTA.  0 = the library decides, 1 = 128 (one TMEM accumulator
 * per tile, the other one belongs to the next tile, so epilogue and main loop overlap),
 * 2 = 256, the "tall" tile: a CTA pair computes 512 x 256, both accumulators of a CTA belong to
 * one tile and share each B block, which moves a quarter less operand data into shared memory
 * per flop at the price of an exposed epilogue.  2 needs the 2-CTA 256-column tile with one
 * 64-wide k-block per stage: ERR_INVALID_ARG together with CTA_GROUP(1), another TILE_N,
 * K_SUBBLOCKS(2) or a SHARE_ALWAYS / SHARE_SUBSTITUTED request.  3 is invalid.
 */
#define EXO_GEMM_FLAG2_CTA_ROWS(r) ((((uint32_t)(r) / 128u) & 3u) << 2)

/*
 * flags2, bits 4-5: the one-tile-per-CTA kernel for problems of less than one wave (the small
 * matrices of the paper's Section 6, where a run is a chain of latencies rather than a stream of
 * tiles).  One CTA per 128 x 64 or 128 x 128 tile, all launched at once; the copies of the first
 * k-blocks are issued before the CTA's set-up barrier, C_in is fetched during the main loop, and
 * no warp waits for another at the end.  It never cuts K and has no strided-batch form.
 * With SPLIT_K(2) or SPLIT_K(4) the K loop of every tile is cut over a cluster of that many CTAs,
 * which exchange their partial sums through distributed shared memory (no workspace).  Together
 * with CTA_GROUP(2) the request means the same kernel structure for a PAIR of CTAs per 256 x 128
 * or 256 x 256 tile (tcgen05 cta_group::2; K is never cut there); the library never picks that
 * form on its own (it measured level with the persistent kernel).
 * 0 = the library decides, 1 = never, 2 = always (ERR_INVALID_ARG together with TILE_N(256)
 * unless CTA_GROUP(2) is given, a SHARE_ALWAYS / SHARE_SUBSTITUTED or CTA_ROWS(256) request,
 * SPLIT_K other than 1, 2, 4 (other than 1 with CTA_GROUP(2)), SPLIT_REDUCE_ADD or a
 * GRID_LIMIT; a batched plan ignores it).  3 is invalid.
 */
#define EXO_GEMM_FLAG2_LEAN_AUTO 0u
#define EXO_GEMM_FLAG2_LEAN_NEVER (1u << 4)
#define EXO_GEMM_FLAG2_LEAN_ALWAYS (2u << 4)

/*
 * Problem descriptor.  Logical shapes: A is M x K, B is K x N, C is M x N.
 * Leading dimensions are in elements: for a row-major matrix ld >= #columns, for
 * a column-major matrix ld >= #rows.
 *
 * Supported set: ab_dtype in {BF16, FP16, FP32}; c_dtype FP32 or equal to ab_dtype;
 * any of the 8 layout combinations; 0 <= M, N, K <= 2^31 - 1.  FP32 operands are
 * multiplied as tf32 (the tensor core reads sign, exponent and the upper 10 fraction
 * bits of each fp32 operand and ignores the rest; products are accumulated in fp32):
 * this is the precision of the paper's own Section 6 kernels and of
 * CUBLAS_TF32_TENSOR_OP_MATH (M/N-contiguous FP32 operands are staged with the 128-byte
 * swizzle in 32-byte atoms that tcgen05 wants for transposed 32-bit operands).  Operands and
 * results move by TMA, which addresses rows by a byte stride that is a multiple of 16: a
 * matrix whose leading dimension times its element size is such a multiple (16-bit:
 * ld % 8 == 0, fp32: ld % 4 == 0) is used in place and its base pointer passed to
 * exo_gemm_run must be 16-byte aligned.  Any other leading dimension is legal too: the plan
 * then owns an aligned copy of that matrix and every run makes one extra pass over it
 * (operands copied in before the GEMM, C copied out after it and, if beta != 0, in before
 * it; the base pointer only needs the alignment of its element type; see
 * exo_gemm_info_t.repacked).  That path has no strided-batch form and is not available to
 * the allocation-free entry point (ERR_UNSUPPORTED from both).  Legal BLAS calls outside
 * this set return EXO_GEMM_ERR_UNSUPPORTED.
 */
typedef struct {
  int64_t M, N, K;
  int32_t ab_dtype;                     /* exo_gemm_dtype_t of both operands (FP32 = tf32 math) */
  int32_t c_dtype;                      /* exo_gemm_dtype_t: FP32 or the same as ab_dtype      */
  int32_t a_layout, b_layout, c_layout; /* exo_gemm_layout_t                                   */
  int32_t device;                       /* CUDA device ordinal; -1 = the current device        */
  int64_t lda, ldb, ldc;                /* elements                                            */
  uint32_t flags;                       /* 0, or EXO_GEMM_FLAG_* overrides                     */
  uint32_t flags2;                      /* 0, or EXO_GEMM_FLAG2_*; bits 6.. must be 0          */
} exo_gemm_desc_t;

/* What a plan decided; filled by exo_gemm_get_info. */
typedef struct {
  int32_t cta_group;      /* 1 or 2 SMs per tile                                               */
  int32_t tile_m, tile_n; /* output tile of one CTA group: tile_m = 128 * cta_group rows, or
                             256 * cta_group (= 512) for the tall tile, EXO_GEMM_FLAG2_CTA_ROWS  */
  int32_t tile_k;         /* k-elements staged per pipeline stage (64 or 128; tf32: 32 or 64)  */
  int32_t stages;         /* depth of the shared-memory operand ring                           */
  int32_t grid;           /* CTAs launched (persistent)                                        */
  int32_t smem_bytes;     /* dynamic shared memory per CTA                                     */
  int32_t tmem_columns;   /* tensor-memory columns allocated per CTA (2 accumulators)          */
  int32_t tiles_m, tiles_n;
  int32_t raster_along_m; /* 1: bands run along M, tiles inside a band walk N first            */
  int32_t raster_band;    /* band width in tiles                                               */
  int32_t swapped;        /* 1: column-major C computed as C^T = B^T A^T                       */
  int32_t sm_count;
  int32_t kernel_launches_per_run; /* 1, or 0 for an empty problem                             */
  int32_t epilogue_buffers; /* staging buffers per epilogue warp (1 or 2)                      */
  int32_t split_k;         /* the most K-slices a tile of the partial last wave is cut into (1 = none) */
  int32_t tail_tiles;      /* tiles in that partial last wave                                  */
  int32_t workspace_bytes; /* device scratch the plan owns for the slices' partial sums        */
  int32_t batch_count;     /* matrices per launch (1 unless created by exo_gemm_create_batched) */
  int32_t cluster_size;    /* CTAs per cluster: cta_group, or 4 when two pairs share the loads of A
                              (tiles_n then counts 2 * tile_n columns per step)                 */
  int32_t tail_workers;    /* workers that share the k-blocks of the tail tiles in equal ranges (0 = none) */
  int32_t stages_direct;   /* depth of the operand ring in runs that store C straight from registers
                              (no staging buffers: beta == 0 and C, ldc and N multiples of 32 bytes);
                              0 if the plan always stages (EXO_GEMM_FLAG_EPI_BUFFERS given)        */
  int32_t lean_kernel;     /* 1: the one-tile-per-CTA kernel runs this plan (EXO_GEMM_FLAG2_LEAN_*): grid =
                              tiles_m * tiles_n CTAs at once, one accumulator, `stages` = its ring         */
  int32_t repacked;        /* bit 0 = A, 1 = B, 2 = C: the matrix's leading dimension times its element size is not a
                              multiple of 16 bytes, so every run copies it through an aligned buffer the plan owns
                              (counted in workspace_bytes)                                                    */
} exo_gemm_info_t;

/*
 * Pure argument check; needs no GPU and touches no CUDA state.  Returns OK,
 * ERR_NULL, ERR_INVALID_ARG or ERR_UNSUPPORTED by the rules above.  (What is legal
 * follows BLAS Sgemm, the routine the paper's Section 6 measures its GEMM kernels
 * against; what is supported is that set cut down to what TMA can address.)
 */
exo_gemm_status_t exo_gemm_validate(const exo_gemm_desc_t* desc);

/*
 * Builds a plan for one problem descriptor: validates, canonicalises
 * (column-major C becomes the transposed product), picks the tile shape, the
 * cta_group, the pipeline depth and the raster, and sizes the persistent grid
 * (the paper's counterpart is the device-function configuration of Section 3.2,
 * clusterDim and warp configuration, and the persistent task loop of
 * Section 4.2).  Allocates host state, one 32-byte device status block and, if the
 * tiles of a partial last wave are to be cut along K (exo_gemm_info_t.split_k > 1),
 * a device workspace of exo_gemm_info_t.workspace_bytes for their partial sums, one
 * arrival counter per such tile and a 64-byte-per-worker table of who computes what;
 * touches no user matrix.  *out is written only on success.
 */
exo_gemm_status_t exo_gemm_create(exo_gemm_handle_t* out, const exo_gemm_desc_t* desc);

/*
 * Strided-batched variant (the paper's Section 6 also measures batched GEMM, against
 * cublasSgemmStridedBatched): `batch_count` independent products
 * C_i = alpha*A_i*B_i + beta*C_i, i = 0 .. batch_count-1, where matrix i of each operand
 * starts stride_x ELEMENTS after matrix i-1 and every matrix has the descriptor's
 * shape, layout and leading dimension.  One persistent launch covers the whole
 * batch (the batch index is the third coordinate of the TMA tensor maps and part of
 * the tile index).  stride_a or stride_b may be 0 (that operand is shared by all
 * products); the C matrices must not overlap (stride_c >= the extent of one C,
 * else ERR_INVALID_ARG); each stride times its element size must be a multiple of
 * 16 bytes (else ERR_UNSUPPORTED); 1 <= batch_count <= 65535.  exo_gemm_run then
 * takes the base pointers of matrix 0.  batch_count == 1 is exo_gemm_create.
 */
exo_gemm_status_t exo_gemm_create_batched(exo_gemm_handle_t* out, const exo_gemm_desc_t* desc, int64_t batch_count,
                                          int64_t stride_a, int64_t stride_b, int64_t stride_c);

/*
 * Enqueues C = alpha*A*B + beta*C on cuda_stream (a cudaStream_t; NULL = the
 * legacy default stream) and returns without synchronising.  This is the operation
 * of the paper's GEMM kernels (Section 6; "D += matmul(A, B)" in the Section 2.2
 * listings) with the alpha/beta form of BLAS Sgemm; one call is one launch of a
 * persistent, warp-specialised kernel (the kernel class of the paper's Section 4.2
 * code generation: persistent task loop, one code path per named warp group).
 *
 *   A, B, C   DEVICE pointers, 16-byte aligned (element-aligned for a matrix the plan
 *             repacks, see the descriptor), laid out as the descriptor says.
 *             The caller owns them and keeps them alive until the stream has
 *             passed the kernel.  C is updated in place; A and B must not
 *             overlap C.  The library never allocates, frees or copies them.
 *   alpha, beta   host floats.  beta == 0: C is never read (NaN/Inf or
 *             uninitialised memory in C do not propagate).  alpha == 0 or K == 0:
 *             A and B are not read and C = beta*C.
 *   M == 0 or N == 0: returns OK without launching.
 *
 * The result is alpha*acc + beta*C_in evaluated in fp32, where acc is the fp32
 * tensor-core accumulation over k, then rounded to nearest-even into c_dtype.
 * For a fixed plan the result is bitwise reproducible from run to run.
 *
 * All checks happen before the launch; on any error nothing is enqueued.  A
 * handle may be used from several host threads (tensor maps are built on the
 * caller's stack), but runs of ONE plan whose exo_gemm_info_t.split_k > 1 or
 * .repacked != 0 must not overlap on the GPU (enqueue them on one stream, or order the
 * streams): they share the plan's partial-sum workspace and arrival counters, or its
 * aligned copies.  Nothing in a launch's parameters depends
 * on how often the plan has run (the counters of a K-slicing plan keep their own run count on the device),
 * so exo_gemm_run may be captured into a CUDA graph and the graph replayed.  Device-side waits are bounded: if one gives up, the kernel
 * records where in the plan's status block and exits cleanly; a later
 * exo_gemm_check reports EXO_GEMM_ERR_DEVICE_TIMEOUT.
 */
exo_gemm_status_t exo_gemm_run(exo_gemm_handle_t plan, const void* A, const void* B, void* C,
                               float alpha, float beta, void* cuda_stream);

/*
 * Reads the plan's device status block (a blocking 32-byte device-to-host copy on the
 * legacy default stream; call it after synchronising the stream(s) the plan ran on).
 * Returns OK or ERR_DEVICE_TIMEOUT, and clears the block.  detail, if not NULL, receives 8
 * words: {code, role, barrier, tile, k_block, cta, 0, 0}.  After a timeout it also puts
 * the counters of a K-slicing plan back to zero (an abandoned run leaves them out of
 * step), so call it while no run of the plan is in flight.  (The paper's kernels have no such
 * status: its Section 5 checks synchronisation before the kernel ever runs; a library
 * that runs on shared GPUs bounds every device-side wait instead and reports here.)
 */
exo_gemm_status_t exo_gemm_check(exo_gemm_handle_t plan, uint32_t* detail);

/*
 * What exo_gemm_create would choose for `desc` on a device with `sm_count` SMs
 * (all of them pairable).  Pure; needs no GPU.  Same status codes as
 * exo_gemm_validate, plus ERR_NULL for info == NULL.
 */
exo_gemm_status_t exo_gemm_plan_preview(const exo_gemm_desc_t* desc, int32_t sm_count, exo_gemm_info_t* info);

/* Reports what the plan chose. */
exo_gemm_status_t exo_gemm_get_info(exo_gemm_handle_t plan, exo_gemm_info_t* info);

/*
 * The same GEMM for callers that must not allocate device memory.  (The paper has
 * no counterpart; this is a library convenience.)  Who needs it: code running
 * where cudaMalloc is off limits or fails by design -- a process whose device
 * memory is entirely owned by a framework's pool, a real-time loop that may not
 * take the allocator's lock or its latency, a plug-in that is forbidden to
 * allocate after initialisation.  exo_gemm_create calls cudaMalloc for the plan's
 * 32-byte status block; this entry point needs no plan and calls no cudaMalloc,
 * cudaFree or other allocating routine: it plans on the host stack and keeps the
 * status block in a 256-byte device array that is part of the library image
 * (every GPU that loads the library holds those 256 bytes until exit).
 *
 *   desc, A, B, C, alpha, beta, cuda_stream   as for exo_gemm_create + exo_gemm_run;
 *             the caller still owns and passes all inputs and outputs.
 *   detail    NULL: asynchronous, like exo_gemm_run.  Not NULL (host pointer to 8
 *             words): the call waits for the stream, copies the status words there
 *             and returns EXO_GEMM_ERR_DEVICE_TIMEOUT if a device-side wait gave up.
 *
 * Limit: the scratch a launch needs must fit the 256-byte array.  The status block
 * is 32 bytes for every problem size, so every supported problem fits; a build
 * whose status block is larger (the development trace build) is refused with
 * EXO_GEMM_ERR_UNSUPPORTED.  Devices with ordinal >= 64 are refused the same way.
 *
 * The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress, once per device); make that first call before any
 * stream capture.  All calls on a device share the one array, which keeps the last
 * call's contents: each call clears the status words on cuda_stream before its
 * kernel, so calls must not overlap on the GPU (two streams, or a plan-less call
 * racing another) -- overlapping calls race on the status words.  Each call repeats
 * the planning work of exo_gemm_create (a few attribute queries), so it costs a few
 * microseconds more of host time than exo_gemm_run on a kept plan.
 */
exo_gemm_status_t exo_gemm_run_static(const exo_gemm_desc_t* desc, const void* A, const void* B, void* C,
                                      float alpha, float beta, void* cuda_stream, uint32_t* detail);

/*
 * fp32 matrix-vector product y = alpha*A*x + beta*y, A an M x N row-major matrix with
 * leading dimension lda >= N (elements): the paper's second workload (Section 6: a
 * full-precision GEMV from warp shuffles and scalar math, memory-bound, roofline
 * 2 FLOP per 4 bytes of A).  A, x, y are DEVICE pointers owned by the caller; y is
 * updated in place; x and A must not overlap y.  beta == 0: y is not read;
 * alpha == 0: A and x are not read.  Enqueued on cuda_stream (current device),
 * returns without synchronising; nothing is allocated.  128-bit loads are used when
 * A and x are 16-byte aligned and lda % 4 == 0, scalar loads otherwise.  Products
 * are accumulated in fp32 (one warp per row, lanes interleaved over the row, then a
 * shuffle tree).  Errors: ERR_INVALID_ARG (negative size, lda < N), ERR_NULL,
 * ERR_ARCH, ERR_CUDA.
 */
exo_gemm_status_t exo_gemv_run(int64_t M, int64_t N, const float* A, int64_t lda, const float* x, float* y,
                               float alpha, float beta, void* cuda_stream);

/*
 * The same product for a COLUMN-major A (M contiguous, leading dimension lda >= M), the other
 * storage order BLAS Sgemv takes.  A lane owns consecutive rows, so every warp load of a
 * column is contiguous; the columns are split over the warps of a CTA and over the CTAs of
 * a thread-block cluster, and the partial sums are added through shared and distributed
 * shared memory in warp and CTA order (the result does not depend on timing).  128-bit
 * loads when A is 16-byte aligned, lda % 4 == 0 and M >= 128; scalar loads otherwise.  Same argument
 * rules, ownership and errors as exo_gemv_run (ERR_INVALID_ARG for lda < M; ERR_UNSUPPORTED
 * if M needs 2^31 or more CTAs).
 */
exo_gemm_status_t exo_gemv_run_colmajor(int64_t M, int64_t N, const float* A, int64_t lda, const float* x, float* y,
                                        float alpha, float beta, void* cuda_stream);

/* Frees the plan and its device status block.  NULL is a no-op returning OK. */
exo_gemm_status_t exo_gemm_destroy(exo_gemm_handle_t plan);

/* Static string for a status code. */
const char* exo_gemm_status_string(exo_gemm_status_t status);

/* The CUDA error code (cudaError_t / CUresult as int) behind the last ERR_CUDA of this thread. */
int exo_gemm_last_cuda_error(void);

/*
 * Host-side enumeration of the persistent tile schedule (Section 4.2 of the
 * paper distributes tasks round-robin in lexicographic order and names a
 * swizzled order as future work; this library uses a band-swizzled raster).
 * Writes the (tile_m, tile_n) indices that worker `worker` of `num_workers`
 * visits, in order, into out_m/out_n (capacity `cap`), and returns how many it
 * visits (which may exceed cap), or -1 on bad arguments.  Needs no GPU; it
 * compiles the same function the kernel uses.
 */
int64_t exo_gemm_schedule_enumerate(int32_t tiles_m, int32_t tiles_n, int32_t band, int32_t along_m,
                                    int32_t num_workers, int32_t worker, int32_t* out_m,
                                    int32_t* out_n, int64_t cap);

/*
 * Host-side enumeration of one worker's work list including the K-slicing of the
 * tail tiles (the paper's Section 6 measures split-K variants of its GEMM against
 * wave quantisation; here only the tiles of the partial last wave are cut: their
 * k-blocks, in tile-major order, are shared out among `tail_workers` workers in equal
 * consecutive ranges, so a range may cover the end of one tile and the beginning of
 * the next; the part of a tile that starts at k-block 0 is slice 0 and owns the
 * output, the other parts contribute partial sums in K order).  The items come in the
 * order the worker executes them: a contributing part (slice > 0) before the worker's
 * whole tiles, an owning part after them, so that the partial sums are in memory
 * before the owner needs them.  `tiles` tiles, `num_workers` workers; tail_workers ==
 * 0 leaves the tail tiles whole.  A range boundary within `snap` k-blocks of a tile
 * boundary is moved onto it (parts of a few k-blocks are not worth an exchange; at
 * most num_k_blocks / 8).  Where tail_workers is a multiple f of the tail tile count, every
 * tail tile is instead cut into f slices at the same k-blocks, slice s of tail tile t goes to
 * worker s * tail_tiles + t, and slice 0 takes `owner_extra` k-blocks more than an even
 * share.  Writes tile index, slice, slices (parts the tile is
 * cut into; 1 = whole) and k-block range [begin, end) of `num_k_blocks` per item
 * (capacity `cap`); returns the item count, or -1 on bad arguments (including
 * tail_workers below the tail tile count, above num_workers, or above the tail's
 * k-block count).  Needs no GPU.
 */
int64_t exo_gemm_schedule_work(int64_t tiles, int32_t num_workers, int32_t tail_workers, int32_t num_k_blocks, int32_t snap,
                               int32_t owner_extra, int32_t worker, int64_t* out_tile, int32_t* out_slice, int32_t* out_slices,
                               int32_t* out_kb_begin, int32_t* out_kb_end, int64_t cap);

/*
 * Test hook for the bounded waits: the next exo_gemm_run on this plan uses
 * `timeout_ms` as the device-side wait limit and, if skip_k_block >= 0, its
 * first CTA's producer skips issuing the loads of that k-block (counted from the
 * start of the CTA's work), so that one wait runs out and the kernel returns an
 * error status without trapping.  The settings apply to one run, then reset.
 * plan == NULL: the settings apply to the next exo_gemm_run_static call of this
 * process instead (that entry point has no plan to attach them to).
 */
exo_gemm_status_t exo_gemm_debug_set(exo_gemm_handle_t plan, int32_t timeout_ms, int64_t skip_k_block);

/*
 * 1 if this build of the library contains the shared-operand cluster variant
 * (EXO_GEMM_FLAG2_SHARE_*), else 0.  The variant is compiled into a separate
 * library file; programs that span several GPUs use the base library.
 */
int32_t exo_gemm_has_shared_operand_clusters(void);

#ifdef __cplusplus
}
#endif
#endif /* EXO_GEMM_H_ */
