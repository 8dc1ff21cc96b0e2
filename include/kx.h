/*
 * kx — BF16 attention output projection with residual addition on B200 (sm_100a).
 *
 *     Y[M,N] = X[M,K] . W[N,K]^T  (+ bias[N])  + R[M,N]        (kx_outproj_residual)
 *     Y[M,N] = X[M,K] . W[N,K]^T                                (kx_gemm_bf16)
 *
 * Operation: the residual GEMM epilogue of the paper's Appendix A ("L1-030:
 * attention output projection with residual", Algorithm 3: the destination is
 * aliased onto the residual and O <- W^T A + O with alpha = beta = 1), written
 * row-major; the optional bias is an extension of this library.  The plain
 * product is the operation of the paper's fixed-shape GEMM study (Section 4.1).
 *
 * All tensors are dense row-major BF16 (leading dimension = row length):
 *   X [M,K], W [N,K] (the nn.Linear layout, K contiguous), bias [N] or NULL,
 *   R [M,N], Y [M,N].  Products are accumulated in FP32; bias and residual are
 *   added in FP32 and the sum is rounded to BF16 once (round-to-nearest-even).
 *
 * Pointers are DEVICE pointers unless an entry point's name ends in `_host`.
 * The caller owns every tensor before, during and after the call; the library
 * never frees, reallocates or keeps a reference to tensor contents (it keeps
 * only encoded TMA descriptors keyed on address and shape).  Calls enqueue
 * work on the caller's stream and return without synchronising.
 *
 * Preconditions (checked; a violated one returns an error and enqueues nothing):
 *   - X, W, R, Y non-NULL (unless the matching extent is zero) and 16-byte aligned;
 *     bias NULL or 16-byte aligned;
 *   - M, N, K >= 0; N % 8 == 0 and K % 8 == 0 (16-byte row pitch for TMA);
 *   - Y may be exactly R (in place, the paper's aliasing); any other overlap of
 *     Y with X, W, bias or R is rejected;
 *   - the current device has compute capability 10.x.
 *   M == 0 or N == 0 is a successful no-op.  K == 0 gives Y = R (+ bias).
 *
 * There is no CPU fallback and no vendor-library GEMM behind these calls.
 */
#ifndef KX_H_
#define KX_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KX_VERSION 100

typedef enum kx_status {
    KX_OK = 0,
    KX_ERR_NULL = 1,            /* a required pointer is NULL                         */
    KX_ERR_SHAPE = 2,           /* negative extent, N or K not a multiple of 8, ...   */
    KX_ERR_ALIGN = 3,           /* a pointer is not 16-byte aligned                   */
    KX_ERR_OVERLAP = 4,         /* Y overlaps an input other than Y == R              */
    KX_ERR_ARCH = 5,            /* current device is not sm_100                       */
    KX_ERR_CUDA = 6,            /* a CUDA runtime/driver call failed                  */
    KX_ERR_WORKSPACE = 7,       /* split-K workspace too small / allocation failed    */
    KX_ERR_DEVICE_TIMEOUT = 8,  /* a bounded device-side wait gave up (see below)     */
    KX_ERR_PLAN = 9,            /* plan override names an unsupported configuration   */
    KX_ERR_LIMIT = 10           /* shape beyond kx_outproj_residual_noalloc's fixed scratch */
} kx_status;

/* Execution paths (the scheduling strategy of Table 1 names split-K and
 * persistent kernels; the per-M specialisation follows Algorithm 3's per-M plan). */
enum { KX_PATH_AUTO = 0, KX_PATH_TILE = 1, KX_PATH_SWAP = 2, KX_PATH_GEMV = 3, KX_PATH_SKINNY = 4 };

/*
 * Plan override for tests, profiling and tuning.  Zero-initialise for "auto".
 *   path          KX_PATH_AUTO / KX_PATH_TILE (128-row output tiles, persistent,
 *                 TMA-store epilogue) / KX_PATH_SWAP (small M: W rows on the MMA
 *                 M axis, split-K, W streamed once) / KX_PATH_GEMV (M <= 4 and K % 8 == 0:
 *                 no tensor core, every CTA streams a few rows of W and reduces over K with
 *                 FP32 warp reductions) / KX_PATH_SKINNY (M <= 32 and K % 8 == 0: the same streaming
 *                 organisation with warp-level tensor-core instructions fed from registers, K shared by
 *                 the 16 warps of a CTA and reduced in its shared memory)
 *   block_n       tile path: 64, 128, 192 or 256 output columns per tile;
 *                 swap path: 16, 32, 64, 128 or 256 X rows per unit;
 *                 GEMV path: 1, 2 or 4 rows of W (output columns) per CTA;
 *                 skinny path: 16 or 32 rows of W per CTA
 *   cta_pair      0 auto, 1 = one CTA per tile, 2 = CTA pair per 256-row tile
 *   split_k       swap path: number of K splits (1..64);
 *                 GEMV path: 1..16 warps per CTA that share the K range of its rows
 *   raster_group  tile path: number of 128-row tile rows that share a raster group
 *   max_ctas      cap on the persistent grid (0 = number of SMs)
 *   spin_limit_us bound on every device-side wait (0 = 2 000 000 us)
 *   stages        pick the kernel variant with this ring depth (0 = default); variants whose stages
 *                 hold two k-blocks have their own (smaller) stage counts
 *   stream_k      tile path: 0 auto, 1 = whole tiles per CTA (round-robin), 2 = stream-K
 *                 (every CTA gets an equal contiguous range of (tile, k-block) units;
 *                 split tiles are summed in the FP32 workspace in a fixed order), 3 = the tiles
 *                 left over after the full waves are split that way and run FIRST, the rest whole
 *                 (the summing of a split tile then overlaps the next tile's main loop)
 *   narrow_tail   tile path: 0 auto, 1 off, 2 = run the tiles left over after the full
 *                 waves as half-width tiles when they then fit in one extra wave, 3 = run each
 *                 of them as two K halves on two CTAs (CTA pairs) at full width instead; the two
 *                 swap, through the FP32 workspace, the 64-column chunks the other one finishes
 *                 (needs at most half as many leftover tiles as CTAs / pairs, else KX_ERR_PLAN)
 *   cluster_reduce  swap path: 0 auto, 1 = sum the K splits through the FP32 workspace
 *                 (last CTA to arrive reduces), 2 = the 2..8 splits of a tile form a
 *                 thread-block cluster and the CTA that finishes a row reads the partials of
 *                 its peers through distributed shared memory, 3 = the same cluster, but every
 *                 CTA stores its partial rows into the shared memory of their finishers and
 *                 signals an mbarrier there (X rows per unit <= 128)
 *   k_cluster     tile path, one CTA per tile: 2 or 4 = split the K range of every tile over a
 *                 thread-block cluster of that many CTAs and sum the partial tiles through
 *                 distributed shared memory (for problems with too few tiles to fill the GPU)
 *   l2_prefetch   number of leading k-blocks of its first work item whose operand tiles a CTA asks
 *                 to be brought into L2 before it waits for the previous kernel in the stream
 *                 (0 = the ring depth, -1 = none).  L2 is the device's coherence point, so a
 *                 tile requested early still shows every later device write when it is loaded.
 *   no_table      1 = ignore the built-in measured plan table and use the heuristic
 *                 (the table is consulted only when no plan field above is set)
 *   no_pdl        1 = launch without programmatic stream serialization (by default the
 *                 kernel's prologue may overlap the tail of the previous kernel in the
 *                 stream; it waits for that kernel before its first global access)
 *   debug_drop_kblocks  test hook: the TMA producer issues this many fewer
 *                 k-blocks than the MMA consumer expects, so the consumer's
 *                 bounded wait expires and the call reports
 *                 KX_ERR_DEVICE_TIMEOUT through kx_last_device_status.  The
 *                 kernel still exits cleanly.  Never set in production.
 */
typedef struct kx_plan_override {
    int32_t path;
    int32_t block_n;
    int32_t cta_pair;
    int32_t split_k;
    int32_t raster_group;
    int32_t max_ctas;
    int32_t spin_limit_us;
    int32_t debug_drop_kblocks;
    int32_t stages;
    int32_t stream_k;
    int32_t narrow_tail;
    int32_t no_pdl;
    int32_t cluster_reduce;
    int32_t no_table;
    int32_t k_cluster;
    int32_t l2_prefetch;
} kx_plan_override;

/* What the planner chose for a shape (kx_plan_query). */
typedef struct kx_plan_info {
    int32_t path;          /* KX_PATH_TILE, KX_PATH_SWAP, KX_PATH_GEMV or KX_PATH_SKINNY */
    int32_t block_n;
    int32_t cta_pair;      /* 1 or 2                                               */
    int32_t stages;        /* depth of the TMA -> MMA shared-memory ring           */
    int32_t split_k;
    int32_t raster_group;
    int32_t grid;          /* CTAs launched                                        */
    int32_t tiles;         /* work units (tiles x splits)                          */
    int32_t launches;      /* kernels enqueued per call                            */
    int32_t smem_bytes;    /* dynamic shared memory per CTA                        */
    int64_t workspace_bytes; /* FP32 split-K / stream-K scratch this plan uses (0 if none) */
    int32_t stream_k;      /* tile path: 1 = stream-K over the last waves, 2 = over the leftover tiles, first */
    int32_t narrow_tiles;  /* number of half-width tail tiles (0 if none)          */
    int32_t cluster_reduce;/* swap path: 0 = workspace, 1 = cluster (partials pulled), 2 = cluster (partials pushed) */
    int32_t from_table;    /* 1 if the built-in measured plan table supplied this plan */
} kx_plan_info;

/*
 * Optional.  Creates the per-device state for `device` (SM count, kernel
 * attributes, the split-K workspace and its counters) so that later calls do
 * no allocation.  Idempotent, thread-safe.  Without it, the first kx_* call on
 * a device does the same lazily (so make that first call outside stream capture).
 *
 * Shared state and concurrency.  Each device has ONE FP32 workspace, one array of tile counters and
 * one status word, shared by every stream and host thread.  Calls whose plan uses the workspace
 * (kx_plan_info.workspace_bytes > 0: split-K through the workspace, i.e. more than 8 splits, a capped
 * grid or cluster_reduce = 1, stream-K, and the K-halves tail) must not overlap on the GPU with one
 * another: order them on one stream or with events, as for kx_outproj_residual_noalloc's built-in
 * scratch.  The heuristic plans of kx_outproj_residual / kx_gemm_bf16 / _strided / _batched use no
 * workspace (cluster reductions and whole tiles) with ONE exception: large-M BF16 shapes with K >= 4096
 * whose tiles do not fill the last wave (at most half of it) take the K-halves tail, which does (the
 * 4096^3 projection is one).  kx_plan_query tells (workspace_bytes), also for an entry of the built-in
 * measured plan table; a caller that must overlap such calls passes narrow_tail = 2 (or 1) through
 * kx_outproj_residual_ex and gets the workspace-free plan.  kx_outproj_residual_host also owns
 * one staging buffer and one set of copy streams per device: its calls must not overlap each other.
 * Host-side entry is thread-safe (the per-device state is built once under a lock; descriptor caches
 * are per thread).
 */
int kx_init(int device);

/* Frees library-owned memory on every initialised device.  Never touches caller tensors. */
int kx_shutdown(void);

/*
 * Y = X W^T (+ bias) + R.   Appendix A, Algorithm 3 (alpha = beta = 1, C = D).
 *   X [M,K], W [N,K], bias_or_null [N], R [M,N] (may equal Y), Y [M,N]: device, BF16.
 *   stream: a cudaStream_t passed as void* (NULL = the legacy default stream).
 * Returns a kx_status.  Asynchronous: errors raised by the kernel itself are
 * visible through kx_last_device_status after the stream has drained.
 */
int kx_outproj_residual(const void* X, const void* W, const void* bias_or_null, const void* R,
                        void* Y, int64_t M, int64_t N, int64_t K, void* stream);

/* Y = X W^T.   Section 4.1's BF16 matrix product (FLOPs counted as 2 M N K). */
int kx_gemm_bf16(const void* X, const void* W, void* Y, int64_t M, int64_t N, int64_t K, void* stream);

/*
 * Same as kx_outproj_residual (R and bias may both be NULL: plain GEMM) with an
 * explicit plan.  `ov` may be NULL (= auto).  Unsupported combinations return
 * KX_ERR_PLAN.
 */
int kx_outproj_residual_ex(const void* X, const void* W, const void* bias_or_null, const void* R,
                           void* Y, int64_t M, int64_t N, int64_t K, void* stream,
                           const kx_plan_override* ov);

/*
 * Host-buffer convenience form of kx_outproj_residual: every tensor pointer is a
 * HOST pointer (pinned memory gives the best copy rate; pageable works).  The
 * call copies X, W, bias, R to library-owned device staging buffers (grown on
 * demand, kept until kx_shutdown), runs the kernel, copies Y back into Y_host
 * and synchronises `stream` before returning.  For M >= 2048 the rows are cut
 * into four slices and copy-in, compute and copy-out of consecutive slices
 * overlap on three streams (two of them library-owned).  R_host and bias_host may be NULL.
 * Not for use under stream capture (it may allocate and it synchronises).
 */
int kx_outproj_residual_host(const void* X_host, const void* W_host, const void* bias_host_or_null,
                             const void* R_host_or_null, void* Y_host,
                             int64_t M, int64_t N, int64_t K, void* stream);

/*
 * Y = X W^T (+ bias) (+ R) for small M without any allocation, ever.  (The paper has no
 * counterpart for this entry point; it exists for the sake of callers, not of the method.)
 *
 * Who needs it: code that must not ask the driver for device memory.  Examples are a
 * serving process whose framework grabbed all of HBM for its own pool at start-up (a
 * cudaMalloc from a library would fail or fragment that pool), a latency-critical loop
 * that cannot tolerate the device-wide synchronisation a cudaMalloc / cudaFree may
 * imply, and plug-ins whose host forbids allocation from worker threads.  The other
 * entry points allocate their split-K workspace in kx_init or on first use; this one
 * calls no cudaMalloc, no cudaFree and no routine that allocates on its behalf.
 *
 * How: it always runs the small-M split-K kernel, and the kernel's scratch (FP32 partial
 * sums plus per-tile arrival counters) is a fixed array of 8 MiB + 16 KiB built into the
 * library's device image.  Every GPU that loads the library carries that array until the
 * process exits.
 *
 * Arguments, layout and preconditions are those of kx_outproj_residual_ex with a NULL
 * plan (bias and R may each be NULL; Y may equal R).  Limits: M <= 256 and
 * N <= 524288 (4096 column tiles); anything larger returns KX_ERR_LIMIT and enqueues
 * nothing.  The split count shrinks as needed so that the partial sums fit in 8 MiB.
 *
 * The first call on each device looks up the array's device address and sets kernel
 * attributes (no allocation); make that first call with the device current and before
 * any stream capture begins.  All calls share the one array and it keeps the previous
 * call's contents: the entry point zeroes the counters on `stream` before each launch,
 * and partial sums are rewritten before they are read.  Two calls that run on the GPU at
 * the same time (different streams, or different host threads on one device) would race
 * on the array: order them on one stream or with events.
 *
 * Errors raised by the kernel itself (a bounded wait that gave up) are read with
 * kx_last_device_status, which allocates nothing either.  Two environment variables, read once at
 * the first call on a device, exist for tests only: KX_NOALLOC_SPIN_US (bound on device-side waits,
 * default 2 000 000) and KX_NOALLOC_DEBUG_DROP (the loader withholds that many stages, so a wait
 * runs out and the call reports KX_ERR_DEVICE_TIMEOUT; the kernel still exits cleanly).
 */
int kx_outproj_residual_noalloc(const void* X, const void* W, const void* bias_or_null,
                                const void* R_or_null, void* Y, int64_t M, int64_t N, int64_t K,
                                void* stream);

/*
 * Z = RMSNorm(H) * gamma, row by row:  z[m,n] = h[m,n] / sqrt(mean_j h[m,j]^2 + eps) * gamma[n].
 * The step that follows the output projection and first residual in the paper's
 * decoder-layer case study (Appendix A, Algorithm 7, "run fused add+RMSNorm ..."); the paper
 * prints no formula, so this is the textbook definition, with the statistics taken from the
 * BF16 values of H, the arithmetic in FP32 and one rounding to BF16.
 *   H [M,N], gamma [N], Z [M,N]: device, BF16, 16-byte aligned; eps >= 0.
 *   N % 8 == 0 and N <= 32768 (a row is held in one CTA's registers); Z may equal H.
 * One memory-bound kernel (each row read once, written once) on `stream`.
 */
int kx_rmsnorm(const void* H, const void* gamma, float eps, void* Z, int64_t M, int64_t N, void* stream);

/*
 * H = X W^T (+ bias) + R, then Z = RMSNorm(H) * gamma: both outputs of the attention block's
 * tail (the new residual stream H and the normalised input Z of the MLP).  Algorithm 3 followed
 * by the RMSNorm step of Algorithm 7.  Two kernels on `stream`, the second launched with
 * programmatic stream serialization so that its prologue overlaps the first one's tail; for
 * outputs up to the size of the L2 cache the second kernel reads H from L2.
 * Arguments as for kx_outproj_residual and kx_rmsnorm.  H may equal R (in place); Z must not
 * overlap any other tensor.
 */
int kx_outproj_residual_rmsnorm(const void* X, const void* W, const void* bias_or_null, const void* R,
                                const void* gamma, float eps, void* H, void* Z,
                                int64_t M, int64_t N, int64_t K, void* stream);

/*
 * Z[M,I] = silu(X Wg^T) * (X Wu^T): the gate and up projections of the MLP with the SwiGLU
 * product fused into the GEMM epilogue (the paper's decoder-layer case study, Appendix A,
 * Algorithm 7: "compute ... gate/up projections" with a "SwiGLU epilogue"; silu(t) = t / (1 + e^-t)).
 *   X [M,K], Wg [I,K], Wu [I,K], Z [M,I]: device, BF16 row-major, 16-byte aligned;
 *   I % 8 == 0, K % 8 == 0; Z must not overlap an input.  FP32 accumulation, activation and
 *   product in FP32, one rounding to BF16.
 * One launch of the large-M tile kernel: each tile accumulates 128 gate and the matching 128 up
 * columns side by side in tensor memory (in a CTA pair one CTA streams Wg, the other Wu), so
 * neither pre-activation ever leaves the chip.  FLOPs = 4 M I K.
 */
int kx_gate_up_swiglu(const void* X, const void* Wg, const void* Wu, void* Z,
                      int64_t M, int64_t I, int64_t K, void* stream);

/*
 * kx_outproj_residual on row-pitched operands: row r of X starts at X + r * ldx elements, and
 * likewise W (ldw), R (ldr), Y (ldy) -- slices of wider buffers (one head group of a fused
 * projection, a window of a ring buffer, a padded allocation) without a packing copy.  Algorithm 3
 * prints the dense case only; the pitches map directly onto the tensor-map row strides, so the
 * kernels and plans are the dense ones.
 *   ldx, ldw >= K; ldy >= N; ldr >= N (ignored when R is NULL); every pitch % 8 == 0 (rows stay
 *   16-byte aligned); base pointers 16-byte aligned.  K and N may be ANY length here (the tail of
 *   the last k-block reads as zeros, the last output columns are clipped), which covers shapes
 *   that are not multiples of 8 once the rows are padded to one.  A ragged N (N % 8 != 0) always
 *   runs the large-M tile kernel, also for small M.
 *   R may equal Y only with ldr == ldy; any other overlap between the spans of Y and an input is
 *   KX_ERR_OVERLAP.  Elements between N and ldy of a Y row are never written when N % 8 == 0;
 *   otherwise the padding up to the next multiple of 8 (the rest of the last 16-byte unit) is
 *   overwritten, nothing beyond it.
 */
int kx_outproj_residual_strided(const void* X, int64_t ldx, const void* W, int64_t ldw,
                                const void* bias_or_null, const void* R_or_null, int64_t ldr,
                                void* Y, int64_t ldy, int64_t M, int64_t N, int64_t K, void* stream);

/*
 * `batch` independent problems of the same shape, dense operands: problem b uses X + b*sx,
 * W + b*sw, bias + b*sb, R + b*sr, Y + b*sy (strides in elements; sw = 0 shares one weight matrix,
 * sb = 0 one bias; bias / R may be NULL for all).  Enqueues one kx_outproj_residual per problem on
 * `stream`, back to back with programmatic dependent launch (each prologue overlaps its
 * predecessor's tail): a convenience for a handful of large problems (per-expert or per-group
 * projections), not a grouped kernel for many tiny ones.  Every stride must keep the 16-byte
 * alignment (multiple of 8); the Y blocks must not overlap each other or an input.  The paper has
 * no batched case; this is the plain generalisation of Algorithm 3's call.
 */
int kx_outproj_residual_batched(const void* X, int64_t sx, const void* W, int64_t sw,
                                const void* bias_or_null, int64_t sb, const void* R_or_null, int64_t sr,
                                void* Y, int64_t sy, int64_t M, int64_t N, int64_t K, int64_t batch,
                                void* stream);

/*
 * ---- INT8 branch of the decoder layer (Appendix A, Algorithm 7: "run fused add+RMSNorm+
 * activation quantization", "quantize gate/up weights in one launch", "compute gate/up GEMM with
 * fused dequantization and SwiGLU epilogue"; the residual add is already part of
 * kx_outproj_residual).  The paper does not print the code book; this library uses the usual
 * symmetric one, per row (per token for activations, per output channel for weights):
 *     a = max_j |z_j|,  scale = a / 127,  q_j = clamp(rint(z_j * (127 / a)), -127, 127)
 * every operation in binary32 (two correctly rounded divisions per row, one product and one
 * round-half-to-even per element); a row of zeros gets scale 1 and codes 0.  Rows holding a NaN
 * or an infinity give unspecified codes.
 *
 * All pointers are device pointers; codes are int8 row-major, scales FP32; matrices 16-byte
 * aligned, scale vectors 16-byte aligned (the row scales of X only need 4); cols / K % 16 == 0
 * (a row of codes is a whole number of 16-byte units), cols <= 32768 for the quantising calls.
 * Work is enqueued on `stream`; errors are returned as for the other entry points.
 */

/* Q[rows,cols], S[rows] = code book of the BF16 matrix A[rows,cols].  Q and S must not overlap A
 * or each other.  One launch, HBM-bound: 3 bytes per element. */
int kx_quantize_rows_int8(const void* A, void* Q, float* S, int64_t rows, int64_t cols, void* stream);

/* The same for the gate and the up weight matrices [I,K] in ONE launch (rows 0..I-1 of the grid
 * take Wg, the rest Wu). */
int kx_quantize_gate_up_int8(const void* Wg, const void* Wu, void* Qg, float* Sg, void* Qu, float* Su,
                             int64_t I, int64_t K, void* stream);

/* Q, S = code book of z = RMSNorm(H) * gamma, where z is the BF16-rounded result kx_rmsnorm
 * would write (bit for bit) but never reaches memory: H [M,N] BF16 is read once (2 bytes per
 * element), Q [M,N] int8 and S [M] written (1 byte per element).  eps >= 0. */
int kx_rmsnorm_quantize_int8(const void* H, const void* gamma, float eps, void* Q, float* S,
                             int64_t M, int64_t N, void* stream);

/*
 * Z[M,I] = silu(g) * u with g = (Xq Wgq^T) sx[m] sg[i], u = (Xq Wuq^T) sx[m] su[i]: INT8 gate/up
 * GEMM (tcgen05 kind::i8, exact 32-bit integer accumulation in tensor memory) with the
 * dequantisation and the SwiGLU product in the epilogue (FP32), one rounding to BF16.
 *   Xq [M,K], Wgq / Wuq [I,K] int8; sx [M], sg / su [I] FP32; Z [M,I] BF16; I % 8 == 0.
 *   |sum| must stay below 2^31 (K <= 133 000 for full-range codes).  OPs = 4 M I K.
 */
int kx_gate_up_swiglu_int8(const void* Xq, const float* sx, const void* Wgq, const float* sg,
                           const void* Wuq, const float* su, void* Z,
                           int64_t M, int64_t I, int64_t K, void* stream);

/*
 * Y[M,N] = (Xq Wq^T) sx[m] sw[n] + bias[n] + R[m,n]: the output projection with residual on INT8
 * codes (the precision axis of the paper's strategy space, Section 3.2, applied to the operator
 * of Algorithm 3).  bias / R as for kx_outproj_residual (NULL = absent; R may equal Y).
 * Large-M tile kernel for every M (no small-M path).
 */
int kx_outproj_residual_int8(const void* Xq, const float* sx, const void* Wq, const float* sw,
                             const void* bias_or_null, const void* R_or_null, void* Y,
                             int64_t M, int64_t N, int64_t K, void* stream);

/*
 * ---- FP8 (E4M3) twins of the five INT8 entry points: the other 8-bit operand type of the
 * precision axis of the paper's strategy space (Section 3.2).  Codes are FP8 E4M3 bit patterns
 * (bias 7, no infinities, 0x7F / 0xFF = NaN, largest finite value 448), one byte each; the code
 * book is
 *     a = max_j |z_j|,  scale = a / 448,  q_j = e4m3(z_j * (448 / a))
 * in binary32, the conversion rounding to nearest (ties to even) and saturating at +-448.  The
 * GEMMs run tcgen05 kind::f8f6f4 with FP32 accumulation; everything else (layouts, alignment,
 * K % 16 == 0, scale vectors, epilogues, error codes) is as for the INT8 calls above.
 */
int kx_quantize_rows_fp8(const void* A, void* Q, float* S, int64_t rows, int64_t cols, void* stream);
int kx_quantize_gate_up_fp8(const void* Wg, const void* Wu, void* Qg, float* Sg, void* Qu, float* Su,
                            int64_t I, int64_t K, void* stream);
int kx_rmsnorm_quantize_fp8(const void* H, const void* gamma, float eps, void* Q, float* S,
                            int64_t M, int64_t N, void* stream);
int kx_gate_up_swiglu_fp8(const void* Xq, const float* sx, const void* Wgq, const float* sg,
                          const void* Wuq, const float* su, void* Z,
                          int64_t M, int64_t I, int64_t K, void* stream);
int kx_outproj_residual_fp8(const void* Xq, const float* sx, const void* Wq, const float* sw,
                            const void* bias_or_null, const void* R_or_null, void* Y,
                            int64_t M, int64_t N, int64_t K, void* stream);

/*
 * Block-scaled FP8 branch (the block-scaled member of the precision axis of Section 3.2; the
 * tensor-core kind is the block-scaled tcgen05 family that Section 4.3 names).  Elements are FP8
 * E4M3 codes; every 32 consecutive elements of a row share one power-of-two scale stored as an
 * E8M0 byte e (value 2^(e-127); 0xFF is NaN and must not appear).
 *
 * Code book (kx_quantize_rows_mxfp8), per block of 32 BF16 values z of a row:
 *     e = clamp(floor(log2 max|z|) - 8 + 127, 0, 254)   (an all-zero block takes e = 127)
 *     q = e4m3(z / 2^(e-127))                           (exact quotient; nearest, ties to even, saturating at +-448)
 * A [rows, cols] BF16 row-major, cols % 32 == 0, cols <= 32768; Q [rows, cols] bytes; all device
 * pointers, 16-byte aligned, written by the call (Q, SF) or only read (A); no overlap.
 * kx_rmsnorm_quantize_mxfp8 is the same code book of RMSNorm(H) * gamma (the step after the projection in
 * the decoder layer of Appendix A, Algorithm 7, with the block-scaled format): z is rounded to BF16
 * exactly as kx_rmsnorm would write it and never reaches memory; H [M, N], gamma [N] BF16, eps >= 0.
 *
 * Scale layout (SF of the code book, SFX / SFW of the projection): chunks of 512 bytes, one per
 * (128 rows, 128 elements of K), ordered [ceil(rows / 128)][ceil(cols / 128)]; inside a chunk the
 * scale of row r and 32-element block j sits at byte (r % 32) * 16 + (r % 128) / 32 * 4 + j % 4.
 * This is the order in which the tensor core's scale copy (32 rows x 16 bytes, repeated for each
 * 32-lane quarter of tensor memory) wants them, so a chunk goes from global to shared to tensor
 * memory without being touched.  kx_mx_scale_bytes gives the size of the whole array (< 0 on
 * negative extents).  Entries of rows >= rows or blocks >= cols / 32 are padding: the code book
 * writes 127 there; arrays built elsewhere must hold any byte other than 0xFF.
 *
 * kx_outproj_residual_mxfp8:
 *     Y[m,n] = bf16( sum_j 2^(ex[m,j]-127) 2^(ew[n,j]-127) sum_{k in block j} xq[m,k] wq[n,k] + bias[n] + R[m,n] )
 * Xq [M,K], Wq [N,K] E4M3 bytes, K contiguous; K % 32 == 0, N % 8 == 0; bias / R / Y as in
 * kx_outproj_residual (R may be Y).  Tiles of 128, 192 or 256 columns by 128 rows (one CTA), or of 128 / 192
 * columns by 256 rows (a CTA pair), FP32 accumulation in tensor memory, tolerance as for the BF16 path
 * against the exact value of the formula.  The _ex form takes a plan override of which block_n
 * (128 / 192 / 256), cta_pair (1 / 2) and raster_group are honoured (tests, tuning); NULL = automatic
 * (single-CTA tiles, width by an estimate of waves x time per tile).
 * Errors: KX_ERR_SHAPE, KX_ERR_NULL, KX_ERR_ALIGN, KX_ERR_OVERLAP as for the calls above.
 */
int64_t kx_mx_scale_bytes(int64_t rows, int64_t cols);
int kx_quantize_rows_mxfp8(const void* A, void* Q, void* SF, int64_t rows, int64_t cols, void* stream);
int kx_rmsnorm_quantize_mxfp8(const void* H, const void* gamma, float eps, void* Q, void* SF,
                              int64_t M, int64_t N, void* stream);
int kx_outproj_residual_mxfp8(const void* Xq, const void* SFX, const void* Wq, const void* SFW,
                              const void* bias_or_null, const void* R_or_null, void* Y,
                              int64_t M, int64_t N, int64_t K, void* stream);
/* Block-scaled gate/up step: kx_quantize_gate_up_mxfp8 writes the code books of the gate and the up weights
 * (Wg, Wu [I, K] BF16 -> Qg, Qu [I, K] codes) and their scale arrays back to back into SFGU (gate first;
 * 2 * kx_mx_scale_bytes(I, K) bytes).  kx_gate_up_swiglu_mxfp8 computes
 *     Z[m,i] = bf16( silu(g) * u ),  g / u = the block-scaled products of row m of Xq with row i of Wgq / Wuq
 * (Appendix A, Algorithm 7's gate/up GEMM with SwiGLU epilogue on block-scaled operands).  K % 32 == 0,
 * I % 8 == 0; Z [M, I] BF16; no bias, no residual; pointers and errors as above. */
int kx_quantize_gate_up_mxfp8(const void* Wg, const void* Wu, void* Qg, void* Qu, void* SFGU,
                              int64_t I, int64_t K, void* stream);
int kx_gate_up_swiglu_mxfp8(const void* Xq, const void* SFX, const void* Wgq, const void* Wuq, const void* SFGU,
                            void* Z, int64_t M, int64_t I, int64_t K, void* stream);
int kx_outproj_residual_mxfp8_ex(const void* Xq, const void* SFX, const void* Wq, const void* SFW,
                                 const void* bias_or_null, const void* R_or_null, void* Y,
                                 int64_t M, int64_t N, int64_t K, void* stream,
                                 const kx_plan_override* override_or_null);

/*
 * 4-bit block-scaled branch (the number format of the Section 4.3 task, E2M1 elements scaled in blocks of 16, and
 * the tensor-core kind it runs on).  Elements are E2M1 codes (sign, two exponent bits, one mantissa bit:
 * magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6), two per byte with the even k index in the low nibble; every 16
 * consecutive elements of a row share one E4M3 scale byte (non-negative, never NaN); one binary32 scale gs
 * belongs to the whole tensor:  value = e2m1(q) * e4m3(s) * gs.
 *
 * Code book (kx_quantize_rows_nvfp4), per block of 16 BF16 values z, every step in binary32:
 *     s = e4m3( max|z| / (6 gs) )        nearest, ties to even, saturating at 448
 *     q = e2m1( z * (1 / (value(s) gs)) )   nearest, ties to the even code, saturating at +-6; all codes 0
 *                                           when s decodes to zero
 * gs > 0 is the caller's (typically max|A| / (448 * 6)).  A [rows, cols] BF16, cols % 16 == 0, cols <= 32768;
 * Q [rows, cols / 2] bytes; SF as below; device pointers, 16-byte aligned, no overlap.
 *
 * Scale layout: chunks of 512 bytes, one per (128 rows, 64 elements of K), ordered
 * [ceil(rows / 128)][ceil(cols / 64)]; inside a chunk the scale of row r and 16-element block j sits at
 * byte (r % 32) * 16 + (r % 128) / 32 * 4 + j % 4 (the 512-byte atom of Section 4.3).
 * kx_nvfp4_scale_bytes gives the size of the array.  Padding entries (rows >= rows, blocks >= cols / 16) are
 * written as 0 by the code book; arrays built elsewhere must hold finite E4M3 bytes there.
 *
 * kx_outproj_residual_nvfp4:
 *     Y[m,n] = bf16( alpha * sum_j e4m3(sx[m,j]) e4m3(sw[n,j]) sum_{k in block j} xq[m,k] wq[n,k] + bias[n] + R[m,n] )
 * with alpha = the product of the two tensor scales.  Xq [M, K/2], Wq [N, K/2] bytes; K % 32 == 0,
 * N % 8 == 0; bias / R / Y as in kx_outproj_residual (R may be Y).  One CTA per 128 x 128 / 192 / 256 tile
 * (tcgen05 kind::mxf4nvf4.block_scale, FP32 accumulation); the override may name block_n and raster_group
 * (NULL = automatic).  Errors as for the calls above.
 */
int64_t kx_nvfp4_scale_bytes(int64_t rows, int64_t cols);
int kx_quantize_rows_nvfp4(const void* A, float gs, void* Q, void* SF, int64_t rows, int64_t cols, void* stream);
/* The other steps of the layer on the 4-bit format, mirroring the block-scaled FP8 calls:
 * kx_rmsnorm_quantize_nvfp4 = code book of RMSNorm(H) * gamma (rounded to BF16 as kx_rmsnorm writes it) with
 * tensor scale gs; kx_quantize_gate_up_nvfp4 = code books of the gate and up weights (tensor scales gsg, gsu),
 * scale arrays back to back in SFGU (gate first; 2 * kx_nvfp4_scale_bytes(I, K) bytes);
 * kx_gate_up_swiglu_nvfp4: Z[m,i] = bf16( silu(alpha_g g) * (alpha_u u) ) with g / u the block-scaled sums of row
 * m of Xq with row i of Wgq / Wuq and alpha_g / alpha_u = tensor scale of X times that of the gate / up
 * weights.  K % 32 == 0, I % 8 == 0. */
int kx_rmsnorm_quantize_nvfp4(const void* H, const void* gamma, float eps, float gs, void* Q, void* SF,
                              int64_t M, int64_t N, void* stream);
int kx_quantize_gate_up_nvfp4(const void* Wg, const void* Wu, float gsg, float gsu, void* Qg, void* Qu, void* SFGU,
                              int64_t I, int64_t K, void* stream);
int kx_gate_up_swiglu_nvfp4(const void* Xq, const void* SFX, const void* Wgq, const void* Wuq, const void* SFGU,
                            float alpha_g, float alpha_u, void* Z, int64_t M, int64_t I, int64_t K, void* stream);
int kx_outproj_residual_nvfp4(const void* Xq, const void* SFX, const void* Wq, const void* SFW, float alpha,
                              const void* bias_or_null, const void* R_or_null, void* Y,
                              int64_t M, int64_t N, int64_t K, void* stream,
                              const kx_plan_override* override_or_null);

/* Fills `out` with the plan the library would use for this shape on the current
 * device (has_residual / has_bias as 0 or 1).  No work is enqueued. */
int kx_plan_query(int64_t M, int64_t N, int64_t K, int has_bias, int has_residual,
                  const kx_plan_override* ov_or_null, kx_plan_info* out);

/*
 * Synchronises `stream`, then reads and clears the current device's kernel
 * status word.  *code_out is KX_OK or KX_ERR_DEVICE_TIMEOUT; *detail_out (may be
 * NULL) identifies which wait gave up.  Debug/test use: it blocks the host.
 * Allocates nothing and needs no kx_init: the status word is part of the library's device
 * image (callers of kx_outproj_residual_noalloc may use it).
 */
int kx_last_device_status(void* stream, int* code_out, int* detail_out);

/* Static string for a kx_status value. */
const char* kx_status_string(int status);

/* KX_VERSION the library was built from. */
int kx_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KX_H_ */
