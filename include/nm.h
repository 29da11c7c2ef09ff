/*
 * nm.h -- C ABI of the B200 (sm_100a) N:M-sparse-weight x dense-activation GEMM.
 *
 *     Y[T x O] = X[T x K] * W~[O x K]^T
 *
 * W~ is a weight pruned so that every aligned group of m consecutive k inside
 * one output row keeps at most n nonzeros (the paper's Section 2.1 definition of
 * N:M sparsity; the linear layers qkv / proj / fc1 / fc2 of a ViT block are the
 * operators it replaces).  X, W and Y are row-major.  T = tokens, K = reduction
 * length (in-features), O = out-features.
 *
 * Conventions for every call
 *   - "host" / "device" in an argument's comment says where the pointer lives.
 *   - The library never allocates or frees device memory: the caller owns every
 *     buffer (packed weight, X, Y, workspace, status word) and passes raw
 *     pointers.  nm_weight / nm_plan are plain structs in caller-owned host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Device work is only enqueued; nothing synchronises unless said.
 *   - Every call returns an nm_status; nothing aborts, traps or prints.
 *   - ld* arguments are row pitches in ELEMENTS of the respective dtype.
 */
#ifndef NM_H_
#define NM_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define NM_API __attribute__((visibility("default")))
#else
#define NM_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  NM_OK = 0,
  NM_ERR_INVALID_ARG = 1, /* null pointer, negative size, bad enum, n>m ...            */
  NM_ERR_SHAPE = 2,       /* K % m != 0, K >= 131072 (int32 overflow bound), m too big */
  NM_ERR_ALIGN = 3,       /* pointer not 16-byte aligned or pitch*elem not 16 B mult.  */
  NM_ERR_NOT_NM = 4,      /* a group of W holds more than n nonzeros                   */
  NM_ERR_UNSUPPORTED = 5, /* the requested plan cannot run this weight / shape         */
  NM_ERR_WORKSPACE = 6,   /* workspace or destination buffer too small                 */
  NM_ERR_ARCH = 7,        /* device is not compute capability 10.0                     */
  NM_ERR_CUDA = 8,        /* a CUDA runtime / driver call failed                       */
  NM_ERR_TIMEOUT = 9      /* device side: a bounded wait expired (see status word)     */
} nm_status;

typedef enum { NM_I8 = 0, NM_F16 = 1 } nm_dtype;                 /* dtype of X and W  */
typedef enum { NM_OUT_I32 = 0, NM_OUT_F32 = 1, NM_OUT_F16 = 2, NM_OUT_I8 = 3 } nm_out_dtype;
/* Legal pairs: NM_I8 -> NM_OUT_I32 (exact int32 accumulation);
 *              NM_I8 -> NM_OUT_I8  (requantising epilogue, nm_spmm_ex only);
 *              NM_F16 -> NM_OUT_F32 or NM_OUT_F16 (fp32 accumulation, RN to fp16). */

/* Device images of a packed weight (bitmask).  The canonical image is always
 * built; the others are re-orderings of it that a kernel can consume directly. */
enum {
  NM_IMG_CANONICAL = 1u, /* header + values + b-bit positions (format below)              */
  NM_IMG_HW24 = 2u,      /* 2:4-compressed values + hardware metadata blocks; exists when
                            every 4-chunk of W holds <= 2 nonzeros (always for n<=2, 4|m) */
  NM_IMG_DENSE = 4u,     /* W~ itself, row pitch rounded to 16 B (n==m reuses canonical)  */
  NM_IMG_REMAP48 = 8u,   /* three-chunk K remap (see NM_PATH_UMMA_REMAP48): exists when every aligned
                            group of 8 k holds <= 4 nonzeros (4:8, 3:8, ...); only built on request */
  NM_IMG_AUTO = 0x80000000u /* let nm_compress choose everything that applies            */
};

/* Execution paths of nm_spmm (nm_plan.path). */
enum {
  NM_PATH_SIMT = 0,       /* CUDA-core kernel over the canonical image; any n:m, any shape */
  NM_PATH_UMMA_DENSE = 1, /* TMA -> smem -> dense tcgen05.mma, accumulators in TMEM        */
  NM_PATH_UMMA_SP24 = 2,  /* TMA -> smem -> tcgen05.mma.sp (2:4 hardware sparsity)         */
  NM_PATH_UMMA_DECODE = 3,/* canonical image -> decode warps build the zero-filled micro-dense
                             tile in smem -> dense tcgen05.mma; any n:m, no extra image.  A
                             correctness fallback for callers with neither a pre-arranged image nor
                             scratch: every W tile is decoded again for every token tile that meets
                             it, measured 2-17x the time of NM_PATH_UMMA_EXPAND / a dense image   */
  NM_PATH_UMMA_EXPAND = 4,/* canonical image -> one small kernel writes the zero-filled dense rows
                             once into the head of the workspace (O x round_up(K*eb,16) bytes,
                             counted in nm_plan.workspace_bytes; it stays in L2) -> the dense
                             tcgen05.mma path reads it.  For token counts where decoding the same
                             W tile again for every token tile would dominate; any n:m, no extra
                             image.  Without enough workspace an automatic plan falls back to
                             NM_PATH_UMMA_DECODE                                          */
  NM_PATH_UMMA_REMAP48 = 5 /* 4:8-type weights on the 2:4 sparse tensor core at 3/4 of the dense MMA
                             count.  A group of 8 k with up to 4 nonzeros is spread over THREE 4-chunks of
                             a longer K axis, each holding <= 2: the two chunks of the group itself, and a
                             third one that repeats the activations k+0, k+1, k+4, k+5 of the group and
                             takes whatever a chunk holds beyond two (any 3 of 4 positions include one of
                             the first two, so the move is always possible).  The third chunks of all
                             groups form an extra K range of K/2, whose activations one small kernel
                             gathers into the head of the workspace (T x round_up(K/2*eb,16) bytes) before
                             the sparse kernel runs over K + K/2.  Opt-in (nm_plan_create never selects
                             it): it needs NM_IMG_REMAP48, single CTAs, no split-K; it loads 1.5x the
                             activation bytes and measured slower than the dense path on B200, whose
                             tcgen05 kernels are bound by operand movement, not by MMA count               */
};

/* Operand residency of the tcgen05 paths (nm_plan.resident).  A persistent CTA walks a
 * contiguous run of output tiles; the operand named here is loaded once per run of tiles
 * that share it, the other operand streams through the shared-memory ring.  A request that
 * does not fit in shared memory degrades to NM_RES_NONE. */
enum {
  NM_RES_NONE = 0, /* both operands stream (also the only mode with split_k > 1)             */
  NM_RES_X = 1,    /* the token tile of X stays; the CTA sweeps out-feature tiles of W       */
  NM_RES_W = 2     /* the out-feature tile of W stays; the CTA sweeps token tiles of X       */
};

/* How the partial sums of a split-K plan are merged (Section 4.3: only in the final stage).
 * Both add the slices of a tile in an order that is fixed by the plan, never by timing: INT8
 * results are identical under either, floating-point results are reproducible run to run for a
 * given plan and differ between the two only by the order of the last split_k additions. */
enum {
  NM_MERGE_WORKSPACE = 0, /* every slice is stored to the workspace (nm_plan.workspace_bytes), then a
                             second kernel adds the slices and applies the epilogue                    */
  NM_MERGE_CLUSTER = 1    /* the K slices of a tile are the CTAs of one thread-block cluster; the
                             partials are exchanged through distributed shared memory and the owner
                             of each 32 x 32 patch adds them and stores the final output.  No
                             workspace.  Single-CTA tcgen05 paths (not the decode path) with
                             tile_t <= 64 and split_k <= 8; NM_ERR_INVALID_ARG otherwise.  Opt-in:
                             nm_plan_create never selects it.  Timed alone it is ~0.9 us faster than
                             the workspace merge while tiles * split_k <= ~0.44 * SMs (every cluster
                             resident at once); between other launches of a stream it overlaps less
                             than the workspace merge's two dependent launches and measured slower  */
};

/* Description of one packed weight.  Filled by nm_compress; POD, caller-owned. */
typedef struct nm_weight {
  uint32_t magic;    /* 'NMWD' */
  uint32_t version;  /* 1 */
  int32_t O, K, n, m;
  int32_t dtype;     /* nm_dtype */
  uint32_t images;   /* NM_IMG_* actually present */
  void* dev_base;    /* device: start of the packed buffer (256-byte aligned) */
  uint64_t bytes;    /* bytes used inside dev_base */
  uint64_t off_canonical;
  uint64_t off_hw24_values, off_hw24_meta, off_dense;  /* 0 when absent */
  uint64_t hw24_row_bytes, dense_row_bytes;            /* row pitches in bytes */
  int32_t hw24_meta_kblocks;                           /* 2 KB metadata blocks per 128-row tile */
  int32_t reserved;
  /* NM_IMG_REMAP48 (0 when absent): a 2:4 image of the remapped weight W' [O x remap_k], whose columns
   * [0, K) are W without the moved elements, [K, remap_k_main) zero padding up to a whole K step, and
   * [remap_k_main, remap_k) the third chunks: column remap_k_main + 4g + j pairs with activation
   * 8g + {0,1,4,5}[j] */
  uint64_t off_remap_values, off_remap_meta, remap_row_bytes;
  int32_t remap_meta_kblocks, remap_k, remap_k_main, reserved2;
} nm_weight;

/* Launch plan: a deterministic function of (T, O, K, n, m, dtypes, images, #SMs). */
typedef struct nm_plan {
  int32_t path;      /* NM_PATH_* */
  int32_t tile_o;    /* out-features per CTA tile (MMA M), 128 on the tcgen05 paths */
  int32_t tile_t;    /* tokens per CTA tile (MMA N): 32..256 */
  int32_t cta_group; /* 1, or 2: a cluster of two CTAs shares one 256-row tile (cta_group::2 MMAs) */
  int32_t split_k;   /* 1, 2, 4, 8 or 16 slices of the K loop */
  int32_t stages;    /* depth of the TMA -> MMA shared-memory ring (upper bound: reduced to fit smem) */
  uint32_t image;    /* NM_IMG_* the path reads */
  int32_t resident;  /* NM_RES_*: operand a CTA keeps in shared memory across consecutive tiles */
  uint64_t workspace_bytes; /* device scratch nm_spmm needs for this plan: the split-K slices (none if split_k==1 or
                               merge==NM_MERGE_CLUSTER), after the dense copy of NM_PATH_UMMA_EXPAND if that is the path */
  float predicted_us;       /* roofline estimate, 0 if unknown */
  int32_t issuers;          /* single-CTA tcgen05 paths: 1, or 2 = a second warp issues the odd K steps of every
                               tile into a second accumulator that the epilogue adds (0 is read as 1) */
  int32_t merge;            /* NM_MERGE_*: where the split_k partial sums of a tile meet (ignored when split_k == 1) */
  int32_t reserved;         /* 0, or NM_PLAN_DIAG_* bits */
} nm_plan;

/* Diagnostic bit of nm_plan.reserved (single-CTA tcgen05 paths; ignored elsewhere).  Every wait in
 * the kernels is a bounded poll: when one runs out, the CTA ORs (NM_ERR_TIMEOUT | 1 << (8 + site))
 * into the status word, raises a CTA-wide abort flag, lets the copies it issued land, frees its
 * tensor memory and returns.  NM_PLAN_DIAG_STALL makes that path observable without a fault: CTA 0
 * arms the barrier of its first K step for 16 bytes more than it requests, so every copy lands,
 * that one barrier never completes, and the waits behind it -- the issuing warp's for the stage
 * (site 2), the epilogue's for the accumulator (site 3), the producer's for the stage to come free
 * again (site 1) -- run out after a poll budget cut to milliseconds for this launch.  The call
 * returns normally, the status word holds NM_ERR_TIMEOUT and the bit of whichever of those sites
 * expired first, Y is unspecified, and the stream stays usable. */
enum { NM_PLAN_DIAG_STALL = 1 };

/* One row of the latency table (Section 5.1: per-operator sparsity-latency LUT). */
typedef struct nm_latency_row {
  int32_t T, O, K, n, m;
  int32_t dtype, out_dtype;
  int32_t path, tile_t, split_k;
  int32_t reps;
  int32_t status;      /* nm_status of the measurement */
  float us_mean, us_min;
} nm_latency_row;

/* ---------------------------------------------------------------------------
 * Packing (Section 4.2, "Weight Packing": B_pack jointly encodes the kept values and
 * their positions inside each N:M window; built once, offline, untimed -- Section 6.1).
 *
 * Canonical image (little-endian; also what nm_export_canonical returns):
 *   header 64 B : "NMW1", u32 version=1, u32 dtype, i32 O, K, n, m, G=K/m,
 *                 b=ceil(log2 m) (0 when n==m), i32 0, u64 val_row_bytes,
 *                 u64 idx_row_bytes, u64 0
 *   values      : O rows of val_row_bytes=roundup16(G*n*elem); slot s=g*n+j is the
 *                 j-th kept element of group g, ascending k
 *   positions   : O rows of idx_row_bytes=roundup16(ceil(G*n*b/8)); slot s owns
 *                 bits [s*b,(s+1)*b) of the row's bit stream, value 0..m-1
 *   A group with fewer than n nonzeros is padded with its smallest unused positions
 *   (value 0) and the slots are sorted by position.  "Zero" is ==0 (fp16 -0.0 too).
 * ------------------------------------------------------------------------- */

/* Bytes of device memory nm_compress needs for (O,K,n,m,dt) with `images`
 * (NM_IMG_AUTO = worst case over everything that may be built).  0 on bad args. */
NM_API size_t nm_packed_size(int O, int K, int n, int m, nm_dtype dt, uint32_t images);

/* Pack a dense, already-pruned weight.
 *   W_dense_host  host, row-major [O x K] of dt, row pitch ldw elements
 *   images        NM_IMG_* wanted (canonical is always added; NM_IMG_AUTO picks
 *                 HW24 when W is 2:4-clean and a row is longer than 128 bytes, else DENSE;
 *                 n==m needs neither)
 *   dev_buf       device, >= nm_packed_size bytes, 256-byte aligned, caller-owned
 *   out           host, receives the descriptor
 *   bad_row/group host, nullable; on NM_ERR_NOT_NM receive the first offender
 * Packs on the host, then copies to dev_buf on `stream` and waits for that copy.
 * Strict: never prunes.  Requesting NM_IMG_HW24 for a weight that is not 2:4-clean
 * returns NM_ERR_UNSUPPORTED. */
NM_API nm_status nm_compress(const void* W_dense_host, int64_t ldw, int O, int K, int n, int m,
                      nm_dtype dt, uint32_t images, void* dev_buf, size_t dev_bytes,
                      void* stream, nm_weight* out, int64_t* bad_row, int64_t* bad_group);

/* Same packing into HOST memory (no GPU needed): host_buf receives the byte-identical
 * blob nm_compress would upload; out->dev_base is left NULL.  To use the blob later, copy
 * out->bytes bytes to a 256-byte-aligned device buffer and set out->dev_base to it. */
NM_API nm_status nm_compress_host(const void* W_dense_host, int64_t ldw, int O, int K, int n, int m,
                                  nm_dtype dt, uint32_t images, void* host_buf, size_t host_bytes,
                                  nm_weight* out, int64_t* bad_row, int64_t* bad_group);

/* In-place magnitude pruning helper (host): keep the n largest |w| of each group,
 * ties to the lower k.  The paper prunes upstream in training; this only makes
 * arbitrary weights legal inputs of nm_compress. */
NM_API nm_status nm_prune_magnitude(void* W_dense_host, int64_t ldw, int O, int K, int n, int m,
                             nm_dtype dt);

/* Rebuild W~ (host, row pitch ldw elements) from the canonical device image.
 * Copies device -> host on `stream` and waits. */
NM_API nm_status nm_decompress(const nm_weight* w, void* W_dense_host, int64_t ldw, void* stream);

/* Copy the canonical image to host memory.  host_buf may be NULL to query *bytes;
 * otherwise *bytes is the capacity on entry and the size written on return. */
NM_API nm_status nm_export_canonical(const nm_weight* w, void* host_buf, size_t* bytes, void* stream);

/* ---------------------------------------------------------------------------
 * Planning (Section 4.3, "Adaptive Parallelism": split-K grows the parallel space
 * from (M, N) tiles to (M, N, splitK); raise splitK until the grid fills the SMs,
 * from a small discrete set aligned to the MMA K step; fall back to a smaller
 * splitK when K is short or the reduction traffic would dominate).
 *   device  CUDA device ordinal whose SM count is used; -1 = assume 148 SMs
 *           (pure host call, usable without a GPU)
 * ------------------------------------------------------------------------- */
NM_API nm_status nm_plan_create(int T, const nm_weight* w, nm_out_dtype od, int device, nm_plan* out);

/* Same rule on bare numbers (no weight needed): `images` says which device images
 * exist; n_sms <= 0 means 148. */
NM_API nm_status nm_plan_shape(int T, int O, int K, int n, int m, nm_dtype dt, nm_out_dtype od,
                        uint32_t images, int n_sms, nm_plan* out);

/* ---------------------------------------------------------------------------
 * The GEMM (Section 4.2 micro-dense execution + Section 4.3 split-K, final-stage merge).
 *   X_dev   device, [T x K] of w->dtype, pitch ldx elements, 16-byte aligned,
 *           ldx*elem a multiple of 16 B
 *   w       host, from nm_compress (its dev_base must still be alive)
 *   plan    host, nullable: NULL = nm_plan_create's choice for the current device
 *   Y_dev   device, [T x O] of `od`, pitch ldy elements, 16-byte aligned
 *   workspace_dev / workspace_bytes  device scratch >= plan->workspace_bytes
 *           (may be NULL/0 when the plan needs none); contents are overwritten
 *   status_dev  device, nullable: one uint32 the kernel ORs with
 *           (NM_ERR_TIMEOUT | 1 << (8 + site)) if a bounded wait expires (low byte: the status;
 *           bits 9..19: which waits ran out -- 1 producer for a free ring stage, 2 issuing warp
 *           for a loaded stage, 3 epilogue for an accumulator, 4 issuing warp for a drained
 *           accumulator, 7-9 resident operand, 10 decode warps, 11 on-chip split-K merge); the
 *           caller zeroes it and reads it after synchronising.  Y is then unspecified.
 * Enqueues on `stream` and returns; no synchronisation, no allocation.
 * The kernels are launched with programmatic stream serialisation: their prologue, and the
 * fetch of the first weight tiles, may overlap the tail of the previous kernel on the stream;
 * X, Y and the workspace are only touched once that kernel has completed.  The packed weight
 * must therefore not be produced by device work enqueued on the same stream right before the
 * call (nm_compress returns only after its copy has finished, which satisfies this).
 * INT8 results are bit-identical for every plan; FP16 results are bit-identical
 * run to run for a fixed plan.
 * ------------------------------------------------------------------------- */
NM_API nm_status nm_spmm(const void* X_dev, int64_t ldx, int T, const nm_weight* w, const nm_plan* plan,
                  void* Y_dev, int64_t ldy, nm_out_dtype od, void* workspace_dev,
                  size_t workspace_bytes, uint32_t* status_dev, void* stream);

/* Fused requantising epilogue for INT8 inference (the paper's end-to-end stack runs INT8 layer
 * to layer, Section 6.3; the GEMM's INT32 accumulator has to come back to INT8 somewhere, and
 * writing 1 byte instead of 4 per output is what lets 2:4 sparsity pay on B200).  Per output:
 *     a = acc[t,o] + bias[o]                      (int32, wraps like the accumulator)
 *     v = (float)a * scale[o]                     (int32 -> fp32 round-to-nearest-even, one fp32 multiply)
 *     v = max(v, 0) if relu
 *     Y[t,o] = (int8) clamp(rint(v), -128, 127)   (round-to-nearest-even, saturating)
 * Every step is a single IEEE operation, so a CPU reproduces the result bit for bit.
 * scale[] must be finite (a NaN product is stored as 0 here and is undefined in C). */
typedef struct nm_epilogue {
  const float* scale_dev;   /* device, [O] fp32, required                        */
  const int32_t* bias_dev;  /* device, [O] int32, nullable                       */
  int32_t relu;             /* 0 / 1                                             */
  int32_t reserved;
} nm_epilogue;

/* nm_spmm with an epilogue.  epi == NULL is exactly nm_spmm.  With an epilogue: w->dtype must
 * be NM_I8, od must be NM_OUT_I8, Y_dev is int8 [T x O] with pitch ldy elements; everything
 * else (plan, workspace, status word, stream semantics) is as for nm_spmm. */
NM_API nm_status nm_spmm_ex(const void* X_dev, int64_t ldx, int T, const nm_weight* w, const nm_plan* plan,
                            void* Y_dev, int64_t ldy, nm_out_dtype od, const nm_epilogue* epi,
                            void* workspace_dev, size_t workspace_bytes, uint32_t* status_dev, void* stream);

/* The same GEMM for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a deployment convenience).  Think of a server whose device memory
 * was handed out at start-up, a latency-critical loop where cudaMalloc would stall the
 * device, or a plug-in inside another framework's memory arena: such a caller cannot
 * provide the split-K workspace that nm_spmm asks for.  Here the partial sums go to a
 * fixed array of NM_STATIC_SCRATCH_BYTES that is part of the library image; every GPU
 * that loads the library holds that array until the process exits.
 *   - Arguments are those of nm_spmm without the workspace pair; X, Y and the packed
 *     weight are still the caller's buffers.
 *   - An explicit plan whose workspace_bytes exceeds NM_STATIC_SCRATCH_BYTES returns
 *     NM_ERR_WORKSPACE; nothing is launched.  Plans with split_k == 1 need no scratch
 *     and always pass.
 *   - plan may be NULL: the automatic plan is then made against the fixed array and
 *     degrades like nm_spmm's (no split-K, or on-chip decode instead of the dense scratch
 *     copy, when the array is too small; the CUDA-core path when X or Y is not 16-byte
 *     aligned): it never fails on scratch size or alignment.
 *   - No cudaMalloc / cudaFree / allocating library routine is called, on any path.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents.  Nothing
 *     needs clearing between calls (each call overwrites what it later reads), but two
 *     calls that overlap on the GPU -- different streams, or graph branches without an
 *     edge between them -- race on it: serialise them. */
#define NM_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
NM_API nm_status nm_spmm_static_scratch(const void* X_dev, int64_t ldx, int T, const nm_weight* w,
                                        const nm_plan* plan, void* Y_dev, int64_t ldy, nm_out_dtype od,
                                        uint32_t* status_dev, void* stream);

/* ---------------------------------------------------------------------------
 * Latency table export (Section 5.1: for each operator shape and candidate N:M ratio,
 * benchmark the sparse GEMM and average repeated runs -> LUT indexed by (shape, sparsity)).
 * Times nm_spmm for every shape x n:m pair on caller buffers: `reps` back-to-back calls are
 * captured in one CUDA graph and replayed (CUDA events around the replay), so a row is the
 * steady-state cost of the operator inside a model, not the cost of one isolated launch.  The
 * work runs on a private stream after the caller's stream has drained.
 *   shapes_TOK  host, n_shapes triples (T, O, K)
 *   nm_pairs    host, n_pairs pairs (n, m)
 *   X_dev       device, >= max T*K elements of dt (contents arbitrary but finite)
 *   Wpack_dev   device, >= max nm_packed_size(..., NM_IMG_AUTO) bytes
 *   Y_dev       device, >= max T*O output elements
 *   workspace_dev/bytes  device scratch, as for nm_spmm (largest plan)
 *   rows_out    host, n_shapes*n_pairs rows, shape-major
 * Weights are synthetic (every group keeps its first n positions).  Synchronises.
 * ------------------------------------------------------------------------- */
NM_API nm_status nm_latency_table(const int32_t* shapes_TOK, int n_shapes, const int32_t* nm_pairs,
                           int n_pairs, nm_dtype dt, nm_out_dtype od, int reps,
                           void* X_dev, void* Wpack_dev, size_t wpack_bytes, void* Y_dev,
                           void* workspace_dev, size_t workspace_bytes,
                           nm_latency_row* rows_out, void* stream);

/* ---------------------------------------------------------------------------
 * Latency predictor (Section 5.1, Eq. (1)): T_pred(s) = sum_l gamma_l * t_l(s_l) + b with
 * gamma_l >= 0 and b >= 0, where t_l(s_l) is the table latency of layer l under its ratio.
 * Host-only functions; all pointers are host pointers; nothing is allocated that outlives
 * the call.
 *
 * nm_predictor_fit calibrates the coefficients by non-negative least squares:
 *   lut_us       [S x L] row-major: row i holds t_l(s_l) of measured configuration i
 *   measured_us  [S] the measured end-to-end latencies of those configurations
 *   gamma_out    [L], b_out: the minimiser of || [lut_us 1] x - measured_us ||_2 over x >= 0
 *   rnorm_out    optional: the residual 2-norm at the solution
 * The solver is the active-set method of Lawson and Hanson; where the minimiser is not unique
 * (rank-deficient table) it returns one minimiser.  NM_ERR_INVALID_ARG for null pointers,
 * S < 1, L < 0 or non-finite inputs; NM_ERR_UNSUPPORTED if the iteration limit (3 (L+1) + 30
 * outer steps) is reached, with the best feasible iterate left in the outputs.
 *
 * nm_predictor_eval evaluates Eq. (1) for n_cfg configurations: t_us [n_cfg x L] -> pred_out[n_cfg].
 * ------------------------------------------------------------------------- */
NM_API nm_status nm_predictor_fit(const double* lut_us, const double* measured_us, int S, int L,
                                  double* gamma_out, double* b_out, double* rnorm_out);
NM_API nm_status nm_predictor_eval(const double* gamma, double b, const double* t_us, int n_cfg, int L,
                                   double* pred_out);

/* ---------------------------------------------------------------------------
 * Hardware-aware layer-wise sparsity search (Section 5.2, Algorithm 1).  Host only.
 *
 * A configuration is y[l] in 1..levels for l < L (N of N:levels, 8 in the paper).  Its latency is
 * Eq. (1) over the table: sum_l gamma[l] * table_us[l * levels + y[l] - 1] + b, summed in layer
 * order in double precision.  Its fitness is `fitness(y, L, user)` if the latency is within
 * target_us and -infinity otherwise (Eq. (4)).
 *
 * Initialisation: the densest uniform configuration within the budget; from it `n_init`
 * candidates, each one pass over the layers in random order densifying a layer by one level
 * when the result still fits; the fittest is the first parent.  Then `generations` times:
 * `offspring` children of the parent, each by
 *   overshoot: min(overshoot_k, #layers below the top level) distinct random layers go one level denser;
 *   repair:    while over budget, a random layer above level 1 goes one level sparser;
 *   refine:    while some layer can go one level denser without lowering the fitness
 *              (Delta Fitness >= 0, -inf if over budget), one such layer, chosen at random, does;
 * and the fittest child (with `elitist` != 0 the parent competes too) becomes the parent.  Ties
 * keep the earliest.  Random choices: splitmix64 seeded with `seed`; an index below n is the high
 * 64 bits of (next output) * n; K distinct members are the head of a partial Fisher-Yates shuffle
 * of the candidate list in ascending order.  A run is therefore reproducible from its arguments.
 *
 * The paper's fitness is the accuracy a configuration inherits from a trained supernet; the caller
 * supplies it as a callback.  nm_fitness_separable is a synthetic stand-in:
 * sum_l gain[l * levels + y[l] - 1] plus noise * (u - 0.5), u in [0,1) from a hash of y.
 *
 * Returns NM_ERR_INVALID_ARG for null pointers, L < 1, levels < 1, offspring < 1, generations < 0
 * or n_init < 1; NM_ERR_UNSUPPORTED when no uniform configuration fits the budget (y_out is then
 * all ones and result->feasible is 0).
 * ------------------------------------------------------------------------- */
typedef double (*nm_fitness_fn)(const int32_t* y, int32_t L, void* user);

typedef struct nm_search_config {
  int32_t L;            /* layers */
  int32_t levels;       /* ratio levels per layer (8: N of N:8) */
  int32_t generations;  /* G */
  int32_t offspring;    /* lambda */
  int32_t overshoot_k;  /* K of Random_K in the overshoot stage */
  int32_t n_init;       /* candidates drawn for the first parent */
  int32_t elitist;      /* 0: best of the offspring (algorithm listing); 1: parent competes ("(1+lambda)") */
  int32_t reserved;
  double target_us;     /* latency budget */
  uint64_t seed;
} nm_search_config;

typedef struct nm_search_result {
  double fitness;          /* Eq. (4) of y_out */
  double latency_us;       /* Eq. (1) of y_out */
  uint64_t fitness_evals;  /* calls of the fitness callback */
  uint64_t latency_evals;  /* evaluations of Eq. (1) */
  int32_t feasible;        /* 1 if latency_us <= target_us */
  int32_t reserved;
} nm_search_result;

typedef struct nm_fitness_separable_args {
  const double* gain;   /* [L x levels] row-major */
  int32_t levels;
  int32_t reserved;
  double noise;         /* amplitude of the configuration-dependent perturbation (0: none) */
  uint64_t seed;
} nm_fitness_separable_args;

NM_API nm_status nm_search(const nm_search_config* cfg, const double* table_us, const double* gamma, double b,
                           nm_fitness_fn fitness, void* user, int32_t* y_out, nm_search_result* result);
/* `user` must point to an nm_fitness_separable_args. */
NM_API double nm_fitness_separable(const int32_t* y, int32_t L, void* user);

NM_API const char* nm_status_string(nm_status s);

/* Number of kernels this library has launched in the calling process (for
 * benchmark bookkeeping). */
NM_API uint64_t nm_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* NM_H_ */
