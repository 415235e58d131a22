/*
 * lrd.h - C ABI of the B200 (sm_100a) library for the training step of low-rank
 * decomposed layers.
 *
 * A dense layer weight W[N x K] (N outputs, K inputs) is replaced by two factors,
 *     V[K x r]  (input side, applied first)   and   U[N x r]  (output side, applied second),
 * so that the layer is two consecutive fully connected layers (paper, Section 2, Fig. 1):
 *     Z[M x r] = X[M x K] V            Y[M x N] = Z U^T + 1 b^T .
 * (The paper writes W in R^{C x S} with C inputs and S outputs and calls the input-side
 * factor U' and the output-side factor V' (Eq. 2); this header uses the letters above.)
 * A k x k convolution is replaced by its Tucker-2 form (Eq. 4): a 1x1 convolution A[C x r1],
 * a k x k core G[r2][k][k][r1] and a 1x1 convolution Bm[S x r2].
 *
 * Conventions that hold for every entry point
 *  - All matrices are row-major.  Leading dimensions are in elements; 0 means packed.
 *  - Pointers named X, V, U, bias, Y, Z_save, dY, dX, dU, dV, dbias, A, G, Bm, Z1_save, Z2_save,
 *    dA, dG, dB and `workspace` are DEVICE pointers owned by the caller.  The library allocates
 *    no device memory, keeps no per-call device state, and never synchronises: all work is
 *    enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = the default stream).
 *  - `workspace` must hold at least lrd_*_workspace_bytes(...) bytes and be 256-byte aligned.
 *    Its contents are scratch: undefined on return, nothing is carried between calls.
 *  - Storage is fp32 or bf16 (lrd_dtype_t); products always accumulate in fp32.  Outputs and
 *    gradients have the storage type of the tensor they belong to and are overwritten.
 *  - Errors are return codes.  Arguments are checked on the host before anything is launched;
 *    nothing aborts, asserts or traps.  Every wait inside a kernel is bounded; a wait that runs
 *    out raises a device-side flag that lrd_check_device_status() reports as LRD_ERR_TIMEOUT.
 *  - Ranks and sizes that do not meet the alignment needs of the tensor-core path (every
 *    leading dimension a multiple of 8 elements and every base pointer 16-byte aligned, bf16)
 *    are supported, not errors.  A bf16 layer whose FACTORS are stored with other leading dimensions
 *    (an unquantized rank stored packed) still runs on the tensor cores: its factors are copied into
 *    the workspace with padded rows (lrd_linear_workspace_bytes accounts for it).  Activations with
 *    such leading dimensions, bases off a 16-byte boundary and fp32 take a slower general path.
 *  - Devices other than compute capability 10.x return LRD_ERR_ARCH.  There is no CPU path.
 */
#ifndef LRD_H_
#define LRD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LRD_OK = 0,
    LRD_ERR_INVALID_ARG = 1,  /* NULL where a pointer is required, non-positive size, bad enum, ld too small */
    LRD_ERR_BAD_RANK = 2,     /* r < 1 or r > min(K, N); no multiple fits in lrd_rank_quantize */
    LRD_ERR_ALIGNMENT = 3,    /* a base pointer is not aligned to its element size / workspace not 256-B aligned */
    LRD_ERR_WORKSPACE = 4,    /* workspace NULL or too small */
    LRD_ERR_UNSUPPORTED = 5,  /* convolution geometry other than k = 3, stride 1, pad 1 */
    LRD_ERR_ARCH = 6,         /* current device is not sm_100 */
    LRD_ERR_CUDA = 7,         /* a CUDA runtime / driver call failed */
    LRD_ERR_TIMEOUT = 8,      /* a bounded device-side wait ran out (see lrd_check_device_status) */
    LRD_ERR_TOO_LARGE = 9     /* a size exceeds the fixed limit of an entry point that brings its own scratch */
} lrd_status_t;

typedef enum { LRD_F32 = 0, LRD_BF16 = 1 } lrd_dtype_t;

/* Which factor of a two-factor layer is frozen this step (Section 2.2, Algorithm 2). */
typedef enum { LRD_FREEZE_NONE = 0, LRD_FREEZE_U = 1, LRD_FREEZE_V = 2 } lrd_freeze_t;

/* Which group of a Tucker-2 layer is frozen: both 1x1 factors (A, Bm) or the core G. */
typedef enum { LRD_TK_FREEZE_NONE = 0, LRD_TK_FREEZE_FACTORS = 1, LRD_TK_FREEZE_CORE = 2 } lrd_tucker_freeze_t;

typedef enum { LRD_ROUND_UP = 0, LRD_ROUND_DOWN = 1, LRD_ROUND_NEAREST = 2 } lrd_round_t;

/* Bits returned by lrd_linear_bwd_plan. */
enum {
    LRD_PLAN_DZ = 1, LRD_PLAN_DX = 2, LRD_PLAN_DU = 4, LRD_PLAN_DB = 8, LRD_PLAN_DV = 16,
    LRD_PLAN_NEEDS_Z = 32, LRD_PLAN_NEEDS_X = 64
};

/* Execution path selector for lrd_set_path (testing and measurement). */
typedef enum {
    LRD_PATH_AUTO = 0,     /* library chooses */
    LRD_PATH_GENERAL = 1,  /* fp32-FMA kernels for every shape and alignment */
    LRD_PATH_UNFUSED = 2,  /* tensor-core GEMMs, rank-r intermediate through the workspace */
    LRD_PATH_FUSED = 3     /* fused tensor-core chain where the shape allows, else UNFUSED */
} lrd_path_t;

typedef struct {
    int64_t M, K, N, r;             /* tokens, inputs, outputs, rank */
    int64_t ldx, ldv, ldu, ldy, ldz; /* leading dimensions of X/dX, V/dV, U/dU, Y/dY, Z_save; 0 = packed */
    int32_t dtype;                  /* lrd_dtype_t of every tensor of the layer */
} lrd_linear_desc_t;

typedef struct {
    int64_t B, H, W, C, S, r1, r2;  /* NHWC activations [B][H][W][C] -> [B][H][W][S] */
    int64_t k, stride, pad;         /* k x k core: k odd, 1..7; stride 1 or 2 (on the core); pad = (k - 1) / 2.
                                     * The output is [B][Ho][Wo][S] with Ho = (H - 1) / stride + 1, Wo likewise.
                                     * k = 3, stride = 1 runs the core on the tensor-core kernels (bf16, shapes
                                     * permitting); every other geometry runs it on the general fp32-FMA kernels.
                                     * Anything else: LRD_ERR_UNSUPPORTED. */
    int32_t dtype;
} lrd_tucker2_desc_t;

/* ---- host-only helpers (no device, no stream) ------------------------------------------ */

/* Rank quantization (Section 2.1, "Rank Optimization": ranks whose dimensions suit the hardware,
 * e.g. 257 -> 256).  Rounds r to a multiple of `multiple` (UP: ceiling, DOWN: floor, NEAREST: ties
 * up), then clamps to [multiple, largest multiple <= min(K, N)].  Returns the rank, or the
 * negated lrd_status_t (-LRD_ERR_INVALID_ARG for non-positive arguments or a bad mode,
 * -LRD_ERR_BAD_RANK when no multiple fits below min(K, N)). */
int64_t lrd_rank_quantize(int64_t r, int64_t multiple, lrd_round_t mode, int64_t K, int64_t N);

/* Sequential freezing (Algorithm 2).  Two-factor layers: even epoch -> the first-applied
 * sub-layer L_r(0) = V is frozen, odd epoch -> L_r(1) = U.  Tucker-2 layers: even epoch ->
 * L_r(0), L_r(2) (the 1x1 factors) frozen, odd epoch -> L_r(1) (the core).  e < 0 is treated by
 * its parity. */
lrd_freeze_t lrd_freeze_for_epoch(int64_t e);
lrd_tucker_freeze_t lrd_tucker_freeze_for_epoch(int64_t e);

/* The products lrd_linear_bwd runs under a freeze mask (Section 2.2: a frozen sub-layer passes the
 * gradient through but gets no weight gradient), as LRD_PLAN_* bits; 0 for a bad mask. */
uint32_t lrd_linear_bwd_plan(lrd_freeze_t freeze);

/* Algorithm 1 (rank search on a measured step-time curve), host only.  t[i] is the measured step time
 * of the layer decomposed at rank R_min + i, i = 0 .. n-1 (so t[n-1] belongs to the starting rank R);
 * T_orig is the step time of the undecomposed layer.  The paper's difference t(r) - t(r-1) refers, with
 * r running downward, to a time not yet measured; the reading taken here: delta(r) = t(r+1) - t(r) for
 * R_min <= r < R is the time saved by stepping down to r, R_opt is the first local maximum of delta met
 * scanning down from R-1 (strictly above both neighbours and above zero; an end point has one neighbour),
 * and with no such peak the global maximum (largest r on ties).
 * min_rel_drop >= 0: on a measured curve every wiggle of the timer is a local maximum of the difference, so a
 * peak (and the fallback maximum) counts only if its drop is at least min_rel_drop * t(r); pass a multiple of the
 * timer's relative spread (Section 2.1's example, 257 -> 256, is a drop of 15 %).  With a positive threshold and
 * no drop that large, R_opt = R.  0 is the plain reading.
 * *use_decomposed (nullable) receives 1 when t(R_opt) < T_orig (the algorithm's closing test: keep the
 * original layer otherwise), else 0.  Returns R_opt, or -(lrd_status_t) for a null curve, n < 1, R_min < 1
 * or a negative threshold.  `t` is host memory. */
int64_t lrd_rank_search(const double* t, int64_t n, int64_t R_min, double T_orig, double min_rel_drop, int* use_decomposed);

/* The quantization multiple a measured curve shows (Section 2.1, "Rank Optimization": which ranks are efficient is
 * a property of the device): the greatest common divisor of the ranks r whose drop t(r+1) - t(r) is positive and at
 * least min_rel_drop * t(r); 1 when there is none.  Same arguments and errors as lrd_rank_search. */
int64_t lrd_rank_multiple(const double* t, int64_t n, int64_t R_min, double min_rel_drop);

/* Starting ranks of the search, host only.  lrd_svd_rank: the largest r with r (C + S) <= C S / alpha (a C x S
 * matrix as two factors at compression ratio alpha).  lrd_tucker_rank: Eq. 5, r1 for a [S, C, k, k] kernel at
 * ratio alpha with r2 = beta r1 (both truncated, as the paper's [512, 512, 3, 3] -> 309 example fixes); *r2
 * (nullable) receives r2.  lrd_tucker_rank_min: Eq. 6, the lower end of the search = Eq. 5 at alpha + 1.
 * Negative (lrd_status_t) on non-positive arguments. */
int64_t lrd_svd_rank(int64_t C, int64_t S, double alpha);
int64_t lrd_tucker_rank(int64_t C, int64_t S, int64_t k, double alpha, double beta, int64_t* r2);
int64_t lrd_tucker_rank_min(int64_t C, int64_t S, int64_t k, double alpha, double beta);

/* The undecomposed 3 x 3 convolution (stride 1, zero padding 1, NHWC; kernel Wk[S][3][3][C]) that a Tucker-2 layer
 * replaces (Eq. 4): the comparison layer of the convolutional workloads and the T of Algorithm 1's closing test.
 * Forward Y = conv(X, Wk); backward dX (nullable: skipped) and dW.  Same conventions as the other entry points;
 * the workspace holds the split partial sums of the filter gradient. */
size_t lrd_conv3x3_workspace_bytes(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype);
lrd_status_t lrd_conv3x3_fwd(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype, const void* X, const void* Wk,
                             void* Y, void* cuda_stream);
lrd_status_t lrd_conv3x3_bwd(int64_t B, int64_t H, int64_t W, int64_t C, int64_t S, int dtype, const void* dY, const void* X,
                             const void* Wk, void* dX, void* dW, void* workspace, size_t workspace_bytes, void* cuda_stream);

const char* lrd_status_string(lrd_status_t s);

/* Process-wide choice of execution path (default LRD_PATH_AUTO).  Returns LRD_ERR_INVALID_ARG
 * for an unknown value.  Not thread-safe against concurrent launches. */
lrd_status_t lrd_set_path(lrd_path_t path);

/* Launch-shape overrides of the fused chain kernel, for measurement sweeps (no counterpart in the
 * paper): blocks per cluster (1, 2 or 4), 64-deep k-blocks per pipeline stage of the first product
 * (1..4), column-chunk width of the second product (64, 128, 192 or 256).  0 = automatic (the default).
 * A shape the override makes infeasible falls back to the unfused products.  Process-wide, not
 * thread-safe against concurrent launches.  Returns LRD_ERR_INVALID_ARG for values outside the lists. */
lrd_status_t lrd_chain_tuning(int cluster_blocks, int kblocks_per_stage, int chunk_columns);

/* The fused chain also runs on pairs of SMs (a cluster of 2 S blocks owns 256 rows; the two blocks of a
 * pair share every MMA and each loads half of the weights): it is taken automatically for layers of more than
 * 128 rows whose rank splits into S slices of whole 32-column groups.  Overrides for measurement sweeps and
 * tests (no counterpart in the paper): blocks_per_mma 1 = single-block chain only, 2 = pairs wherever the shape
 * allows (else the unfused products), 0 = automatic; pairs_per_cluster S (1..4), 64-deep k-blocks per
 * pipeline stage of the first product (1..4), column-chunk width of the second product (64, 128, 192, 256);
 * 0 = automatic.  Process-wide, test-only: not thread-safe against concurrent launches.  Returns
 * LRD_ERR_INVALID_ARG for values outside the lists. */
lrd_status_t lrd_chain_pair_tuning(int blocks_per_mma, int pairs_per_cluster, int kblocks_per_stage, int chunk_columns);

/* Launch-shape override of the unsplit products (the dense layer's forward and input gradient, the two
 * products of an unfused decomposed layer), for measurement sweeps (no counterpart in the paper):
 * blocks per MMA, 1 (every SM works on its own 128-row tiles) or 2 (pairs of SMs share 256-row tiles and
 * each loads half of the B operand); 0 = automatic (the default).  2 is ignored for products of at most
 * 128 rows.  Process-wide, not thread-safe against concurrent launches.  Returns LRD_ERR_INVALID_ARG for
 * other values. */
lrd_status_t lrd_gemm_tuning(int blocks_per_mma);

/* lrd_tucker2_bwd enqueues its independent launches side by side (the dB + dbias product from the start, the
 * core's filter gradient once dZ2 exists, both on streams the library owns; the data path and dA on the
 * caller's stream, which waits for the others before the call returns) when `on` is non-zero - the default -
 * and one after the other on the caller's stream when it is zero.  Same results either way.  With the default,
 * make a host thread's first backward call on a device outside any stream capture (it creates that thread's
 * streams).  The switch is process-wide; no counterpart in the paper. */
lrd_status_t lrd_tucker2_overlap(int on);

/* Synchronises the current device, then reports and clears the device-side timeout flag:
 * LRD_OK, LRD_ERR_TIMEOUT, or LRD_ERR_CUDA if the synchronisation itself failed. */
lrd_status_t lrd_check_device_status(void);

/* Debug mode (no counterpart in the paper).  With the environment variable LRD_DEBUG set (to anything but 0) when the
 * library is loaded, every compute entry point below waits for the work it has enqueued and returns what went wrong
 * in it: LRD_ERR_CUDA for a launch or execution error, LRD_ERR_TIMEOUT for a bounded device wait that ran out (the
 * flag is cleared, as by lrd_check_device_status).  A call whose stream is being captured is left alone.  Off by
 * default, where the library never synchronises and errors surface at lrd_check_device_status(). */

/* Self-test of the bounded device-side wait (no counterpart in the paper): enqueues one small block that waits,
 * through the same routine and with the same limit as every pipeline wait of the library's kernels, on a barrier
 * nothing ever arrives at.  The wait runs out after a second or so, raises the timeout flag and the block
 * returns in order (nothing is in flight, no tensor memory is held).  The next lrd_check_device_status() returns
 * LRD_ERR_TIMEOUT once, the one after LRD_OK, and every other entry point keeps working.  Returns
 * LRD_ERR_ARCH / LRD_ERR_CUDA as the other entry points do. */
lrd_status_t lrd_selftest_wait_timeout(void* cuda_stream);

/* Number of kernels this library has enqueued since it was loaded (host-side counter, all
 * streams; memset nodes of zero-filled gradients are not counted).  For launch accounting. */
uint64_t lrd_launch_count(void);

/* Scratch bytes lrd_linear_fwd (is_bwd = 0), lrd_linear_bwd (is_bwd = 1) or lrd_linear_bwd_accumulate
 * (is_bwd = 2) needs for this layer and mask, for whichever path the library may take.  0 on a bad descriptor. */
size_t lrd_linear_workspace_bytes(const lrd_linear_desc_t* desc, lrd_freeze_t freeze, int is_bwd);
size_t lrd_tucker2_workspace_bytes(const lrd_tucker2_desc_t* desc, lrd_tucker_freeze_t freeze, int is_bwd);
size_t lrd_dense_workspace_bytes(const lrd_linear_desc_t* desc, int is_bwd);

/* ---- decomposed fully connected layer (Section 2, Fig. 1; freezing: Section 2.2) --------- */

/* Forward: Z = X V, Y = Z U^T + bias.
 *   X[M x K] (ldx), V[K x r] (ldv), U[N x r] (ldu), bias[N] or NULL, Y[M x N] (ldy) out.
 *   Z_save[M x r] (ldz) out: the rank-r intermediate kept for dU.  Required (non-NULL) unless
 *   freeze == LRD_FREEZE_U, in which case it must be NULL and Z is never written to memory the
 *   caller sees.  In bf16, Z is rounded to bf16 once between the two products. */
lrd_status_t lrd_linear_fwd(const lrd_linear_desc_t* desc, const void* X, const void* V, const void* U,
                            const void* bias, void* Y, void* Z_save, lrd_freeze_t freeze,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Backward: dZ = dY U, dX = dZ V^T always (dX = NULL skips the second product);
 *   U not frozen: dU[N x r] = dY^T Z_save, dbias[N] = column sums of dY (dbias may be NULL);
 *   V not frozen: dV[K x r] = X^T dZ.
 * A frozen factor's weight-gradient product is never launched; if its gradient pointer (and, for
 * U, dbias) is non-NULL it is filled with zeros.  X may be NULL when V is frozen, Z_save may be
 * NULL when U is frozen; the gradient pointer of an unfrozen factor must be non-NULL. */
lrd_status_t lrd_linear_bwd(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* V,
                            const void* U, const void* Z_save, void* dX, void* dU, void* dV, void* dbias,
                            lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The backward pass in two calls, for callers that schedule the weight gradients themselves (Section 2.2: with one
 * factor frozen only the other one's product is left, and nothing later in the backward pass of the network waits
 * for it): lrd_linear_bwd_data forms dZ = dY U and dX = dZ V^T (dX nullable) and leaves dZ in the workspace when V is
 * unfrozen; lrd_linear_bwd_weights forms the unfrozen factor's gradients (dU = dY^T Z_save with dbias, dV = X^T dZ),
 * zero-fills the frozen one's buffers, and may run on another stream beside the next layer's data call.  When V is
 * unfrozen the weights call reads the dZ its layer's data call left in the SAME workspace: order it after that call
 * (same stream, or an event) and let nothing else use the workspace in between.  Together the two calls do what
 * lrd_linear_bwd does, with launch shapes chosen to leave room for each other: the data call takes the fused chain on
 * pairs of SMs where the shape allows (fewer blocks), the weights call splits its reduction over the tokens into fewer,
 * larger shares (blocks in clusters of 2, which find free SMs next to a running data call, instead of clusters of up
 * to 8).  The same products are therefore added in a different grouping: results agree with lrd_linear_bwd within
 * rounding; repeated calls give identical bits.  Arguments, layouts and errors as there. */
lrd_status_t lrd_linear_bwd_data(const lrd_linear_desc_t* desc, const void* dY, const void* V, const void* U, void* dX,
                                 lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream);
lrd_status_t lrd_linear_bwd_weights(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* Z_save, void* dU,
                                    void* dV, void* dbias, lrd_freeze_t freeze, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream);

/* Backward with gradient accumulation: as lrd_linear_bwd, but the unfrozen factor's dU, dbias and dV are ADDED to
 * what the buffers hold (gradient accumulation over micro-batches) instead of overwritten; dX is overwritten as
 * usual.  A frozen factor's gradient buffers are not touched at all (its gradient is zero), and may be NULL.
 * This step's gradients are formed in scratch at the end of the workspace, rounded to the storage type, then
 * added in fp32 and rounded once more.  Workspace: lrd_linear_workspace_bytes(desc, freeze, 2).  The paper's
 * Section 2.2 trains with plain steps; accumulation is a convenience with no counterpart there. */
lrd_status_t lrd_linear_bwd_accumulate(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* V,
                                       const void* U, const void* Z_save, void* dX, void* dU, void* dV, void* dbias,
                                       lrd_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- groups of independent decomposed layers -------------------------------------------------------
 * The n layers of a group depend on nothing the others produce (the query, key and value projections
 * of an attention block, which read the same X, are the model case; the paper's Section 2 treats every
 * layer on its own, so grouping is a launch-level matter with no counterpart there).  Layer i is given
 * by descs[i] and the i-th entries of the pointer arrays, each with the meaning, layout and rules of the
 * same argument of lrd_linear_fwd / lrd_linear_bwd; the arrays themselves are HOST arrays of n entries.
 * `bias`, `Z_save`, and in the backward `X`, `Z_save`, `dX`, `dU`, `dV`, `dbias` may be NULL as a whole
 * where the single-layer call allows NULL for every layer.  Inputs may be shared between layers;
 * outputs and workspaces must not overlap one another (every layer writes its own dX: the caller adds
 * them up where the layers share X).  One mask applies to the whole group.
 *
 * The layers are enqueued side by side: layer 0 on `cuda_stream`, the others on streams the library
 * owns (created on first use, one set per host thread and device, never freed), which start after the work already in
 * `cuda_stream` and which `cuda_stream` waits for before the call returns - so to the caller the group
 * behaves like n single-layer calls on `cuda_stream`, and it may be captured into a CUDA graph.  Each
 * launch is shaped for 1/n of the SMs.  In the backward, a layer's dU (+ dbias) product runs beside its
 * data chain.  Z_save, dU, dV and dbias have the bits of the single-layer calls; Y and dX agree with them to
 * rounding (the fused kernel sums over the rank in an order that depends on its cluster size, which follows
 * the launch's share of the SMs).  n = 1 is allowed (then only the dU overlap differs from lrd_linear_bwd).
 *
 * Errors: LRD_ERR_INVALID_ARG for n outside [0, LRD_MAX_GROUP] or a NULL required array; otherwise the
 * first failing layer's status.  All layers are validated before anything is enqueued.  Every host
 * thread has its own set of library streams, so groups may run from several threads at once.  Make a
 * thread's first group call on a device outside any stream capture (it creates that set). */
#define LRD_MAX_GROUP 8
lrd_status_t lrd_linear_group_fwd(int n, const lrd_linear_desc_t* descs, const void* const* X, const void* const* V,
                                  const void* const* U, const void* const* bias, void* const* Y, void* const* Z_save,
                                  lrd_freeze_t freeze, void* const* workspace, const size_t* workspace_bytes,
                                  void* cuda_stream);
lrd_status_t lrd_linear_group_bwd(int n, const lrd_linear_desc_t* descs, const void* const* dY, const void* const* X,
                                  const void* const* V, const void* const* U, const void* const* Z_save, void* const* dX,
                                  void* const* dU, void* const* dV, void* const* dbias, lrd_freeze_t freeze,
                                  void* const* workspace, const size_t* workspace_bytes, void* cuda_stream);

/* ---- the undecomposed layer, for comparison (the "original layer" of Algorithm 1) -------- */

/* Y = X W^T + bias with W[N x K] (leading dimension desc->ldv; desc->r, ldu, ldz ignored). */
lrd_status_t lrd_dense_fwd(const lrd_linear_desc_t* desc, const void* X, const void* W, const void* bias, void* Y,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);
/* dX = dY W (NULL skips), dW = dY^T X, dbias = column sums of dY (NULL skips). */
lrd_status_t lrd_dense_bwd(const lrd_linear_desc_t* desc, const void* dY, const void* X, const void* W, void* dX,
                           void* dW, void* dbias, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- bias gradient for callers that cannot allocate device memory --------------------------- */

/* The paper has no counterpart for this entry point; it exists for the sake of its callers.
 *
 * dbias[N] = column sums of dY[M x N] (leading dimension ldy, 0 = packed), the same quantity and the
 * same kernels as the dbias output of lrd_linear_bwd, but WITHOUT a workspace argument: the partial
 * sums go to a fixed 2 MiB array that lives inside the library's device image.  It is meant for code
 * that has no way to obtain scratch memory when it needs the result - for instance a plug-in that is
 * handed ready-made tensors by a framework whose allocator it must not call, a callback running where
 * cudaMalloc is forbidden, or a process whose memory pool is already fully committed.  The function
 * itself calls no cudaMalloc, cudaFree or any other allocating routine.
 *
 *  - Limit: N <= 8192 (the array holds 64 partial rows of that width); larger N returns
 *    LRD_ERR_TOO_LARGE and nothing is launched.  M is unlimited.  Every GPU on which the library is
 *    loaded carries the 2 MiB array until the process exits, whether or not this function is used.
 *  - First use on a device looks up the array's device address (one runtime query, cached per
 *    device).  Make that first call with the intended device current and before starting any stream
 *    capture; later calls do no set-up.
 *  - All calls share the one array.  Nothing in it needs clearing between calls (every partial that
 *    is read has been written by the same call), but two calls that can run at the same time on the
 *    GPU - different streams, or different host threads - would overwrite each other's partial sums:
 *    keep calls to this function ordered with respect to each other.
 *  - dY and dbias are device pointers of type `dtype`; the work is enqueued on `cuda_stream`. */
lrd_status_t lrd_bias_grad_noalloc(const void* dY, int64_t ldy, int64_t M, int64_t N, void* dbias,
                                   lrd_dtype_t dtype, void* cuda_stream);

/* ---- Tucker-2 decomposed k x k convolution (Eq. 4, Fig. 1) -------------------------------- */

/* Forward: Z1 = X A (1x1, C -> r1); Z2 = conv(Z1, G) (cross-correlation, k x k, the layer's stride, zero pad
 * (k - 1) / 2, r1 -> r2: output pixel (ho, wo) reads input pixels (ho stride + kh - pad, wo stride + kw - pad));
 * Y = Z2 Bm^T + bias (1x1, r2 -> S).  NHWC: X[B][H][W][C], Y[B][Ho][Wo][S]; A[C x r1], G[r2][k][k][r1],
 * Bm[S x r2], bias[S] or NULL.
 *   Z1_save[B][H][W][r1]: required unless freeze == LRD_TK_FREEZE_CORE (then must be NULL);
 *   Z2_save[B][Ho][Wo][r2]: required unless freeze == LRD_TK_FREEZE_FACTORS (then must be NULL). */
lrd_status_t lrd_tucker2_fwd(const lrd_tucker2_desc_t* desc, const void* X, const void* A, const void* G,
                             const void* Bm, const void* bias, void* Y, void* Z1_save, void* Z2_save,
                             lrd_tucker_freeze_t freeze, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Backward (dY[B][Ho][Wo][S]): dZ2 = dY Bm; dZ1 = conv^T(dZ2, G); dX[B][H][W][C] = dZ1 A^T (NULL skips);
 *   factors not frozen: dB[S x r2] = dY^T Z2_save, dA[C x r1] = X^T dZ1, dbias = column sums of dY;
 *   core not frozen:    dG[o][kh][kw][i] = sum_p dZ2[p][o] Z1_save[p stride + (kh, kw) - pad][i] (p: output pixels).
 * Frozen groups: product not launched, non-NULL gradient pointers are zero-filled. */
lrd_status_t lrd_tucker2_bwd(const lrd_tucker2_desc_t* desc, const void* dY, const void* X, const void* A,
                             const void* G, const void* Bm, const void* Z1_save, const void* Z2_save, void* dX,
                             void* dA, void* dG, void* dB, void* dbias, lrd_tucker_freeze_t freeze,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LRD_H_ */
