/*
 * mixgcn.h -- C ABI of libmixgcn.so: the single-GPU (sm_100a) hot path of full-graph GCN
 * training as the MixGCN paper states it -- per layer, sparse neighbour aggregation with the
 * propagation matrix followed by the dense node update (Eq. 3; Algorithm 2), then the loss,
 * the backward pass and the weight update (Algorithm 2, last two lines of the iteration).
 *
 * Conventions
 *  - Node-major storage: X = H^T is n x d, row-major fp32, with a leading dimension `ld`
 *    (in elements) that is a multiple of 4 and >= d; every matrix pointer is 16-byte aligned.
 *    Pad columns [d, ld) are never read as data; the library writes zeros or leaves them.
 *    Weights W_l = [W^(l)]^T are d_in x d_out row-major, dense (ld = d_out), fp32.
 *  - "device" pointers must be ordinary device memory of the context's GPU; "host" pointers
 *    are ordinary host memory.  The caller owns every buffer passed in; the library owns only
 *    the opaque context (status word, workspace, two internal streams) and graph objects.
 *  - All compute calls are asynchronous on the caller's stream (`stream` is a cudaStream_t
 *    passed as void*; NULL = legacy default stream) unless stated otherwise.
 *  - Every function returns a mixgcn_status and never throws, aborts or traps.  On an error
 *    detected on the host nothing is launched and outputs are untouched; the message is kept
 *    per thread in mixgcn_last_error().  Conditions only the device can see (empty train
 *    mask, label out of range) are written to the context's device status word, the kernel
 *    produces zeros, and mixgcn_ctx_poll_status() reports them.
 *  - Deterministic: no atomics on floating-point data; the same inputs give bitwise the same
 *    outputs on every call.
 *  - Threads: a context and the objects created from it (graphs, row plans) keep scratch buffers
 *    and options in the context; use them from one host thread at a time.  Different contexts are
 *    independent.
 */
#ifndef MIXGCN_H_
#define MIXGCN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MIXGCN_OK = 0,
    MIXGCN_EINVAL = 1,        /* null / negative / misaligned argument */
    MIXGCN_ENOMEM = 2,        /* device or host allocation failed */
    MIXGCN_ECUDA = 3,         /* a CUDA runtime call failed; see mixgcn_last_error() */
    MIXGCN_EUNSUPPORTED = 4,  /* valid request this build cannot serve */
    MIXGCN_EBADGRAPH = 5,     /* node id out of range, unsorted CSR, n or nnz too large */
    MIXGCN_ETIMEOUT = 6,      /* a bounded device-side wait gave up */
    MIXGCN_EDEVICE = 7        /* a kernel reported bad data (empty mask, bad label) */
} mixgcn_status;

typedef struct mixgcn_ctx mixgcn_ctx;
typedef struct mixgcn_graph mixgcn_graph;
typedef struct mixgcn_rowplan mixgcn_rowplan;   /* see mixgcn_rowplan_create */

const char* mixgcn_status_string(mixgcn_status s);
const char* mixgcn_last_error(void); /* thread-local, never NULL */

/* Create / destroy a context bound to CUDA device `device`.  Allocates the status word and
 * two internal streams.  Destroy synchronises the device. */
mixgcn_status mixgcn_ctx_create(mixgcn_ctx** out, int device);
mixgcn_status mixgcn_ctx_destroy(mixgcn_ctx* ctx);

/* Pre-size the context's workspace (split-K partials, column-sum partials, loss partials) so
 * that later calls allocate nothing.  Without it the workspace grows on demand (a
 * cudaMalloc inside the first call that needs more). */
mixgcn_status mixgcn_ctx_reserve(mixgcn_ctx* ctx, int64_t bytes);

/* Synchronises the context's device, reads and clears the device status word.
 * Returns MIXGCN_OK, MIXGCN_EDEVICE or MIXGCN_ETIMEOUT; *code (nullable) receives the raw
 * code: 0 none, 1 empty train mask, 2 label out of range, 3 bounded wait expired,
 * 4 gout_row_count does not match gout_row_mask, 5 (bounds-checked debug build only) a kernel met an index
 * outside its range -- mixgcn_last_error() then names the kind of index and its value. */
mixgcn_status mixgcn_ctx_poll_status(mixgcn_ctx* ctx, int32_t* code);

/* The bounds-checked debug build (libmixgcn_debug.so: the same sources compiled with -DMIXGCN_DEBUG_BOUNDS; no
 * counterpart in the paper -- it stands in for a memory checker).  Every index a kernel takes from memory -- an
 * aggregation's column ids, the rows and entry ranges of its schedule records, its segment tables, the row lists
 * of the row-sparse backward -- is tested before it addresses anything; a bad one is recorded (code 5 above), the
 * access is skipped, the kernel finishes and the context stays usable.  The release build has none of these tests.
 * mixgcn_build_info: *debug_bounds (nullable) receives 1 in that build, 0 otherwise.
 * mixgcn_debug_poke_col: the test hook of those checks, MIXGCN_EUNSUPPORTED in the release build: synchronises the
 * device and overwrites column id `entry` (in [0, nnz), else MIXGCN_EINVAL) of the graph's forward CSR with
 * `value`; *old_value (nullable, host) receives what was there. */
mixgcn_status mixgcn_build_info(int32_t* debug_bounds);
mixgcn_status mixgcn_debug_poke_col(mixgcn_graph* g, int64_t entry, int32_t value, int32_t* old_value);

/* Tuning options.  MIXGCN_OPT_SPMM_SLICE_COLS: width of the feature-column slices an aggregation is
 * processed in (Algorithm 2's p:q-1 column ranges on one GPU): 0 = slices of 256 columns (default:
 * the two-float4-per-lane kernels keep four CTAs per SM; measured fastest at width 1024); otherwise
 * a multiple of 4 in [4, 1024].  Narrow slices shrink the part of the input
 * that must stay in the L2 at the price of re-reading the index once per slice; results do not
 * depend on the slicing. */
#define MIXGCN_OPT_SPMM_SLICE_COLS 1
/* MIXGCN_OPT_LOSS_TRAIN_ROWS_ONLY: 0 (default) = mixgcn_loss_softmax_xent as documented; 1 = rows
 * outside the train mask are not looked at: their logits are not read, their dlogits rows are
 * left UNCHANGED (not zeroed) and pred, if given, receives -1 there.  Loss, n_correct and the
 * train rows of dlogits are unchanged.  For use with MIXGCN_LAYER_OUT_ROWS_ONLY and a row-sparse
 * backward pass, which read train rows only.  2 = every row's logits are read (pred for all nodes) but
 * the dlogits rows of non-train nodes are left UNCHANGED instead of zeroed: for a backward pass that
 * reads train rows only (gout_plan, or gout_row_mask with a count below n/4 in agg-first order). */
#define MIXGCN_OPT_LOSS_TRAIN_ROWS_ONLY 2
/* Test hooks of the bounded device-side waits (the failure-detection path), both 0 by default.
 * MIXGCN_OPT_DEBUG_WAIT_LIMIT: > 0 = number of polls after which a wait inside the tensor-core kernels
 * gives up (default about four million).  MIXGCN_OPT_DEBUG_DROP_LOAD: 1 = the next tensor-core products
 * in the K-major form leave the first stage of every CTA unfilled, so that the wait on it runs out: the
 * kernel records code 3 in the status word, frees its tensor memory and returns with C undefined;
 * mixgcn_ctx_poll_status then gives MIXGCN_ETIMEOUT.  Nothing traps, spins without limit or faults. */
#define MIXGCN_OPT_DEBUG_WAIT_LIMIT 3
#define MIXGCN_OPT_DEBUG_DROP_LOAD 4
/* MIXGCN_OPT_GEMM_CTA_PAIRS: 1 (default) = wide and deep K-major products (N >= 512, K >= 512, M >= 4096)
 * run on pairs of CTAs that share one 256 x 256 tile (tcgen05 .cta_group::2); 0 = every product on single
 * CTAs with 128 x 256 tiles.  Same results up to the order of fp32 accumulation inside the tensor core. */
#define MIXGCN_OPT_GEMM_CTA_PAIRS 5
mixgcn_status mixgcn_ctx_set_option(mixgcn_ctx* ctx, int32_t option, int64_t value);

/* Which kernel served the dense products of this context since it was created: counts[0] fp32 FMA
 * kernel, counts[1] tcgen05 with TF32 operands, counts[2] tcgen05 with BF16 operands; counts[3] = how
 * many of the tcgen05 products ran on CTA pairs.  A TF32 or BF16 request whose shape or alignment the
 * tensor-core kernels do not take is served by the next kernel down that list (never a lower precision
 * than asked for); these counters make that visible. */
mixgcn_status mixgcn_ctx_gemm_paths(const mixgcn_ctx* ctx, int64_t counts[4]);

/* Per-phase profiling.  While enabled the library brackets every kernel it launches with
 * CUDA events on the launching stream.  mixgcn_ctx_profile_read synchronises and returns, for
 * each phase, accumulated milliseconds and launch counts since the last read, then resets.
 * Phases: 0 spmm (dense input), 1 gemm, 2 elementwise/epilogue, 3 loss, 4 adam, 5 graph build,
 * 6 spmm with a row-sparse input.
 * `launches_total` (nullable) receives the number of kernels launched by this context since
 * creation (counted whether or not profiling is enabled). */
#define MIXGCN_N_PHASES 7
mixgcn_status mixgcn_ctx_profile_enable(mixgcn_ctx* ctx, int enable);
mixgcn_status mixgcn_ctx_profile_read(mixgcn_ctx* ctx, double ms[MIXGCN_N_PHASES],
                                      int64_t launches[MIXGCN_N_PHASES], int64_t* launches_total);

/* ------------------------------------------------------------------------------------------
 * Graph: the propagation matrix A_hat = D^-1/2 (A + I) D^-1/2 with D_uu = sum_v (A+I)_uv
 * (Section 2.1), kept in CSR (the adjacency index format of Section 3.2.1) together with the
 * CSR of its transpose (aliased when the stored matrix is symmetric) and a degree-sorted row
 * schedule for the aggregation kernels.
 * ------------------------------------------------------------------------------------------ */
#define MIXGCN_GRAPH_SYMMETRISE     1u /* store (v,u) for every (u,v) */
#define MIXGCN_GRAPH_ADD_SELF_LOOPS 2u /* the "+ I" of Section 2.1 */
#define MIXGCN_GRAPH_EDGES_ON_DEVICE 4u /* src/dst (or rowptr/col) are device pointers */
/* Values of the stored matrix.  Default: the symmetric normalisation of Section 2.1,
 * val_uv = 1/sqrt(deg_u deg_v).  The paper's evaluation also names GraphSAGE and GIN without defining
 * them; their textbook aggregation matrices are offered on the same structure and kernels:
 * NORM_ROW  val_uv = 1 / (entries in row u): the row mean (GraphSAGE's mean aggregator); A_hat^T then
 *           differs from A_hat even on a symmetric structure, and the library keeps its own copy;
 * NORM_NONE val_uv = 1: the plain sum (GIN's sum aggregator; its (1 + eps) self term is the
 *           aggregation epilogue's residual).  At most one of the two. */
#define MIXGCN_GRAPH_NORM_ROW  8u
#define MIXGCN_GRAPH_NORM_NONE 16u

/* Build from an edge list of m pairs (src[e], dst[e]) meaning entry (src, dst) of A.
 * Input self-loops are dropped, duplicates collapse (A is binary), then one diagonal entry
 * per node is added if ADD_SELF_LOOPS.  rowptr is int64[n+1], col int32[nnz] ascending per
 * row, val fp32: dinv_u = 1/sqrt(deg_u) (IEEE sqrt then IEEE reciprocal, each rounded to
 * fp32), val_uv = dinv_u * dinv_v (one rounded multiply), deg_u = entries in row u.
 * Requires 0 < n < 2^31 - 1 and 0 <= m; ids in [0, n) else MIXGCN_EBADGRAPH.
 * Synchronises before returning.  *out is owned by the caller until mixgcn_graph_destroy. */
mixgcn_status mixgcn_graph_create(mixgcn_ctx* ctx, int64_t n, int64_t m, const int32_t* src,
                                  const int32_t* dst, uint32_t flags, mixgcn_graph** out);

/* Build from the CSR structure of A + I (or of any binary matrix): validates monotone rowptr,
 * ids in range and strictly ascending columns per row (else MIXGCN_EBADGRAPH), then
 * normalises as above.  Only EDGES_ON_DEVICE is honoured in flags.  Synchronises. */
mixgcn_status mixgcn_graph_create_from_csr(mixgcn_ctx* ctx, int64_t n, const int64_t* rowptr,
                                           const int32_t* col, uint32_t flags, mixgcn_graph** out);

mixgcn_status mixgcn_graph_info(const mixgcn_graph* g, int64_t* n, int64_t* nnz,
                                int32_t* max_deg, int32_t* symmetric);

/* Copy the CSR (transposed != 0: of A_hat^T) to HOST arrays; any output may be NULL.
 * rowptr int64[n+1], col int32[nnz], val fp32[nnz], deg int32[n] (entries per row of the
 * non-transposed matrix), dinv fp32[n].  Synchronises. */
mixgcn_status mixgcn_graph_export(const mixgcn_graph* g, int transposed, int64_t* rowptr,
                                  int32_t* col, float* val, int32_t* deg, float* dinv);

/* Copy the degree-sorted row schedule to HOST: perm int32[n] lists row ids by descending
 * entry count (ties by ascending id). */
mixgcn_status mixgcn_graph_export_schedule(const mixgcn_graph* g, int transposed, int32_t* perm);

/* A graph may be used only while its context exists; it may be destroyed after it. */
mixgcn_status mixgcn_graph_destroy(mixgcn_graph* g);

/* Node reordering for the fine-grain pipeline (Section 3.2.2).
 * mixgcn_graph_bandwidth: b = max over stored entries (u,v) of p_v - p_u, where p is the position
 *   of a node in the processing sequence `order` (host int32[n], order[k] = node at position k;
 *   NULL = the identity).  Runs on the device; synchronises.
 * mixgcn_graph_rcm: the reverse Cuthill-McKee order of a symmetric graph into `order` (host
 *   int32[n]): components start from the unvisited node with the fewest entries (lowest id on ties), a
 *   visited node appends its unvisited neighbours by increasing entry count (lowest id on ties), and
 *   the sequence is reversed.  Runs on the device as a level-synchronous breadth-first search (a
 *   level's nodes sorted by the position of their earliest-placed neighbour, then entry count, then id:
 *   the order a one-node-at-a-time queue gives); the paper's preprocessing is a CPU program.
 *   Synchronises (once per level).  MIXGCN_EUNSUPPORTED if not symmetric.
 * mixgcn_pipeline_stages: the stage count ceil(2n / (n - b)) of Proposition 3.5 (idleness is
 *   eliminated when (n - b) / (2n) >= 1 / s); MIXGCN_EINVAL when b >= n.
 * mixgcn_graph_create_permuted: a new graph in which node order[k] has become node k (same
 *   entries, relabelled); the caller permutes features, labels and masks the same way. */
mixgcn_status mixgcn_graph_bandwidth(const mixgcn_graph* g, const int32_t* order, int64_t* bandwidth);
mixgcn_status mixgcn_graph_rcm(const mixgcn_graph* g, int32_t* order);
mixgcn_status mixgcn_pipeline_stages(int64_t n, int64_t b, int64_t* stages);
mixgcn_status mixgcn_graph_create_permuted(mixgcn_ctx* ctx, const mixgcn_graph* g, const int32_t* order,
                                           mixgcn_graph** out);

/* ------------------------------------------------------------------------------------------
 * Building blocks (device pointers).  The layer calls below are compositions of these.
 * ------------------------------------------------------------------------------------------ */

/* Epilogue applied to each output element y of an aggregation or an update, in this order:
 *   y += bias[j]                       if bias != NULL
 *   y  = max(y, 0)                     if relu
 *   y  = drop_mask[i*d+j] ? y*keep_scale : 0      if drop_mask != NULL   (uint8, dense n x d)
 *   y  = gate[i*ld_gate+j] > 0 ? y*gate_scale : 0 if gate != NULL        (fp32, n x d)
 * The gate form is the backward sampled aggregation of Eq. 4 (M = ReLU mask). */
typedef struct {
    const float* bias;
    int32_t relu;
    const uint8_t* drop_mask;
    float keep_scale;
    const float* gate;
    int64_t ld_gate;
    float gate_scale;
    /* y = y + residual_scale * residual[i*ld_residual + j], applied FIRST (before the bias), when
     * residual != NULL (fp32, n x d; may be the aggregation's own input, must not overlap its output).
     * Aggregation only (mixgcn_spmm, mixgcn_spmm_rowplan): it turns A_hat Y into (s I + A_hat) Y, the
     * form sum-aggregator layers with a weighted self term use (GIN's (1 + eps) h + sum of
     * neighbours; the paper names that architecture in its evaluation without defining it).
     * mixgcn_gemm rejects it. */
    const float* residual;
    int64_t ld_residual;
    float residual_scale;
    /* Bit-packed masks (the bitmap mask buffer of Section 3.2.1): n x ld words of 32 bits, bit (j & 31) of
     * word [i*ld + (j >> 5)] belongs to element (i, j); ld >= ceil(d / 32).
     *   gate_bits  (nullable) stands in for `gate` (which is then ignored): set bit = y*gate_scale, clear bit = 0.
     *   sign_bits  (nullable) is an OUTPUT: receives bit = (final y > 0) for every element, bits of columns
     *              >= d in a row's last word are cleared.  With relu this is the mask a later gate_bits reads
     *              -- 1 bit per element instead of re-reading the fp32 tensor.  Written by the kernel that
     *              produces y where it can, else by one more pass over the result.
     * K-major / plain products and aggregations only (mixgcn_gemm with trans_a = 1 rejects both). */
    const uint32_t* gate_bits;
    int64_t ld_gate_bits;
    uint32_t* sign_bits;
    int64_t ld_sign_bits;
} mixgcn_epilogue;

/* Neighbour aggregation Z = A_hat Y (transposed != 0: A_hat^T Y), n x w (Algorithm 2,
 * aggregation line; column slices as in its p:q-1 ranges are taken internally).
 * Y and Z must not overlap.  epi may be NULL.  Row sums are accumulated in fp32 in a fixed
 * order. */
mixgcn_status mixgcn_spmm(mixgcn_ctx* ctx, const mixgcn_graph* g, int transposed, int32_t w,
                          const float* Y, int64_t ldy, float* Z, int64_t ldz,
                          const mixgcn_epilogue* epi, void* stream);

/* Sampled aggregation (the paper's S-SpMM, Eq. 4): Z = (A_hat Y) (.) M for a binary output mask M held as
 * a BITMAP (the output mask buffer of Section 3.2.1): bit (j % 32) of word mask_bits[u * ld_bits + j / 32]
 * says whether output (u, j) is kept.  Masked outputs are written as zero and are not computed: a lane all
 * of whose output columns of a row are masked skips its gathers of that row's neighbours (on a GPU a
 * gather moves 16 bytes per lane, so whole 16-byte groups must be masked for a load to disappear; a 50 %
 * element mask removes few of them -- the call exists for parity with the paper's operation and for
 * masks with structure).  The mask is applied after the epilogue's other terms.  Other arguments as
 * mixgcn_spmm.  mixgcn_mask_pack builds a bitmap: bit (u, j) = (X == NULL or X[u*ldx + j] > 0) and
 * (bytes == NULL or bytes[u*w + j] != 0) -- the ReLU mask of an activation (backward form) and / or a
 * dropout byte mask (forward form); ld_bits >= ceil(w / 32) words per row. */
mixgcn_status mixgcn_spmm_sampled(mixgcn_ctx* ctx, const mixgcn_graph* g, int transposed, int32_t w,
                                  const float* Y, int64_t ldy, float* Z, int64_t ldz, const uint32_t* mask_bits,
                                  int64_t ld_bits, const mixgcn_epilogue* epi, void* stream);
mixgcn_status mixgcn_mask_pack(mixgcn_ctx* ctx, int64_t n, int32_t w, const float* X, int64_t ldx,
                               const uint8_t* bytes, uint32_t* bits, int64_t ld_bits, void* stream);

#define MIXGCN_PREC_FP32 0 /* fp32 FMA on the CUDA cores */
#define MIXGCN_PREC_TF32 1 /* tensor cores, TF32 operands, fp32 accumulate */
#define MIXGCN_PREC_BF16 2 /* tensor cores, BF16 operands (the fp32 operands rounded to nearest even),
                              fp32 accumulate, fp32 results */

/* Dense update GEMM  C = op(A) op(B)  with fp32 storage (Algorithm 2, update line, and its
 * two backward products).  op(A) is M x K, op(B) is K x N, C is M x N row-major with ldc.
 *   trans_a = 0: A is M x K row-major (lda >= K);  trans_a = 1: A is K x M row-major (lda >= M)
 *   trans_b = 0: B is K x N row-major (ldb >= N);  trans_b = 1: B is N x K row-major (ldb >= K)
 * epi (nullable) applies to C's rows/columns with d = N.  C must not overlap A or B.
 * With trans_a = 1 and large K the product is split over K into partial sums held in the
 * context workspace and combined in a fixed order. */
mixgcn_status mixgcn_gemm(mixgcn_ctx* ctx, int32_t precision, int32_t trans_a, int32_t trans_b,
                          int64_t M, int64_t N, int64_t K, const float* A, int64_t lda,
                          const float* B, int64_t ldb, float* C, int64_t ldc,
                          const mixgcn_epilogue* epi, void* stream);

/* ------------------------------------------------------------------------------------------
 * One GCN layer, X_out = drop * keep_scale * ReLU(A_hat X_in W + 1 b^T)   (Eq. 3)
 * ------------------------------------------------------------------------------------------ */
#define MIXGCN_ORDER_AUTO 0
#define MIXGCN_ORDER_AGG_FIRST 1 /* (A_hat X) W : aggregate at width d_in  */
#define MIXGCN_ORDER_UPD_FIRST 2 /* A_hat (X W) : aggregate at width d_out */

#define MIXGCN_LAYER_RELU 1u        /* sigma = ReLU (omit on the last layer) */
#define MIXGCN_LAYER_FIRST 2u       /* X_in is data: backward computes no input gradient */
#define MIXGCN_LAYER_GATE_GIN 4u    /* backward: G_in = (A_hat^T ...) * 1[X_in > 0] * in_scale,
                                       i.e. the ReLU mask of the layer below is applied by this
                                       layer's aggregation epilogue (Eq. 4, backward form) */
#define MIXGCN_LAYER_GOUT_GATED 8u  /* backward: G_out already carries this layer's ReLU/dropout
                                       mask (the layer above used GATE_GIN) */

#define MIXGCN_LAYER_OUT_ROWS_ONLY 16u /* forward: only the rows of X_out whose gout_row_mask byte is
                                       non-zero are wanted (the last layer of a training step: the
                                       loss reads train rows only; the paper computes every row of
                                       H^(L) in Algorithm 2, the gradients are the same).  The other
                                       rows of X_out and of `saved` are left UNCHANGED.  Needs
                                       gout_row_mask and gout_row_count (> 0, exact); no dropout
                                       mask; n_chunks is ignored.  The backward call must then be
                                       given the same gout_row_mask. */

#define MIXGCN_LAYER_SAVED_IS_VALID 64u /* forward of a FIRST layer in agg-first order: `saved` already
                                       holds A_hat X_in from an earlier call and neither the graph
                                       nor X_in has changed since (full-graph training feeds the
                                       same features every epoch, and the first layer's backward
                                       leaves `saved` intact): the aggregation is skipped.  Not in
                                       the paper, which recomputes it every iteration. */
#define MIXGCN_LAYER_SAVED_LP_ONLY 128u /* agg-first order with MIXGCN_PREC_BF16 and a saved_lp companion: the
                                       forward writes A_hat X_in to saved_lp ONLY -- both products that read it
                                       (the update and, in the backward, the weight gradient) read the bf16
                                       copy anyway, so the fp32 copy is a write nobody reads.  `saved` (fp32) is
                                       then left unchanged by the forward; the backward still uses it as scratch
                                       and must be given the same flag and saved_lp.  Not with n_chunks > 1, a
                                       row-sparse backward (gout_row_mask / gout_plan), OUT_ROWS_ONLY or
                                       SAVED_IS_VALID; MIXGCN_EUNSUPPORTED if the BF16 kernels cannot take the
                                       shape (there is then no fp32 operand to fall back on). */
#define MIXGCN_LAYER_GIN_ROWS_ONLY 32u /* backward with gout_plan: write only the rows of G_in in the
                                       plan's out_row_mask (the other rows are exactly zero and
                                       are left unchanged) */

typedef struct {
    int32_t d_in, d_out;
    int64_t ld_in, ld_out, ld_saved;
    int32_t order;      /* MIXGCN_ORDER_* ; AUTO picks by the per-node FLOP model of Appendix A */
    int32_t precision;  /* MIXGCN_PREC_* for the dense products */
    uint32_t flags;     /* MIXGCN_LAYER_* */
    float keep_scale;   /* 1/(1-p) for this layer's dropout mask; 1 if none */
    float in_scale;     /* keep_scale of the layer below, used with GATE_GIN; 1 if none */
    int32_t n_chunks;   /* >1: split rows into this many chunks and overlap the aggregation of
                           chunk k+1 with the update of chunk k on two streams; 0/1: off */
    /* Row-sparse backward (all optional; NULL / 0 = dense).  The gradient of a masked loss is non-zero
     * on train rows only, and one aggregation later on their neighbours only; telling the library
     * which rows may be non-zero lets it skip the rest -- the sampled form of Eq. 4 applied to the
     * rows of the operand instead of the elements of the output.  Results are those of the dense
     * computation with its exactly-zero terms left out.
     *   gout_row_mask   device uint8[n]: rows of G_out whose byte is 0 ARE exactly zero (caller's promise)
     *   gout_row_count  number of non-zero bytes in gout_row_mask if known, else 0; when it is below
     *                   n/4 (agg-first order) the dense products run on the compacted rows; a wrong
     *                   count is reported through the status word (code 4), never a memory fault
     *   gin_row_mask    device uint8[n], written: 0 for rows of G_in that are exactly zero */
    const uint8_t* gout_row_mask;
    int64_t gout_row_count;
    uint8_t* gin_row_mask;
    /* Backward with a row plan (optional; replaces gout_row_mask / gout_row_count / gin_row_mask in
     * mixgcn_layer_bwd): a plan of A_hat^T created from the row mask of G_out.  The dense products run
     * on the plan's compacted rows and the aggregation on its restricted matrix.  The rows of G_in that
     * can be non-zero are the plan's out_row_mask; with MIXGCN_LAYER_GIN_ROWS_ONLY only those rows of
     * G_in are written (for a layer below that itself runs with a plan made from that mask). */
    const mixgcn_rowplan* gout_plan;
    /* bf16 companions of the activations, used with MIXGCN_PREC_BF16 only (all optional).  The dense
     * products then read bf16 operands; the kernel that PRODUCES an activation (the aggregation's or the
     * update's epilogue) writes its bf16 copy beside the fp32 one, so no product has to convert its
     * operand first.  A NULL companion is replaced by a conversion pass inside the call (same result,
     * one more read of the fp32 operand).  Device uint16 (bf16 bits), 16-byte aligned, n rows; leading
     * dimensions in bf16 elements, multiples of 8, at least the tensor's width.
     *   saved_lp   n x ld_saved_lp   copy of `saved`: written by layer_fwd (agg-first: bf16(A_hat X_in)) and
     *                                read by layer_bwd; upd-first backward uses it as scratch.  With
     *                                MIXGCN_LAYER_SAVED_IS_VALID it must be valid as well.
     *   x_in_lp    n x ld_in_lp      copy of X_in, read (upd-first order: forward product and dW)
     *   x_out_lp   n x ld_out_lp     layer_fwd writes the copy of X_out (the next layer's x_in_lp)
     *   g_out_lp   n x ld_out_lp     layer_bwd reads the copy of G_out; used only when G_out arrives
     *                                already gated (MIXGCN_LAYER_GOUT_GATED, or a layer without ReLU and
     *                                dropout), i.e. when this call does not change G_out first
     *   g_in_lp    n x ld_in_lp      layer_bwd writes the copy of G_in (the layer below's g_out_lp) */
    uint16_t* saved_lp;
    int64_t ld_saved_lp;
    const uint16_t* x_in_lp;
    int64_t ld_in_lp;
    uint16_t* x_out_lp;
    int64_t ld_out_lp;
    uint16_t* g_out_lp;
    uint16_t* g_in_lp;
    /* Sign bitmaps of the activations (optional; the bitmap mask buffer of Section 3.2.1 for the ReLU masks the
     * backward pass applies -- Eq. 4's M): device uint32, n rows of ld words, bit (j & 31) of word (j >> 5) of a
     * row = (activation > 0).
     *   x_out_bits  n x ld_out_bits (>= ceil(d_out / 32)): with MIXGCN_LAYER_RELU, layer_fwd also writes the bitmap
     *               of X_out (after ReLU and dropout) -- the x_in_bits of the layer above
     *   x_in_bits   n x ld_in_bits (>= ceil(d_in / 32)): with MIXGCN_LAYER_GATE_GIN, layer_bwd reads the gate from
     *               this bitmap instead of the sign of X_in: one bit per element instead of four bytes */
    uint32_t* x_out_bits;
    int64_t ld_out_bits;
    const uint32_t* x_in_bits;
    int64_t ld_in_bits;
} mixgcn_layer_desc;

/* Row plan of a row-sparse aggregation.  Which rows of a gradient are non-zero depends on the graph
 * and the train mask only, so what follows from it is computed once and reused every iteration: the
 * kept rows (ascending) and the CSR of A_hat (transposed != 0: A_hat^T) restricted to the kept columns,
 * renumbered to positions in the compacted input, with its own aggregation schedule.  in_row_mask is a
 * device uint8[n] (non-zero = kept); it is read during the call only.  Synchronises the device.
 * A plan may be used only while its context and graph exist; it may be destroyed after them.
 * (The paper's sampled SpMM, Eq. 4, masks outputs; this is its counterpart on the operand's rows.) */
mixgcn_status mixgcn_rowplan_create(mixgcn_ctx* ctx, const mixgcn_graph* g, int transposed,
                                    const uint8_t* in_row_mask, mixgcn_rowplan** out);
mixgcn_status mixgcn_rowplan_destroy(mixgcn_rowplan* plan);
/* in_count kept input rows; out_count output rows with at least one kept entry; nnz kept entries.
 * All nullable. */
mixgcn_status mixgcn_rowplan_info(const mixgcn_rowplan* plan, int64_t* in_count, int64_t* out_count,
                                  int64_t* nnz);
/* Copies to DEVICE buffers (nullable): in_rows int32[in_count], the kept rows ascending;
 * out_row_mask uint8[n], 1 for output rows with at least one kept entry (exactly the rows of the
 * result that can be non-zero). */
mixgcn_status mixgcn_rowplan_export(const mixgcn_rowplan* plan, int32_t* in_rows, uint8_t* out_row_mask,
                                    void* stream);
/* Z = epilogue(A_restricted Yc): Yc is the COMPACTED input, in_count x ldy, row i = row in_rows[i] of
 * the full input; Z is n x ldz.  The same sum as mixgcn_spmm on the full input whose other rows are
 * zero.  rows_only != 0: only the rows of Z in the plan's out_row_mask are written (the others are
 * exactly zero in the full result and are left unchanged here).  Other arguments as mixgcn_spmm. */
mixgcn_status mixgcn_spmm_rowplan(mixgcn_ctx* ctx, const mixgcn_rowplan* plan, int32_t w, const float* Yc,
                                  int64_t ldy, float* Z, int64_t ldz, const mixgcn_epilogue* epi,
                                  int32_t rows_only, void* stream);

/* out[j] = sum_i X[i*ld + j] for j < d (the bias gradient of an update, db = 1^T dP): per-block
 * partial sums in a fixed order, then one pass over the partials in fp64.  X is n x ld on the device,
 * 16-byte aligned with ld a multiple of 4 (the activations' layout; MIXGCN_EINVAL otherwise);
 * out has d floats. */
mixgcn_status mixgcn_colsum(mixgcn_ctx* ctx, int64_t n, int32_t d, const float* X, int64_t ld, float* out,
                            void* stream);

/* Resolves MIXGCN_ORDER_AUTO: cost(agg-first) = c * d_in with c = 1 for a FIRST layer (its
 * backward needs no aggregation) else 2; cost(upd-first) = 2 * d_out; the smaller wins, ties
 * go to agg-first.  *saved_cols receives the number of columns the `saved` buffer needs
 * (d_in for agg-first, d_out for upd-first). */
mixgcn_status mixgcn_layer_plan(const mixgcn_layer_desc* desc, int32_t* order, int32_t* saved_cols);

/* Forward.  bias, drop_mask nullable.  `saved` is n x ld_saved:
 *   agg-first: receives A_hat X_in and must be handed unchanged to mixgcn_layer_bwd;
 *   upd-first: scratch for X_in W (contents not needed afterwards).
 * X_out is n x ld_out.  Buffers must not overlap. */
mixgcn_status mixgcn_layer_fwd(mixgcn_ctx* ctx, const mixgcn_graph* g, const mixgcn_layer_desc* desc,
                               const float* X_in, const float* W, const float* bias,
                               const uint8_t* drop_mask, float* saved, float* X_out, void* stream);

/* The last layer's forward and the loss in one call (Algorithm 2: the last aggregation + update and the loss
 * line).  Same results as mixgcn_layer_fwd (without a dropout mask) followed by mixgcn_loss_softmax_xent with
 * dlogits aliasing the logits -- *loss, pred (required here) and *n_correct (nullable) as there; `dlogits`
 * (n x ld_out) receives the gradient on train rows and zeros elsewhere, or, with
 * MIXGCN_OPT_LOSS_TRAIN_ROWS_ONLY = 2, is left unchanged elsewhere; `saved` as in mixgcn_layer_fwd -- but where
 * a whole row of logits is in one thread group's hands at the place that produces it, the loss is taken there
 * and the logits are never written: in the aggregation's epilogue for an update-first layer, in the tensor-core
 * product's epilogue for an aggregate-first layer with TF32 or BF16 products; both for d_out <= 256, no ReLU,
 * n_chunks <= 1.  (Same formulas; the sums within a row may run in another order than in the separate calls.)
 * Every other layer runs as the two separate steps inside this call.  MIXGCN_EUNSUPPORTED with OUT_ROWS_ONLY or
 * MIXGCN_OPT_LOSS_TRAIN_ROWS_ONLY = 1.  Device-visible conditions (empty mask, label out of range) as in
 * mixgcn_loss_softmax_xent.  The update-first form keeps 4 n bytes of scratch (the per-row loss terms) in the
 * context, allocated by the first call that needs it (a cudaMalloc; not covered by mixgcn_ctx_reserve). */
mixgcn_status mixgcn_layer_fwd_loss(mixgcn_ctx* ctx, const mixgcn_graph* g, const mixgcn_layer_desc* desc,
                                    const float* X_in, const float* W, const float* bias, float* saved,
                                    float* dlogits, const int32_t* labels, const uint8_t* train_mask,
                                    float* loss, int32_t* pred, int64_t* n_correct, void* stream);

/* Backward.  G_out (n x ld_out) is the gradient w.r.t. X_out and is OVERWRITTEN (it becomes
 * the gradient w.r.t. the pre-activation).  `saved` is consumed: agg-first reads A_hat X_in
 * from it and then overwrites it; upd-first uses it as scratch.  dW is d_in x d_out, dbias
 * d_out (nullable).  G_in (n x ld_in) receives the gradient w.r.t. X_in and must be NULL iff
 * MIXGCN_LAYER_FIRST is set.  X_out and drop_mask are the forward's. */
mixgcn_status mixgcn_layer_bwd(mixgcn_ctx* ctx, const mixgcn_graph* g, const mixgcn_layer_desc* desc,
                               const float* X_in, float* saved, const float* X_out,
                               const uint8_t* drop_mask, const float* W, float* G_out,
                               float* G_in, float* dW, float* dbias, void* stream);

/* Number of non-zero bytes of a device row mask (uint8[n]); *count is a HOST int64.  For callers
 * that want to hand layer_bwd the exact gout_row_count of a mask the library produced
 * (gin_row_mask).  Synchronises `stream`.  Not in the paper: bookkeeping of the row-sparse backward. */
mixgcn_status mixgcn_count_rows(mixgcn_ctx* ctx, int64_t n, const uint8_t* row_mask, int64_t* count,
                                void* stream);

/* Masked softmax cross-entropy (the loss line of Algorithm 2; mean over train nodes, natural
 * log): loss = -(1/#T) sum_{v in T} log softmax(logits_v)[label_v]; dlogits_v =
 * (softmax(logits_v) - e_label) / #T on T and 0 elsewhere; pred_v = lowest index of the row
 * maximum; *n_correct = #{v in T : pred_v == label_v}.  logits n x C with ld; labels
 * int32[n]; train_mask uint8[n]; loss device fp32 scalar; dlogits (nullable, may alias
 * logits, same ld); pred int32[n] (nullable); n_correct device int64 scalar (nullable).
 * 1 <= C <= 4096.  Empty mask or a label outside [0,C) on a train node: outputs are zeros
 * and the status word is set. */
mixgcn_status mixgcn_loss_softmax_xent(mixgcn_ctx* ctx, int64_t n, int32_t C, const float* logits,
                                       int64_t ld, const int32_t* labels, const uint8_t* train_mask,
                                       float* loss, float* dlogits, int32_t* pred,
                                       int64_t* n_correct, void* stream);

/* The same loss for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a deployment variant of mixgcn_loss_softmax_xent.)  A process that has given the whole
 * GPU to its own memory pool, or a latency-critical loop that cannot afford the device-wide
 * synchronisation of cudaMalloc/cudaFree, cannot create a mixgcn_ctx (its status word and
 * workspace are cudaMalloc'd).  This entry point needs no context and calls no allocator: its
 * scratch (train-node counter, status word, one fp64 partial per 1024 rows) lives in a fixed
 * 256 KB array inside the library image, present on every GPU that loads the library until the
 * process exits.
 *  - Runs on the calling thread's CURRENT device; all pointers are device pointers of it.
 *  - Arguments and results as mixgcn_loss_softmax_xent; `status` (device int32, nullable)
 *    receives 0, 1 (empty train mask), 2 (label outside [0,C)) or 3 (a bounded wait inside the
 *    kernel gave up; loss, dlogits and pred are then undefined) when the stream reaches it.
 *  - Limit: n <= 33,554,432 rows (32768 partials x 1024 rows) and 1 <= C <= 4096; larger sizes
 *    return MIXGCN_EUNSUPPORTED and launch nothing.
 *  - The first call on each device looks up the scratch array's device address (one
 *    cudaGetSymbolAddress, cached per device in an atomic pointer, so host threads may race to be
 *    first); make that first call before any stream capture.
 *  - All calls on a device share the one array, which keeps the previous call's contents; each
 *    call clears the counter and status word first.  Two calls that overlap on the GPU (different
 *    streams, no ordering between them) race on it: order them. */
mixgcn_status mixgcn_loss_softmax_xent_noalloc(int64_t n, int32_t C, const float* logits, int64_t ld,
                                               const int32_t* labels, const uint8_t* train_mask,
                                               float* loss, float* dlogits, int32_t* pred,
                                               int64_t* n_correct, int32_t* status, void* stream);

/* Adam over n_tensors parameter tensors (HOST arrays of DEVICE pointers and element counts):
 * m = b1 m + (1-b1) g; v = b2 v + (1-b2) g^2; theta -= lr * (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + eps),
 * t >= 1, no weight decay (the weight-update step of Algorithm 2). */
mixgcn_status mixgcn_adam_step(mixgcn_ctx* ctx, int32_t n_tensors, float* const* param,
                               const float* const* grad, float* const* m, float* const* v,
                               const int64_t* numel, int64_t t, float lr, float beta1, float beta2,
                               float eps, void* stream);

/* One whole training iteration (Algorithm 2's loop body) with HOST inputs and outputs: copies
 * features, labels, mask, weights, biases and Adam moments to the device, runs forward, loss,
 * backward and Adam, and copies back the loss, the updated weights, biases and moments.
 * dims is int32[L+1] (d_0 .. d_L); W, b, mW, vW, mb, vb are host arrays of L host pointers
 * (dense fp32, updated in place); X is n x d_0 dense fp32; loss host fp32 scalar; pred
 * (nullable) host int32[n].  Uses AUTO ordering, ReLU on all layers but the last, no dropout.
 * When pred is NULL and the backward pass runs row-sparse, the last layer, the loss and its
 * gradient are computed on the train rows alone (nothing returned depends on the other rows).
 * The row plans of the backward pass are kept in the context and reused by the next call while the
 * graph and the train mask are unchanged (the mask is compared on the device every call).
 * Device buffers are taken from the context workspace (grown on demand).  Synchronises the streams it
 * used, except for a feature copy started for the next call (mixgcn_train_step_host_prefetch). */
mixgcn_status mixgcn_train_step_host(mixgcn_ctx* ctx, const mixgcn_graph* g, int32_t L,
                                     const int32_t* dims, int32_t precision, const float* X,
                                     const int32_t* labels, const uint8_t* train_mask,
                                     float* const* W, float* const* b, float* const* mW,
                                     float* const* vW, float* const* mb, float* const* vb,
                                     int64_t t, float lr, float beta1, float beta2, float eps,
                                     float* loss, int32_t* pred);

/* Announces the features the NEXT mixgcn_train_step_host call on this context will be given (host
 * pointer, same n x d_0 shape; pinned memory if the copy is to overlap anything).  The call that runs
 * before it then starts that host-to-device copy itself, on a second stream, as soon as its own
 * features are no longer needed (after the first layer's forward in agg-first order, whose backward
 * reads A_hat X from `saved` and not X), so the copy overlaps the rest of that iteration; the next
 * call, given the same pointer, waits for it instead of copying again.  The buffer must stay valid and
 * unchanged until that next call returns.  One announcement serves one call; with a first layer in
 * upd-first order, or when the next call passes another pointer, nothing is lost but the overlap.
 * Not in the paper: Algorithm 2 keeps its inputs resident. */
mixgcn_status mixgcn_train_step_host_prefetch(mixgcn_ctx* ctx, const float* X_next);

/* Measurement helper (the paper has no counterpart): `table` is rows x 128 fp32 on the device; every
 * warp of a grid that fills the GPU reads gathers_per_warp (a multiple of 8) pseudo-random rows of 512
 * bytes, eight in flight, and discards them.  *total_gathers (host, nullable) receives the number of rows
 * read; time the call with events on `stream`: rows * 512 bytes / time is the row-gather rate of the
 * memory level the table lives in (L2 when it fits, HBM otherwise) -- the denominator the benchmark
 * quotes aggregations with an L2-resident input against.  `sink` is one device float, never written
 * in practice. */
mixgcn_status mixgcn_probe_gather(mixgcn_ctx* ctx, const float* table, int64_t rows, int64_t gathers_per_warp,
                                  uint64_t seed, float* sink, int64_t* total_gathers, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MIXGCN_H_ */
