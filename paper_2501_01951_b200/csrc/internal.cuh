// Internal declarations shared by the translation units of libmixgcn.so.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "mixgcn.h"

namespace mixgcn {

void set_error(const char* fmt, ...);

#define MIXGCN_FAIL(status, ...)          \
    do {                                  \
        ::mixgcn::set_error(__VA_ARGS__); \
        return (status);                  \
    } while (0)

#define MIXGCN_CUDA(expr)                                                                    \
    do {                                                                                     \
        cudaError_t _e = (expr);                                                             \
        if (_e != cudaSuccess) {                                                             \
            ::mixgcn::set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(_e),      \
                                __FILE__, __LINE__);                                         \
            return _e == cudaErrorMemoryAllocation ? MIXGCN_ENOMEM : MIXGCN_ECUDA;           \
        }                                                                                    \
    } while (0)

#define MIXGCN_TRY(expr)                     \
    do {                                     \
        mixgcn_status _s = (expr);           \
        if (_s != MIXGCN_OK) return _s;      \
    } while (0)

enum Phase { PH_SPMM = 0, PH_GEMM = 1, PH_ELEM = 2, PH_LOSS = 3, PH_ADAM = 4, PH_GRAPH = 5, PH_SPMM_SPARSE = 6 };

// device status word codes
enum { DEV_OK = 0, DEV_EMPTY_MASK = 1, DEV_BAD_LABEL = 2, DEV_WAIT_EXPIRED = 3, DEV_BAD_ROW_COUNT = 4, DEV_BAD_INDEX = 5 };

// Bounds-checked debug build (-DMIXGCN_DEBUG_BOUNDS): every index a kernel takes FROM MEMORY (a column id, a
// schedule record's row and entry range, a segment table, a row list) is tested before it addresses anything.
// A bad one is recorded in the status word (code DEV_BAD_INDEX, the site in word 1, the value in words 2-3;
// the first report wins) and the access is skipped, so the kernel finishes and the context stays usable.
// The release build compiles these tests away.
#ifdef MIXGCN_DEBUG_BOUNDS
constexpr bool DEBUG_BOUNDS = true;
#else
constexpr bool DEBUG_BOUNDS = false;
#endif
enum { SITE_SPMM_COL = 1, SITE_SPMM_ROW = 2, SITE_SPMM_RANGE = 3, SITE_SPMM_POS = 4, SITE_SPMM_SEG = 5, SITE_ROW_LIST = 6 };
#ifdef __CUDACC__
__device__ __forceinline__ bool index_ok(int64_t i, int64_t limit, int32_t* status, int site) {
    if constexpr (DEBUG_BOUNDS) {
        if (i < 0 || i >= limit) {
            if (atomicCAS(status, DEV_OK, DEV_BAD_INDEX) == DEV_OK) {
                status[1] = site; status[2] = (int32_t)(uint32_t)i; status[3] = (int32_t)(i >> 32);
            }
            return false;
        }
    }
    return true;
}
#endif

struct ProfSpan {
    cudaEvent_t a, b;
    int phase;
};

}  // namespace mixgcn

struct mixgcn_ctx {
    int device;
    int sm_count;
    int32_t* d_status;        // device status word (int32[4])
    void* workspace;          // grow-on-demand scratch of the dense products, column sums and the loss
    int64_t workspace_bytes;
    void* workspace_rows;     // scratch of the row-sparse backward (row list, positions, compact operands)
    int64_t workspace_rows_bytes;
    void* workspace_spmm;     // scratch of the aggregation (partial rows of long-row segments); separate so
    int64_t workspace_spmm_bytes;  // that an aggregation and a dense product may overlap on two streams
    cudaStream_t side_stream[2];
    cudaEvent_t fork_ev, join_ev[2];
    cudaEvent_t chunk_ev[64];
    void* workspace_loss;     // scratch of the loss taken inside a layer's last kernel (count, partial sums, per-row terms): its own
    int64_t workspace_loss_bytes;   // block, because the product that takes the loss packs its weights into `workspace`
    void* workspace_lp;       // bf16 copies of fp32 operands converted on the fly (BF16 products whose caller gave no copy)
    int64_t workspace_lp_bytes;
    int64_t gemm_path[3];     // dense products served by: 0 fp32 FMA kernel, 1 tcgen05 TF32, 2 tcgen05 BF16
    int64_t gemm_pair_launches;   // of those, products that ran on CTA pairs (tcgen05 .cta_group::2)
    int no_cta_pairs;         // 1: keep every product on single CTAs (option, for comparison)
    int debug_wait_limit;     // > 0: polls after which the tensor-core kernels' waits give up (test of that path)
    int debug_drop_load;      // 1: the next K-major tensor-core product leaves one stage unfilled (test of that path)
    int spmm_slice_cols;      // 0 = default (one slice up to 1024 columns)
    int loss_train_rows_only; // 1 = the loss skips rows outside the train mask entirely
    // profiling
    int profile;
    mixgcn::ProfSpan* spans;
    int n_spans, cap_spans;
    int64_t launches_total;
    int64_t phase_launches[MIXGCN_N_PHASES];
    // device arena of mixgcn_train_step_host (activations, parameters, gradients), grown on demand
    void* arena;
    int64_t arena_bytes;
    // row plans of the last mixgcn_train_step_host call, reused while graph and train mask stay the same
    struct HostStepCache* step_cache;
    struct HostStepPrefetch* step_prefetch;
};

// One unit of aggregation work: `len` stored entries starting at `begin`.  For an ordinary row `row`
// is the output row; for a segment of a long row it is the ordinal of that row among the long rows.
struct __align__(16) SpmmRec {
    int64_t begin;
    int32_t len;
    int32_t row;
};

// Aggregation schedule of the rows [row0, row0 + n_rows) of one CSR orientation.
// Rows longer than SPMM_SEG entries are cut into segments at dyadic column-block boundaries and
// every SPMM_SEG entries; the segment records [0, total_segs) run in order of their first column, so
// that segments of different long rows that gather the same rows of Y run close in time (those rows
// are then served by the L2).  Every other row is one record, in perm order (records
// [total_segs, total_segs + n_rows - n_long)).
struct SpmmSchedule {
    int64_t row0, n_rows;
    int32_t* perm;             // [n_rows] row ids by descending entry count (ties by ascending id)
    int32_t max_deg;
    SpmmRec* rec;
    int64_t n_long, total_segs;
    int64_t* seg_off;          // [n_long+1] segments of long row i are numbered seg_off[i] .. seg_off[i+1]-1 in entry order
    int64_t* seg_pos;          // [total_segs] record position (= partial-row slot) of segment number q
    int64_t rows_above[3];     // rows with more than SPMM_PACK_DEG[i] entries (bucket boundaries in perm order)
};

// One CSR orientation of A_hat plus its aggregation schedules: one over all rows, and (built on
// first use) one per row chunk of the two-stream pipeline.
struct CsrView {
    int64_t* rowptr;   // [n+1]
    int32_t* col;      // [nnz]
    float* val;        // [nnz]
    SpmmSchedule full;
    SpmmSchedule* chunk;   // [n_chunk] schedules of the chunks floor(n*k/n_chunk) .. floor(n*(k+1)/n_chunk)
    int n_chunk;
};

struct mixgcn_graph {
    mixgcn_ctx* ctx;
    uint64_t uid;      // unique per created graph (a freed graph's address may be reused)
    int device;        // kept apart from ctx: a graph may be destroyed after its context
    int64_t n, nnz;
    int symmetric;     // the stored STRUCTURE is symmetric
    int bwd_is_fwd;    // bwd aliases fwd (symmetric structure and symmetric values)
    int norm;          // 0 symmetric normalisation, 1 row mean, 2 ones
    int has_diagonal;  // 1: every row stores its diagonal entry, 0: none does, 2: some do
    int32_t* deg;      // [n] entries per row of the stored matrix
    float* dinv;       // [n]
    CsrView fwd, bwd;  // bwd aliases fwd when symmetric
};

// Everything about a row-sparse aggregation that depends only on the graph and on WHICH rows of the
// input are non-zero: the kept rows, their positions, and the orientation's CSR restricted to the kept
// columns (column ids renumbered to positions in the compacted input) with its own schedule.
struct mixgcn_rowplan {
    mixgcn_ctx* ctx;
    int device;          // kept apart from ctx: a plan may be destroyed after its context
    const mixgcn_graph* g;
    int transposed;
    int64_t n, in_count, out_count, nnz;   // nnz: entries of the restricted matrix
    int32_t* idx;        // [in_count] kept input rows, ascending
    CsrView view;        // n rows; columns in [0, in_count)
    uint8_t* out_mask;   // [n] 1 for output rows that have at least one kept entry
};

namespace mixgcn {

constexpr int SPMM_SEG = 512;               // rows longer than this are cut into segments of at most this many entries
constexpr int SPMM_BLK_MIN_ENTRIES = 64;    // a long row uses 2^k column blocks while it keeps >= this many entries per block
constexpr int SPMM_MAX_LOG_BLOCKS = 8;      // at most 2^this column blocks per row
constexpr int SPMM_PACK_DEG[3] = {12, 5, 2};   // rows up to these lengths share a warp 2-, 4-, 8-fold

// Launch bookkeeping: counts the launch and, when profiling, brackets it with events.
struct LaunchScope {
    mixgcn_ctx* ctx;
    cudaStream_t stream;
    int span;
    LaunchScope(mixgcn_ctx* c, int phase, cudaStream_t s, int n_launches = 1);
    ~LaunchScope();
};

mixgcn_status ensure_workspace(mixgcn_ctx* ctx, int64_t bytes);
mixgcn_status ensure_workspace_spmm(mixgcn_ctx* ctx, int64_t bytes);
// Builds (once) the schedules of the `chunks` row chunks of this orientation.  Synchronises on first use.
mixgcn_status ensure_chunk_schedules(const mixgcn_graph* g, const CsrView& A, int chunks);

// Row-sparse input of an aggregation: rows v with in_mask[v] == 0 are exactly zero and skipped; a
// kept row v is read from row in_pos[v] of Y (null: row v); out_mask (nullable) receives which
// output rows received a contribution.
struct SpmmRowSparse {
    const uint8_t* in_mask;
    const int32_t* in_pos;
    uint8_t* out_mask;
};

// kernels' host launchers (all asynchronous on `s`)
// Aggregation over all rows (chunks <= 1) or over chunk k of `chunks` row chunks.
// Optional behaviour of one aggregation call.
// The loss taken inside the aggregation that produces the logits (last layer in upd-first order): each row's
// soft-max, arg-max, loss term and gradient are computed from the registers that hold the aggregated row, so
// the logits are never written.  Filled by loss_fuse_begin (count of train nodes, per-row loss scratch).
struct LossFuse {
    const int32_t* labels = nullptr;
    const uint8_t* train_mask = nullptr;
    const unsigned long long* count = nullptr;   // device: number of train nodes
    float* row_loss = nullptr;                   // device [n]: lse - logit[label] of every train row
    int32_t* pred = nullptr;                     // device [n]
    int zero_rows = 1;                           // 1: rows outside the train mask receive a zero gradient; 0: they are left alone
    double* part = nullptr;                      // device: partial sums of the final pass
    int n_part = 0;
};
mixgcn_status loss_fuse_begin(mixgcn_ctx* ctx, int64_t n, const int32_t* labels, const uint8_t* train_mask, int32_t* pred,
                              int64_t* n_correct, cudaStream_t s, LossFuse* out);
mixgcn_status loss_fuse_end(mixgcn_ctx* ctx, int64_t n, int32_t C, const LossFuse& lf, float* loss, int64_t* n_correct, cudaStream_t s);

struct SpmmOpts {
    const LossFuse* loss = nullptr;          // non-null: soft-max cross-entropy epilogue (width <= 256, bias only); Z receives the gradient
    const SpmmRowSparse* sparse = nullptr;   // row-sparse input: test the input's row mask inside the kernel
    const uint8_t* row_filter = nullptr;     // compute only the output rows whose byte is non-zero (not with `sparse`)
    int phase = PH_SPMM;                     // profiling phase the launches are booked under
    int64_t row_limit = -1;                  // >= 0: only the first row_limit rows of the schedule (longest first)
    uint16_t* Z_lp = nullptr;                // nullable: also write a bf16 copy of Z (after the epilogue), ldz_lp a multiple of 4
    int64_t ldz_lp = 0;
    const uint32_t* out_bits = nullptr;      // nullable: bit-packed output mask of a sampled aggregation (Eq. 4), n x ld_bits words
    int64_t ld_bits = 0;
    int64_t y_rows = -1;                     // rows of Y and entries of the view, where they differ from the graph's n and
    int64_t nnz = -1;                        // nnz (a row plan's restricted matrix, a compacted input): limits of the debug build's index tests
};
mixgcn_status launch_spmm(mixgcn_ctx* ctx, const mixgcn_graph* g, const CsrView& A, int chunks, int k,
                          int32_t w, const float* Y, int64_t ldy, float* Z, int64_t ldz,
                          const mixgcn_epilogue* epi, cudaStream_t s, const SpmmOpts& opts = SpmmOpts());
// schedule of all n rows of a view whose column ids lie in [0, n_cols); release of a view's memory
mixgcn_status build_view_schedule(int64_t n_cols, int64_t n, CsrView& v, cudaStream_t s);
void release_view(CsrView& v);
// colsum_b of launch_gemm (weight-gradient form, trans_a = 1, only): also out[n] = sum_k B[k][n], the bias
// gradient when B = dP -- produced inside the product's kernel where that kernel reads B as fp32 words,
// by the column-sum kernels otherwise.
// bf16 companions of one dense product (all nullable): copies of A and of B (the MM form's second
// activation operand) that a producer already wrote, and a bf16 copy of C to write for the next product.
// Leading dimensions in bf16 elements, multiples of 8; pointers 16-byte aligned.
struct GemmLP {
    bool a_fp32_missing = false;      // the fp32 A holds no data (only its bf16 copy was written): no fallback below bf16
    const LossFuse* loss = nullptr;   // K-major form, N <= 256, C = logits of a masked loss: the epilogue writes every row's arg-max to
                                      // loss->pred and only the rows of loss->train_mask to C (the others zeroed if loss->zero_rows, else
                                      // left alone); MIXGCN_EUNSUPPORTED, nothing computed, if no tensor-core kernel takes the product
    const uint16_t* A = nullptr; int64_t lda = 0;
    const uint16_t* B = nullptr; int64_t ldb = 0;
    uint16_t* C = nullptr; int64_t ldc = 0;
};
mixgcn_status launch_gemm(mixgcn_ctx* ctx, int precision, int ta, int tb, int64_t M, int64_t N, int64_t K,
                          const float* A, int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc,
                          const mixgcn_epilogue* epi, int64_t epi_row0, cudaStream_t s, const GemmLP* lp = nullptr,
                          float* colsum_b = nullptr);
mixgcn_status launch_gemm_simt(mixgcn_ctx* ctx, int ta, int tb, int64_t M, int64_t N, int64_t K,
                               const float* A, int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc,
                               const mixgcn_epilogue* epi, int64_t epi_row0, cudaStream_t s);
mixgcn_status launch_gemm_tc(mixgcn_ctx* ctx, int kind, int ta, int tb, int64_t M, int64_t N, int64_t K, const void* A,
                             int64_t lda, const void* B, int64_t ldb, float* C, int64_t ldc,
                             const mixgcn_epilogue* epi, int64_t epi_row0, cudaStream_t s, uint16_t* C_lp, int64_t ldc_lp,
                             float* colsum_b = nullptr, bool* colsum_done = nullptr, const LossFuse* loss = nullptr,
                             bool* bits_done = nullptr);
// bits[u][j] = (X == null || X[u][j] > 0) && (bytes == null || bytes[u*w + j] != 0), n x ld_bits words
mixgcn_status launch_mask_pack(mixgcn_ctx* ctx, int64_t n, int32_t w, const float* X, int64_t ldx, const uint8_t* bytes,
                               uint32_t* bits, int64_t ld_bits, cudaStream_t s);
mixgcn_status launch_splitk_reduce(mixgcn_ctx* ctx, int64_t M, int64_t N, int splits, const float* part, float* C,
                                   int64_t ldc, const mixgcn_epilogue* epi, cudaStream_t s);
mixgcn_status launch_to_bf16(mixgcn_ctx* ctx, int64_t rows, int32_t d, const float* src, int64_t ld_src, uint16_t* dst,
                             int64_t ld_dst, cudaStream_t s);
mixgcn_status ensure_workspace_lp(mixgcn_ctx* ctx, int64_t bytes);
mixgcn_status launch_colsum(mixgcn_ctx* ctx, int64_t n, int32_t d, const float* X, int64_t ld, float* out,
                            cudaStream_t s);
mixgcn_status launch_gate(mixgcn_ctx* ctx, int64_t n, int32_t d, float* G, int64_t ldg, const float* X_out,
                          int64_t ldx, int relu, const uint8_t* drop_mask, float keep_scale, cudaStream_t s);

// Row set of a row-sparse backward call, carved from the context's row workspace.
struct RowSet {
    int32_t* idx;    // [count] kept rows, ascending
    int32_t* pos;    // [n] position of a kept row in idx, -1 otherwise
    float* a;        // count x ld_a compact operand
    float* b;        // count x ld_b compact operand
    int64_t count;
};
mixgcn_status build_row_set(mixgcn_ctx* ctx, int64_t n, const uint8_t* mask, int64_t count, int64_t ld_a, int64_t ld_b,
                            RowSet* rs, cudaStream_t s);
mixgcn_status launch_gather_rows(mixgcn_ctx* ctx, int64_t n_rows, int64_t count, int32_t d, const int32_t* idx, const float* src,
                                 int64_t ld_src, float* dst, int64_t ld_dst, cudaStream_t s);

mixgcn_status ensure_workspace_rows(mixgcn_ctx* ctx, int64_t bytes);
void free_step_cache(mixgcn_ctx* ctx);
// dst[idx[i], :] = src[i, :] for i < count (the inverse of launch_gather_rows)
mixgcn_status launch_scatter_rows(mixgcn_ctx* ctx, int64_t n_rows, int64_t count, int32_t d, const int32_t* idx, const float* src,
                                  int64_t ld_src, float* dst, int64_t ld_dst, cudaStream_t s);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace mixgcn
