// Context, error reporting, profiling, and the per-layer composition of aggregation and update
// (Eq. 3 and Algorithm 2 of the paper): ordering choice from the per-node FLOP model of
// Appendix A, and the row-chunked aggregation -> update pipeline on two streams (the fine-grain
// sparse/dense pipeline of Section 3.2.2 mapped onto one GPU).
#include <stdarg.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "internal.cuh"

using namespace mixgcn;

namespace {
thread_local char g_err[512] = "";
}

namespace mixgcn {

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

LaunchScope::LaunchScope(mixgcn_ctx* c, int phase, cudaStream_t s, int n_launches) : ctx(c), stream(s), span(-1) {
    ctx->launches_total += n_launches;
    ctx->phase_launches[phase] += n_launches;
    if (!ctx->profile) return;
    if (ctx->n_spans == ctx->cap_spans) {
        int cap = ctx->cap_spans ? ctx->cap_spans * 2 : 256;
        ProfSpan* ns = (ProfSpan*)realloc(ctx->spans, cap * sizeof(ProfSpan));
        if (!ns) return;
        for (int i = ctx->cap_spans; i < cap; ++i) { ns[i].a = nullptr; ns[i].b = nullptr; }
        ctx->spans = ns; ctx->cap_spans = cap;
    }
    span = ctx->n_spans++;
    ProfSpan& sp = ctx->spans[span];
    if (!sp.a) { cudaEventCreate(&sp.a); cudaEventCreate(&sp.b); }
    sp.phase = phase;
    cudaEventRecord(sp.a, stream);
}

LaunchScope::~LaunchScope() {
    if (span >= 0) cudaEventRecord(ctx->spans[span].b, stream);
}

mixgcn_status ensure_workspace(mixgcn_ctx* ctx, int64_t bytes) {
    if (bytes <= ctx->workspace_bytes) return MIXGCN_OK;
    int64_t want = bytes + (bytes >> 2);
    want = (want + 255) & ~(int64_t)255;
    void* p = nullptr;
    // the old block may still be in use by enqueued kernels: wait before releasing it
    MIXGCN_CUDA(cudaDeviceSynchronize());
    if (ctx->workspace) cudaFree(ctx->workspace);
    ctx->workspace = nullptr; ctx->workspace_bytes = 0;
    cudaError_t e = cudaMalloc(&p, (size_t)want);
    if (e != cudaSuccess) {
        cudaGetLastError();
        MIXGCN_FAIL(MIXGCN_ENOMEM, "workspace of %lld bytes could not be allocated", (long long)want);
    }
    ctx->workspace = p; ctx->workspace_bytes = want;
    return MIXGCN_OK;
}

mixgcn_status ensure_workspace_spmm(mixgcn_ctx* ctx, int64_t bytes) {
    if (bytes <= ctx->workspace_spmm_bytes) return MIXGCN_OK;
    int64_t want = bytes + (bytes >> 2);
    want = (want + 255) & ~(int64_t)255;
    void* p = nullptr;
    MIXGCN_CUDA(cudaDeviceSynchronize());
    if (ctx->workspace_spmm) cudaFree(ctx->workspace_spmm);
    ctx->workspace_spmm = nullptr; ctx->workspace_spmm_bytes = 0;
    if (cudaMalloc(&p, (size_t)want) != cudaSuccess) {
        cudaGetLastError();
        MIXGCN_FAIL(MIXGCN_ENOMEM, "aggregation workspace of %lld bytes could not be allocated", (long long)want);
    }
    ctx->workspace_spmm = p; ctx->workspace_spmm_bytes = want;
    return MIXGCN_OK;
}

mixgcn_status ensure_workspace_lp(mixgcn_ctx* ctx, int64_t bytes) {
    if (bytes <= ctx->workspace_lp_bytes) return MIXGCN_OK;
    int64_t want = bytes + (bytes >> 3);
    want = (want + 255) & ~(int64_t)255;
    void* p = nullptr;
    MIXGCN_CUDA(cudaDeviceSynchronize());
    if (ctx->workspace_lp) cudaFree(ctx->workspace_lp);
    ctx->workspace_lp = nullptr; ctx->workspace_lp_bytes = 0;
    if (cudaMalloc(&p, (size_t)want) != cudaSuccess) {
        cudaGetLastError();
        MIXGCN_FAIL(MIXGCN_ENOMEM, "bf16 operand workspace of %lld bytes could not be allocated", (long long)want);
    }
    ctx->workspace_lp = p; ctx->workspace_lp_bytes = want;
    return MIXGCN_OK;
}

mixgcn_status launch_gemm(mixgcn_ctx* ctx, int precision, int ta, int tb, int64_t M, int64_t N, int64_t K,
                          const float* A, int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc,
                          const mixgcn_epilogue* epi, int64_t epi_row0, cudaStream_t s, const GemmLP* lp, float* colsum_b) {
    // BF16 requests go to the tcgen05 kind::f16 kernels on bf16 copies of the activation operands: the
    // copies a producer already wrote (lp), else copies made here by a conversion kernel.  TF32
    // requests, and BF16 requests whose shape the bf16 kernels do not take, go to the kind::tf32
    // kernels (at least the requested precision); whatever those do not take, and fp32 requests, use the
    // FMA kernel.  ctx->gemm_path counts which kernel served each product.
    uint16_t* c_lp = lp ? lp->C : nullptr;
    const int64_t ldc_lp = lp ? lp->ldc : 0;
    const LossFuse* loss = lp ? lp->loss : nullptr;
    bool c_lp_done = false, bits_done = false;
    if (ta && epi && (epi->gate_bits || epi->sign_bits)) MIXGCN_FAIL(MIXGCN_EINVAL, "gemm: bit-packed masks belong to the K-major form (trans_a = 0)");
    mixgcn_status st = MIXGCN_EUNSUPPORTED;
    const bool fp32_layout = aligned16(A) && (lda & 3) == 0 && (!ta || (aligned16(B) && (ldb & 3) == 0));
    if (precision == MIXGCN_PREC_BF16 && !(ta && tb) && fp32_layout && M > 0 && N > 0 && K > 0) {
        auto round8 = [](int64_t x) { return (x + 7) & ~(int64_t)7; };
        auto up = [](int64_t x) { return (x + 255) & ~(int64_t)255; };
        const int64_t a_rows = ta ? K : M, a_cols = ta ? M : K;
        const uint16_t* a_lp = lp ? lp->A : nullptr;
        int64_t lda_lp = lp ? lp->lda : 0;
        const uint16_t* b_lp = (ta && lp) ? lp->B : nullptr;
        int64_t ldb_lp = (ta && lp) ? lp->ldb : 0;
        const int64_t need_a = a_lp ? 0 : up(a_rows * round8(a_cols) * 2);
        const int64_t need_b = (ta && !b_lp) ? up(K * round8(N) * 2) : 0;
        if (need_a + need_b > 0) MIXGCN_TRY(ensure_workspace_lp(ctx, need_a + need_b));
        if (!a_lp) {
            uint16_t* dst = reinterpret_cast<uint16_t*>(ctx->workspace_lp);
            lda_lp = round8(a_cols);
            MIXGCN_TRY(launch_to_bf16(ctx, a_rows, (int32_t)a_cols, A, lda, dst, lda_lp, s));
            a_lp = dst;
        }
        if (ta && !b_lp) {
            uint16_t* dst = reinterpret_cast<uint16_t*>(reinterpret_cast<char*>(ctx->workspace_lp) + need_a);
            ldb_lp = round8(N);
            MIXGCN_TRY(launch_to_bf16(ctx, K, (int32_t)N, B, ldb, dst, ldb_lp, s));
            b_lp = dst;
        }
        st = launch_gemm_tc(ctx, 1, ta, tb, M, N, K, a_lp, lda_lp, ta ? (const void*)b_lp : (const void*)B, ta ? ldb_lp : ldb,
                            C, ldc, epi, epi_row0, s, ta ? nullptr : c_lp, ldc_lp, nullptr, nullptr, loss, &bits_done);
        if (st == MIXGCN_OK) { ctx->gemm_path[2]++; c_lp_done = !ta && c_lp; }
    }
    if (st == MIXGCN_EUNSUPPORTED && lp && lp->a_fp32_missing)
        MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "gemm: the bf16 kernels cannot take this product and its fp32 operand was not kept (SAVED_LP_ONLY)");
    bool colsum_done = false;
    if (colsum_b && !ta) MIXGCN_FAIL(MIXGCN_EINVAL, "gemm: column sums of B are a by-product of the weight-gradient form only");
    if (st == MIXGCN_EUNSUPPORTED && precision != MIXGCN_PREC_FP32) {
        st = launch_gemm_tc(ctx, 0, ta, tb, M, N, K, A, lda, B, ldb, C, ldc, epi, epi_row0, s, ta ? nullptr : c_lp, ldc_lp,
                            colsum_b, &colsum_done, loss, &bits_done);
        if (st == MIXGCN_OK) { ctx->gemm_path[1]++; c_lp_done = !ta && c_lp; }
    }
    if (st == MIXGCN_EUNSUPPORTED && loss) return st;      // the caller runs the product and the loss separately
    if (st == MIXGCN_EUNSUPPORTED) {
        st = launch_gemm_simt(ctx, ta, tb, M, N, K, A, lda, B, ldb, C, ldc, epi, epi_row0, s);
        if (st == MIXGCN_OK) ctx->gemm_path[0]++;
    }
    if (st != MIXGCN_OK) return st;
    if (c_lp && !c_lp_done) MIXGCN_TRY(launch_to_bf16(ctx, M, (int32_t)N, C, ldc, c_lp, ldc_lp, s));
    // sign bitmap of the result where the kernel's epilogue did not write it: one more pass over C
    if (epi && epi->sign_bits && !bits_done)
        MIXGCN_TRY(launch_mask_pack(ctx, M, (int32_t)N, C, ldc, nullptr, epi->sign_bits + epi_row0 * epi->ld_sign_bits, epi->ld_sign_bits, s));
    if (colsum_b && !colsum_done) MIXGCN_TRY(launch_colsum(ctx, K, (int32_t)N, B, ldb, colsum_b, s));
    return MIXGCN_OK;
}

}  // namespace mixgcn

extern "C" const char* mixgcn_status_string(mixgcn_status s) {
    switch (s) {
        case MIXGCN_OK: return "ok";
        case MIXGCN_EINVAL: return "invalid argument";
        case MIXGCN_ENOMEM: return "out of memory";
        case MIXGCN_ECUDA: return "CUDA runtime error";
        case MIXGCN_EUNSUPPORTED: return "unsupported";
        case MIXGCN_EBADGRAPH: return "malformed graph";
        case MIXGCN_ETIMEOUT: return "device wait timed out";
        case MIXGCN_EDEVICE: return "device reported bad data";
    }
    return "unknown status";
}

extern "C" const char* mixgcn_last_error(void) { return g_err; }

extern "C" mixgcn_status mixgcn_ctx_create(mixgcn_ctx** out, int device) {
    if (!out) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_create: null out");
    int count = 0;
    MIXGCN_CUDA(cudaGetDeviceCount(&count));
    if (device < 0 || device >= count) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_create: device %d not in [0,%d)", device, count);
    MIXGCN_CUDA(cudaSetDevice(device));
    cudaDeviceProp prop;
    MIXGCN_CUDA(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "ctx_create: device %d is sm_%d%d; this library is built for sm_100a only", device, prop.major, prop.minor);
    mixgcn_ctx* c = new (std::nothrow) mixgcn_ctx();
    if (!c) MIXGCN_FAIL(MIXGCN_ENOMEM, "ctx_create: host allocation failed");
    memset(c, 0, sizeof(*c));
    c->device = device;
    c->sm_count = prop.multiProcessorCount;
    MIXGCN_CUDA(cudaMalloc((void**)&c->d_status, 4 * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMemset(c->d_status, 0, 4 * sizeof(int32_t)));
    for (int i = 0; i < 2; ++i) MIXGCN_CUDA(cudaStreamCreateWithFlags(&c->side_stream[i], cudaStreamNonBlocking));
    MIXGCN_CUDA(cudaEventCreateWithFlags(&c->fork_ev, cudaEventDisableTiming));
    for (int i = 0; i < 2; ++i) MIXGCN_CUDA(cudaEventCreateWithFlags(&c->join_ev[i], cudaEventDisableTiming));
    for (int i = 0; i < 64; ++i) MIXGCN_CUDA(cudaEventCreateWithFlags(&c->chunk_ev[i], cudaEventDisableTiming));
    *out = c;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_ctx_destroy(mixgcn_ctx* ctx) {
    if (!ctx) return MIXGCN_OK;
    cudaSetDevice(ctx->device);
    cudaDeviceSynchronize();
    for (int i = 0; i < ctx->cap_spans; ++i) {
        if (ctx->spans[i].a) cudaEventDestroy(ctx->spans[i].a);
        if (ctx->spans[i].b) cudaEventDestroy(ctx->spans[i].b);
    }
    free(ctx->spans);
    for (int i = 0; i < 64; ++i) if (ctx->chunk_ev[i]) cudaEventDestroy(ctx->chunk_ev[i]);
    for (int i = 0; i < 2; ++i) { if (ctx->join_ev[i]) cudaEventDestroy(ctx->join_ev[i]); if (ctx->side_stream[i]) cudaStreamDestroy(ctx->side_stream[i]); }
    if (ctx->fork_ev) cudaEventDestroy(ctx->fork_ev);
    free_step_cache(ctx);
    cudaFree(ctx->workspace);
    cudaFree(ctx->workspace_spmm);
    cudaFree(ctx->workspace_rows);
    cudaFree(ctx->workspace_lp);
    cudaFree(ctx->workspace_loss);
    cudaFree(ctx->arena);
    cudaFree(ctx->d_status);
    delete ctx;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_ctx_reserve(mixgcn_ctx* ctx, int64_t bytes) {
    if (!ctx || bytes < 0) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_reserve: bad argument");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    return ensure_workspace(ctx, bytes);
}

extern "C" mixgcn_status mixgcn_ctx_poll_status(mixgcn_ctx* ctx, int32_t* code) {
    if (!ctx) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_poll_status: null ctx");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    MIXGCN_CUDA(cudaDeviceSynchronize());
    int32_t w[4] = {0, 0, 0, 0};
    MIXGCN_CUDA(cudaMemcpy(w, ctx->d_status, sizeof(w), cudaMemcpyDeviceToHost));
    MIXGCN_CUDA(cudaMemset(ctx->d_status, 0, sizeof(w)));
    const int32_t h = w[0];
    if (code) *code = h;
    if (h == DEV_OK) return MIXGCN_OK;
    if (h == DEV_BAD_INDEX) {
        static const char* const sites[] = {"?", "aggregation: column id", "aggregation: row of a schedule record", "aggregation: entry range of a schedule record",
                                            "aggregation: position of a kept row", "aggregation: segment table", "row list of a gather / scatter"};
        const int site = w[1] >= 1 && w[1] <= 6 ? w[1] : 0;
        const long long value = (long long)(((uint64_t)(uint32_t)w[3] << 32) | (uint32_t)w[2]);
        MIXGCN_FAIL(MIXGCN_EDEVICE, "bounds-checked build: index out of range (%s, value %lld); the access was skipped", sites[site], value);
    }
    if (h == DEV_WAIT_EXPIRED) MIXGCN_FAIL(MIXGCN_ETIMEOUT, "a bounded device-side wait expired");
    MIXGCN_FAIL(MIXGCN_EDEVICE, h == DEV_EMPTY_MASK ? "loss: the train mask is empty" : h == DEV_BAD_LABEL ? "loss: a label lies outside [0, C)" : "layer_bwd: gout_row_count does not match gout_row_mask");
}

extern "C" mixgcn_status mixgcn_build_info(int32_t* debug_bounds) {
    if (debug_bounds) *debug_bounds = DEBUG_BOUNDS ? 1 : 0;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_debug_poke_col(mixgcn_graph* g, int64_t entry, int32_t value, int32_t* old_value) {
    if (!DEBUG_BOUNDS) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "debug_poke_col: this is not the bounds-checked debug build");
    if (!g || entry < 0 || entry >= g->nnz) MIXGCN_FAIL(MIXGCN_EINVAL, "debug_poke_col: entry outside [0, nnz)");
    MIXGCN_CUDA(cudaSetDevice(g->device));
    MIXGCN_CUDA(cudaDeviceSynchronize());
    if (old_value) MIXGCN_CUDA(cudaMemcpy(old_value, g->fwd.col + entry, sizeof(int32_t), cudaMemcpyDeviceToHost));
    MIXGCN_CUDA(cudaMemcpy(g->fwd.col + entry, &value, sizeof(int32_t), cudaMemcpyHostToDevice));
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_ctx_set_option(mixgcn_ctx* ctx, int32_t option, int64_t value) {
    if (!ctx) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_set_option: null ctx");
    if (option == MIXGCN_OPT_SPMM_SLICE_COLS) {
        if (value != 0 && (value < 4 || value > 1024 || (value & 3)))
            MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_set_option: slice width must be 0 or a multiple of 4 in [4, 1024] (got %lld)", (long long)value);
        ctx->spmm_slice_cols = (int)value;
        return MIXGCN_OK;
    }
    if (option == MIXGCN_OPT_LOSS_TRAIN_ROWS_ONLY) {
        if (value < 0 || value > 2) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_set_option: loss rows option takes 0, 1 or 2 (got %lld)", (long long)value);
        ctx->loss_train_rows_only = (int)value;
        return MIXGCN_OK;
    }
    if (option == MIXGCN_OPT_GEMM_CTA_PAIRS) {
        if (value != 0 && value != 1) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_set_option: cta-pairs takes 0 or 1 (got %lld)", (long long)value);
        ctx->no_cta_pairs = value ? 0 : 1;
        return MIXGCN_OK;
    }
    if (option == MIXGCN_OPT_DEBUG_WAIT_LIMIT) {
        if (value < 0 || value > (1ll << 30)) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_set_option: wait limit must lie in [0, 2^30] (got %lld)", (long long)value);
        ctx->debug_wait_limit = (int)value;
        return MIXGCN_OK;
    }
    if (option == MIXGCN_OPT_DEBUG_DROP_LOAD) {
        if (value != 0 && value != 1) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_set_option: drop-load takes 0 or 1 (got %lld)", (long long)value);
        ctx->debug_drop_load = (int)value;
        return MIXGCN_OK;
    }
    MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_set_option: unknown option %d", option);
}

extern "C" mixgcn_status mixgcn_ctx_gemm_paths(const mixgcn_ctx* ctx, int64_t counts[4]) {
    if (!ctx || !counts) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_gemm_paths: null argument");
    for (int i = 0; i < 3; ++i) counts[i] = ctx->gemm_path[i];
    counts[3] = ctx->gemm_pair_launches;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_ctx_profile_enable(mixgcn_ctx* ctx, int enable) {
    if (!ctx) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_profile_enable: null ctx");
    ctx->profile = enable ? 1 : 0;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_ctx_profile_read(mixgcn_ctx* ctx, double ms[MIXGCN_N_PHASES],
                                                 int64_t launches[MIXGCN_N_PHASES], int64_t* launches_total) {
    if (!ctx) MIXGCN_FAIL(MIXGCN_EINVAL, "ctx_profile_read: null ctx");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    MIXGCN_CUDA(cudaDeviceSynchronize());
    if (ms) for (int i = 0; i < MIXGCN_N_PHASES; ++i) ms[i] = 0.0;
    for (int i = 0; i < ctx->n_spans; ++i) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, ctx->spans[i].a, ctx->spans[i].b) == cudaSuccess && ms) ms[ctx->spans[i].phase] += t;
    }
    cudaGetLastError();
    ctx->n_spans = 0;
    if (launches) for (int i = 0; i < MIXGCN_N_PHASES; ++i) { launches[i] = ctx->phase_launches[i]; ctx->phase_launches[i] = 0; }
    if (launches_total) *launches_total = ctx->launches_total;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_gemm(mixgcn_ctx* ctx, int32_t precision, int32_t trans_a, int32_t trans_b,
                                     int64_t M, int64_t N, int64_t K, const float* A, int64_t lda,
                                     const float* B, int64_t ldb, float* C, int64_t ldc,
                                     const mixgcn_epilogue* epi, void* stream) {
    if (!ctx || !A || !B || !C) MIXGCN_FAIL(MIXGCN_EINVAL, "gemm: null argument");
    if (M <= 0 || N <= 0 || K <= 0) MIXGCN_FAIL(MIXGCN_EINVAL, "gemm: M, N, K must be positive");
    if (precision < MIXGCN_PREC_FP32 || precision > MIXGCN_PREC_BF16) MIXGCN_FAIL(MIXGCN_EINVAL, "gemm: unknown precision %d", precision);
    const int64_t min_lda = trans_a ? M : K, min_ldb = trans_b ? K : N;
    if (lda < min_lda || ldb < min_ldb || ldc < N)
        MIXGCN_FAIL(MIXGCN_EINVAL, "gemm: leading dimensions must cover the matrix (lda=%lld ldb=%lld ldc=%lld)",
                    (long long)lda, (long long)ldb, (long long)ldc);
    if (C == A || C == B) MIXGCN_FAIL(MIXGCN_EINVAL, "gemm: C must not overlap A or B");
    if (epi && epi->residual) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "gemm: the residual term is an aggregation epilogue");
    if (epi && ((epi->gate_bits && epi->ld_gate_bits < (N + 31) / 32) || (epi->sign_bits && epi->ld_sign_bits < (N + 31) / 32)))
        MIXGCN_FAIL(MIXGCN_EINVAL, "gemm: a bit-packed mask needs ld >= ceil(N / 32) words");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    return launch_gemm(ctx, precision, trans_a, trans_b, M, N, K, A, lda, B, ldb, C, ldc, epi, 0, (cudaStream_t)stream);
}

// ------------------------------------------------------------------------------------------------
// Layer composition
// ------------------------------------------------------------------------------------------------

namespace {

int resolve_order(const mixgcn_layer_desc* d) {
    if (d->order == MIXGCN_ORDER_AGG_FIRST || d->order == MIXGCN_ORDER_UPD_FIRST) return d->order;
    // Appendix A: aggregating costs deg(v) * width per node, so the width at which the sparse
    // product runs decides.  A first layer aggregates once (forward only) in agg-first order.
    const int64_t c = (d->flags & MIXGCN_LAYER_FIRST) ? 1 : 2;
    const int64_t cost_agg = c * (int64_t)d->d_in, cost_upd = 2 * (int64_t)d->d_out;
    return cost_agg <= cost_upd ? MIXGCN_ORDER_AGG_FIRST : MIXGCN_ORDER_UPD_FIRST;
}

mixgcn_status check_desc(const mixgcn_layer_desc* d, const char* who) {
    if (!d) MIXGCN_FAIL(MIXGCN_EINVAL, "%s: null layer descriptor", who);
    if (d->d_in <= 0 || d->d_out <= 0) MIXGCN_FAIL(MIXGCN_EINVAL, "%s: widths must be positive", who);
    if (d->order < 0 || d->order > 2) MIXGCN_FAIL(MIXGCN_EINVAL, "%s: unknown order %d", who, d->order);
    if (d->precision < 0 || d->precision > 2) MIXGCN_FAIL(MIXGCN_EINVAL, "%s: unknown precision %d", who, d->precision);
    const int order = resolve_order(d);
    const int saved_cols = order == MIXGCN_ORDER_AGG_FIRST ? d->d_in : d->d_out;
    if (d->ld_in < d->d_in || d->ld_out < d->d_out || d->ld_saved < saved_cols || (d->ld_in & 3) || (d->ld_out & 3) || (d->ld_saved & 3))
        MIXGCN_FAIL(MIXGCN_EINVAL, "%s: leading dimensions must be multiples of 4 with ld_in >= d_in, ld_out >= d_out, ld_saved >= %d", who, saved_cols);
    if (d->n_chunks < 0 || d->n_chunks > 64) MIXGCN_FAIL(MIXGCN_EINVAL, "%s: n_chunks must lie in [0, 64]", who);
    // bf16 companions: 16-byte aligned, leading dimensions multiples of 8 that cover the width
    auto lp_ok = [](const void* ptr, int64_t ld, int64_t cols) { return !ptr || (aligned16(ptr) && (ld & 7) == 0 && ld >= cols); };
    if (!lp_ok(d->saved_lp, d->ld_saved_lp, saved_cols) || !lp_ok(d->x_in_lp, d->ld_in_lp, d->d_in) || !lp_ok(d->g_in_lp, d->ld_in_lp, d->d_in) ||
        !lp_ok(d->x_out_lp, d->ld_out_lp, d->d_out) || !lp_ok(d->g_out_lp, d->ld_out_lp, d->d_out))
        MIXGCN_FAIL(MIXGCN_EINVAL, "%s: bf16 companions must be 16-byte aligned with leading dimensions that are multiples of 8 and cover the width", who);
    if ((d->x_out_bits && d->ld_out_bits < (d->d_out + 31) / 32) || (d->x_in_bits && d->ld_in_bits < (d->d_in + 31) / 32))
        MIXGCN_FAIL(MIXGCN_EINVAL, "%s: a sign bitmap needs ld >= ceil(width / 32) words", who);
    if (d->flags & MIXGCN_LAYER_SAVED_LP_ONLY) {
        if (order != MIXGCN_ORDER_AGG_FIRST || d->precision != MIXGCN_PREC_BF16 || !d->saved_lp || d->n_chunks > 1 ||
            d->gout_row_mask || d->gout_plan || (d->flags & (MIXGCN_LAYER_OUT_ROWS_ONLY | MIXGCN_LAYER_SAVED_IS_VALID)))
            MIXGCN_FAIL(MIXGCN_EINVAL, "%s: SAVED_LP_ONLY needs agg-first order, BF16 products, saved_lp, one chunk and a dense backward", who);
    }
    return MIXGCN_OK;
}

// The bf16 companions of a layer are used only when its dense products run in BF16.
struct LayerLP {
    uint16_t* saved; int64_t ld_saved;
    const uint16_t* x_in; int64_t ld_in;
    uint16_t* x_out; uint16_t* g_out; int64_t ld_out;
    uint16_t* g_in;
    explicit LayerLP(const mixgcn_layer_desc* d) {
        const bool on = d->precision == MIXGCN_PREC_BF16;
        saved = on ? d->saved_lp : nullptr; ld_saved = d->ld_saved_lp;
        x_in = on ? d->x_in_lp : nullptr; ld_in = d->ld_in_lp;
        x_out = on ? d->x_out_lp : nullptr; g_out = on ? d->g_out_lp : nullptr; ld_out = d->ld_out_lp;
        g_in = on ? d->g_in_lp : nullptr;
    }
};

// Row range of chunk i of m over k rows: the floor(k*i/m) boundaries of Algorithm 2's update loop.
inline int64_t chunk_bound(int64_t k, int i, int m) { return (k * (int64_t)i) / m; }

}  // namespace

extern "C" mixgcn_status mixgcn_colsum(mixgcn_ctx* ctx, int64_t n, int32_t d, const float* X, int64_t ld, float* out,
                                       void* stream) {
    if (!ctx || !X || !out) MIXGCN_FAIL(MIXGCN_EINVAL, "colsum: null argument");
    if (n <= 0 || d <= 0 || ld < d) MIXGCN_FAIL(MIXGCN_EINVAL, "colsum: need n > 0, d > 0 and ld >= d");
    if (!aligned16(X) || (ld & 3)) MIXGCN_FAIL(MIXGCN_EINVAL, "colsum: X must be 16-byte aligned with ld a multiple of 4 (ld=%lld)", (long long)ld);
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    return launch_colsum(ctx, n, d, X, ld, out, (cudaStream_t)stream);
}

extern "C" mixgcn_status mixgcn_layer_plan(const mixgcn_layer_desc* desc, int32_t* order, int32_t* saved_cols) {
    if (!desc) MIXGCN_FAIL(MIXGCN_EINVAL, "layer_plan: null descriptor");
    if (desc->d_in <= 0 || desc->d_out <= 0 || desc->order < 0 || desc->order > 2)
        MIXGCN_FAIL(MIXGCN_EINVAL, "layer_plan: bad widths or order");
    const int o = resolve_order(desc);
    if (order) *order = o;
    if (saved_cols) *saved_cols = o == MIXGCN_ORDER_AGG_FIRST ? desc->d_in : desc->d_out;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_layer_fwd(mixgcn_ctx* ctx, const mixgcn_graph* g, const mixgcn_layer_desc* d,
                                          const float* X_in, const float* W, const float* bias,
                                          const uint8_t* drop_mask, float* saved, float* X_out, void* stream) {
    if (!ctx || !g || !X_in || !W || !saved || !X_out) MIXGCN_FAIL(MIXGCN_EINVAL, "layer_fwd: null argument");
    MIXGCN_TRY(check_desc(d, "layer_fwd"));
    if (!aligned16(X_in) || !aligned16(saved) || !aligned16(X_out) || !aligned16(W))
        MIXGCN_FAIL(MIXGCN_EINVAL, "layer_fwd: matrices must be 16-byte aligned");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t n = g->n;
    const int order = resolve_order(d);
    mixgcn_epilogue epi{};
    epi.bias = bias;
    epi.relu = (d->flags & MIXGCN_LAYER_RELU) ? 1 : 0;
    epi.drop_mask = drop_mask;
    epi.keep_scale = d->keep_scale;
    const int64_t ldw = d->d_out;  // W is dense; the GEMM uses scalar loads for it when d_out % 4 != 0
    int chunks = d->n_chunks > 1 ? d->n_chunks : 1;
    const bool saved_valid = (d->flags & MIXGCN_LAYER_SAVED_IS_VALID) != 0;
    if (saved_valid) {
        if (!(d->flags & MIXGCN_LAYER_FIRST) || order != MIXGCN_ORDER_AGG_FIRST)
            MIXGCN_FAIL(MIXGCN_EINVAL, "layer_fwd: SAVED_IS_VALID is for a FIRST layer in agg-first order");
        chunks = 1;
    }

    if (d->flags & MIXGCN_LAYER_OUT_ROWS_ONLY) {
        // Only the rows in gout_row_mask are wanted: aggregate those rows alone; in agg-first order the
        // update then runs on the compacted rows and its result is scattered back.
        const uint8_t* rows = d->gout_row_mask;
        const int64_t cnt = d->gout_row_count;
        SpmmOpts filter_rows; filter_rows.row_filter = rows;
        if (!rows || cnt <= 0 || cnt > n)
            MIXGCN_FAIL(MIXGCN_EINVAL, "layer_fwd: OUT_ROWS_ONLY needs gout_row_mask and its exact count (mask %s, count %lld, n %lld)",
                        rows ? "given" : "null", (long long)cnt, (long long)n);
        if (drop_mask) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "layer_fwd: OUT_ROWS_ONLY does not take a dropout mask");
        if (order == MIXGCN_ORDER_AGG_FIRST) {
            if (!saved_valid)
                MIXGCN_TRY(launch_spmm(ctx, g, g->fwd, 1, 0, d->d_in, X_in, d->ld_in, saved, d->ld_saved, nullptr, s, filter_rows));
            RowSet rs;
            const int64_t lda = (d->d_in + 3) / 4 * 4, ldb = (d->d_out + 3) / 4 * 4;
            MIXGCN_TRY(build_row_set(ctx, n, rows, cnt, lda, ldb, &rs, s));
            MIXGCN_TRY(launch_gather_rows(ctx, n, cnt, d->d_in, rs.idx, saved, d->ld_saved, rs.a, lda, s));
            MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 0, cnt, d->d_out, d->d_in, rs.a, lda, W, ldw, rs.b, ldb, &epi, 0, s));
            MIXGCN_TRY(launch_scatter_rows(ctx, n, cnt, d->d_out, rs.idx, rs.b, ldb, X_out, d->ld_out, s));
            return MIXGCN_OK;
        }
        MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 0, n, d->d_out, d->d_in, X_in, d->ld_in, W, ldw, saved, d->ld_saved,
                               nullptr, 0, s));
        MIXGCN_TRY(launch_spmm(ctx, g, g->fwd, 1, 0, d->d_out, saved, d->ld_saved, X_out, d->ld_out, &epi, s, filter_rows));
        return MIXGCN_OK;
    }

    const LayerLP lp(d);
    if (epi.relu && d->x_out_bits) { epi.sign_bits = d->x_out_bits; epi.ld_sign_bits = d->ld_out_bits; }   // the ReLU mask, one bit per element
    if (order == MIXGCN_ORDER_AGG_FIRST) {
        SpmmOpts agg_opts; agg_opts.Z_lp = lp.saved; agg_opts.ldz_lp = lp.ld_saved;     // the aggregation also writes bf16(A_hat X)
        if (chunks == 1) {
            const bool lp_only = (d->flags & MIXGCN_LAYER_SAVED_LP_ONLY) != 0;
            if (!saved_valid)
                MIXGCN_TRY(launch_spmm(ctx, g, g->fwd, 1, 0, d->d_in, X_in, d->ld_in, lp_only ? nullptr : saved, d->ld_saved, nullptr, s, agg_opts));
            GemmLP glp; glp.A = lp.saved; glp.lda = lp.ld_saved; glp.C = lp.x_out; glp.ldc = lp.ld_out; glp.a_fp32_missing = lp_only;
            MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 0, n, d->d_out, d->d_in, saved, d->ld_saved, W, ldw, X_out,
                                   d->ld_out, &epi, 0, s, &glp));
            return MIXGCN_OK;
        }
        // aggregation of chunk k+1 on stream A overlaps the update of chunk k on stream B
        MIXGCN_TRY(ensure_chunk_schedules(g, g->fwd, chunks));
        cudaStream_t sa = ctx->side_stream[0], sb = ctx->side_stream[1];
        MIXGCN_CUDA(cudaEventRecord(ctx->fork_ev, s));
        MIXGCN_CUDA(cudaStreamWaitEvent(sa, ctx->fork_ev, 0));
        MIXGCN_CUDA(cudaStreamWaitEvent(sb, ctx->fork_ev, 0));
        for (int k = 0; k < chunks; ++k) {
            const int64_t r0 = chunk_bound(n, k, chunks), r1 = chunk_bound(n, k + 1, chunks);
            if (r1 <= r0) continue;
            MIXGCN_TRY(launch_spmm(ctx, g, g->fwd, chunks, k, d->d_in, X_in, d->ld_in, saved, d->ld_saved, nullptr, sa, agg_opts));
            MIXGCN_CUDA(cudaEventRecord(ctx->chunk_ev[k], sa));
            MIXGCN_CUDA(cudaStreamWaitEvent(sb, ctx->chunk_ev[k], 0));
            // without the caller's bf16 copy of `saved` a BF16 product would convert into the one shared
            // workspace from two streams: the chunks then run TF32 (at least the requested precision)
            GemmLP glp;
            glp.A = lp.saved ? lp.saved + r0 * lp.ld_saved : nullptr; glp.lda = lp.ld_saved;
            glp.C = lp.x_out ? lp.x_out + r0 * lp.ld_out : nullptr; glp.ldc = lp.ld_out;
            const int prec_k = (d->precision == MIXGCN_PREC_BF16 && !lp.saved) ? MIXGCN_PREC_TF32 : d->precision;
            MIXGCN_TRY(launch_gemm(ctx, prec_k, 0, 0, r1 - r0, d->d_out, d->d_in, saved + r0 * d->ld_saved,
                                   d->ld_saved, W, ldw, X_out + r0 * d->ld_out, d->ld_out, &epi, r0, sb, &glp));
        }
        MIXGCN_CUDA(cudaEventRecord(ctx->join_ev[0], sa));
        MIXGCN_CUDA(cudaEventRecord(ctx->join_ev[1], sb));
        MIXGCN_CUDA(cudaStreamWaitEvent(s, ctx->join_ev[0], 0));
        MIXGCN_CUDA(cudaStreamWaitEvent(s, ctx->join_ev[1], 0));
        return MIXGCN_OK;
    }
    // update first: Q = X_in W (into `saved`), then X_out = epilogue(A_hat Q).  Every row of Q is
    // needed before any aggregated row can be produced, so there is nothing to chunk here.
    {
        GemmLP glp; glp.A = lp.x_in; glp.lda = lp.ld_in;
        MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 0, n, d->d_out, d->d_in, X_in, d->ld_in, W, ldw, saved, d->ld_saved,
                               nullptr, 0, s, &glp));
    }
    SpmmOpts out_opts; out_opts.Z_lp = lp.x_out; out_opts.ldz_lp = lp.ld_out;
    MIXGCN_TRY(launch_spmm(ctx, g, g->fwd, 1, 0, d->d_out, saved, d->ld_saved, X_out, d->ld_out, &epi, s, out_opts));
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_layer_fwd_loss(mixgcn_ctx* ctx, const mixgcn_graph* g, const mixgcn_layer_desc* d,
                                               const float* X_in, const float* W, const float* bias, float* saved,
                                               float* dlogits, const int32_t* labels, const uint8_t* train_mask,
                                               float* loss, int32_t* pred, int64_t* n_correct, void* stream) {
    if (!ctx || !g || !X_in || !W || !saved || !dlogits || !labels || !train_mask || !loss || !pred)
        MIXGCN_FAIL(MIXGCN_EINVAL, "layer_fwd_loss: null argument");
    MIXGCN_TRY(check_desc(d, "layer_fwd_loss"));
    if (!aligned16(X_in) || !aligned16(saved) || !aligned16(dlogits) || !aligned16(W))
        MIXGCN_FAIL(MIXGCN_EINVAL, "layer_fwd_loss: matrices must be 16-byte aligned");
    if ((d->flags & MIXGCN_LAYER_OUT_ROWS_ONLY) || ctx->loss_train_rows_only == 1)
        MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "layer_fwd_loss: every row's logits are produced here (no OUT_ROWS_ONLY, no MIXGCN_OPT_LOSS_TRAIN_ROWS_ONLY = 1)");
    if (d->d_out > 4096) MIXGCN_FAIL(MIXGCN_EINVAL, "layer_fwd_loss: at most 4096 classes");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t n = g->n;
    const int order = resolve_order(d);
    // The loss can be taken where the logits are produced if a whole row is in one thread group's hands there:
    // at most 256 classes, nothing but the bias between the sums and the logits, all rows in one piece.
    const bool plain = !(d->flags & (MIXGCN_LAYER_RELU | MIXGCN_LAYER_SAVED_IS_VALID | MIXGCN_LAYER_SAVED_LP_ONLY)) && d->n_chunks <= 1 && d->d_out <= 256;
    mixgcn_epilogue epi{};
    epi.bias = bias; epi.keep_scale = 1.0f;
    if (plain && order == MIXGCN_ORDER_UPD_FIRST) {
        // logits = A_hat (X_in W) + b: the aggregation's epilogue takes the loss
        const LayerLP lp(d);
        GemmLP glp; glp.A = lp.x_in; glp.lda = lp.ld_in;
        MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 0, n, d->d_out, d->d_in, X_in, d->ld_in, W, d->d_out, saved, d->ld_saved,
                               nullptr, 0, s, &glp));
        LossFuse lf;
        MIXGCN_TRY(loss_fuse_begin(ctx, n, labels, train_mask, pred, n_correct, s, &lf));
        SpmmOpts opts; opts.loss = &lf;
        MIXGCN_TRY(launch_spmm(ctx, g, g->fwd, 1, 0, d->d_out, saved, d->ld_saved, dlogits, d->ld_out, &epi, s, opts));
        return loss_fuse_end(ctx, n, d->d_out, lf, loss, n_correct, s);
    }
    if (plain && order == MIXGCN_ORDER_AGG_FIRST && d->precision != MIXGCN_PREC_FP32) {
        // logits = (A_hat X_in) W + b: the tensor-core product's epilogue finds every row's arg-max and writes the
        // logits of the train rows only; the loss then runs over those rows in place
        const LayerLP lp(d);
        SpmmOpts agg_opts; agg_opts.Z_lp = lp.saved; agg_opts.ldz_lp = lp.ld_saved;
        MIXGCN_TRY(launch_spmm(ctx, g, g->fwd, 1, 0, d->d_in, X_in, d->ld_in, saved, d->ld_saved, nullptr, s, agg_opts));
        LossFuse lf;
        lf.train_mask = train_mask; lf.pred = pred; lf.zero_rows = ctx->loss_train_rows_only == 2 ? 0 : 1;
        GemmLP glp; glp.A = lp.saved; glp.lda = lp.ld_saved; glp.loss = &lf;
        const mixgcn_status st = launch_gemm(ctx, d->precision, 0, 0, n, d->d_out, d->d_in, saved, d->ld_saved, W, d->d_out, dlogits,
                                             d->ld_out, &epi, 0, s, &glp);
        if (st == MIXGCN_OK) {
            const int keep = ctx->loss_train_rows_only;
            ctx->loss_train_rows_only = 1;               // train rows only, in place; pred is already complete
            const mixgcn_status sl = mixgcn_loss_softmax_xent(ctx, n, d->d_out, dlogits, d->ld_out, labels, train_mask, loss, dlogits,
                                                              nullptr, n_correct, stream);
            ctx->loss_train_rows_only = keep;
            return sl;
        }
        if (st != MIXGCN_EUNSUPPORTED) return st;
        // no tensor-core kernel for this shape: the product and the loss as two steps (the aggregation is in `saved`)
        MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 0, n, d->d_out, d->d_in, saved, d->ld_saved, W, d->d_out, dlogits, d->ld_out,
                               &epi, 0, s, nullptr));
        return mixgcn_loss_softmax_xent(ctx, n, d->d_out, dlogits, d->ld_out, labels, train_mask, loss, dlogits, pred, n_correct, stream);
    }
    // everything else: the layer, then the loss in place over its output
    MIXGCN_TRY(mixgcn_layer_fwd(ctx, g, d, X_in, W, bias, nullptr, saved, dlogits, stream));
    return mixgcn_loss_softmax_xent(ctx, n, d->d_out, dlogits, d->ld_out, labels, train_mask, loss, dlogits, pred, n_correct, stream);
}

extern "C" mixgcn_status mixgcn_layer_bwd(mixgcn_ctx* ctx, const mixgcn_graph* g, const mixgcn_layer_desc* d,
                                          const float* X_in, float* saved, const float* X_out,
                                          const uint8_t* drop_mask, const float* W, float* G_out, float* G_in,
                                          float* dW, float* dbias, void* stream) {
    if (!ctx || !g || !X_in || !saved || !X_out || !W || !G_out || !dW) MIXGCN_FAIL(MIXGCN_EINVAL, "layer_bwd: null argument");
    MIXGCN_TRY(check_desc(d, "layer_bwd"));
    const bool first = (d->flags & MIXGCN_LAYER_FIRST) != 0;
    if (first != (G_in == nullptr)) MIXGCN_FAIL(MIXGCN_EINVAL, "layer_bwd: G_in must be NULL exactly when MIXGCN_LAYER_FIRST is set");
    if (!aligned16(X_in) || !aligned16(saved) || !aligned16(X_out) || !aligned16(W) || !aligned16(G_out) ||
        !aligned16(dW) || (G_in && !aligned16(G_in)))
        MIXGCN_FAIL(MIXGCN_EINVAL, "layer_bwd: matrices must be 16-byte aligned");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t n = g->n;
    const int order = resolve_order(d);
    const int relu = (d->flags & MIXGCN_LAYER_RELU) ? 1 : 0;
    const int64_t ldw = d->d_out;

    // gradient w.r.t. the pre-activation, in place in G_out
    LayerLP lp(d);
    if (!(d->flags & MIXGCN_LAYER_GOUT_GATED) && (relu || drop_mask)) {
        MIXGCN_TRY(launch_gate(ctx, n, d->d_out, G_out, d->ld_out, X_out, d->ld_out, relu, drop_mask, d->keep_scale, s));
        lp.g_out = nullptr;      // the caller's bf16 copy predates the gate
    }

    mixgcn_epilogue gin_epi{};
    const mixgcn_epilogue* gin = nullptr;
    if (d->flags & MIXGCN_LAYER_GATE_GIN) {
        gin_epi.gate = X_in; gin_epi.ld_gate = d->ld_in; gin_epi.gate_scale = d->in_scale; gin_epi.keep_scale = 1.0f;
        if (d->x_in_bits) { gin_epi.gate_bits = d->x_in_bits; gin_epi.ld_gate_bits = d->ld_in_bits; }     // read instead of X_in's sign
        gin = &gin_epi;
    }
    if (const mixgcn_rowplan* plan = d->gout_plan) {
        // Row plan: dense products on the plan's compacted rows, aggregation on its restricted matrix.
        if (plan->ctx != ctx || plan->g != g || !plan->transposed) MIXGCN_FAIL(MIXGCN_EINVAL, "layer_bwd: gout_plan must be a plan of this graph's transposed orientation");
        const int64_t cnt = plan->in_count;
        const int64_t lda = (d->d_in + 3) / 4 * 4, ldb = (d->d_out + 3) / 4 * 4;
        auto up = [](int64_t x) { return (x + 255) & ~(int64_t)255; };
        const int64_t rows_alloc = cnt > 0 ? cnt : 1;
        MIXGCN_TRY(ensure_workspace_rows(ctx, up(rows_alloc * lda * 4) + up(rows_alloc * ldb * 4)));
        float* ca = reinterpret_cast<float*>(ctx->workspace_rows);
        float* cb = reinterpret_cast<float*>(reinterpret_cast<char*>(ctx->workspace_rows) + up(rows_alloc * lda * 4));
        // rows of the restricted matrix are scheduled longest first: its non-empty rows are the first out_count
        SpmmOpts plan_all; plan_all.phase = PH_SPMM_SPARSE;
        plan_all.y_rows = cnt; plan_all.nnz = plan->nnz;          // the restricted matrix gathers from the compacted rows
        SpmmOpts plan_opts = plan_all; plan_opts.row_limit = (d->flags & MIXGCN_LAYER_GIN_ROWS_ONLY) ? plan->out_count : -1;
        plan_opts.Z_lp = lp.g_in; plan_opts.ldz_lp = lp.ld_in;
        plan_all.Z_lp = lp.saved; plan_all.ldz_lp = lp.ld_saved;
        MIXGCN_TRY(launch_gather_rows(ctx, n, cnt, d->d_out, plan->idx, G_out, d->ld_out, cb, ldb, s));         // dP_T
        if (order == MIXGCN_ORDER_AGG_FIRST) {
            MIXGCN_TRY(launch_gather_rows(ctx, n, cnt, d->d_in, plan->idx, saved, d->ld_saved, ca, lda, s));     // Z_T
            // dW = Z_T^T dP_T, and db = 1^T dP_T as its by-product
            MIXGCN_TRY(launch_gemm(ctx, d->precision, 1, 0, d->d_in, d->d_out, cnt, ca, lda, cb, ldb, dW, ldw, nullptr, 0, s, nullptr, dbias));
            if (!first) {
                MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 1, cnt, d->d_in, d->d_out, cb, ldb, W, ldw, ca, lda, nullptr, 0, s));
                MIXGCN_TRY(launch_spmm(ctx, g, plan->view, 1, 0, d->d_in, ca, lda, G_in, d->ld_in, gin, s, plan_opts));
            }
            return MIXGCN_OK;
        }
        // update first: dQ = A_hat^T dZ from the compacted rows (into `saved`, every row), then the dense products
        if (dbias) MIXGCN_TRY(launch_colsum(ctx, cnt, d->d_out, cb, ldb, dbias, s));
        MIXGCN_TRY(launch_spmm(ctx, g, plan->view, 1, 0, d->d_out, cb, ldb, saved, d->ld_saved, nullptr, s, plan_all));
        GemmLP wlp; wlp.A = lp.x_in; wlp.lda = lp.ld_in; wlp.B = lp.saved; wlp.ldb = lp.ld_saved;
        MIXGCN_TRY(launch_gemm(ctx, d->precision, 1, 0, d->d_in, d->d_out, n, X_in, d->ld_in, saved, d->ld_saved, dW, ldw, nullptr, 0, s, &wlp));
        if (!first) {
            GemmLP xlp; xlp.A = lp.saved; xlp.lda = lp.ld_saved; xlp.C = lp.g_in; xlp.ldc = lp.ld_in;
            MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 1, n, d->d_in, d->d_out, saved, d->ld_saved, W, ldw, G_in, d->ld_in, gin, 0, s, &xlp));
        }
        return MIXGCN_OK;
    }
    const uint8_t* rmask = d->gout_row_mask;
    SpmmRowSparse sp{rmask, nullptr, d->gin_row_mask};
    SpmmOpts sparse_opts; sparse_opts.sparse = rmask ? &sp : nullptr;
    SpmmOpts gin_opts = sparse_opts; gin_opts.Z_lp = lp.g_in; gin_opts.ldz_lp = lp.ld_in;         // aggregations that produce G_in
    SpmmOpts dq_opts = sparse_opts; dq_opts.Z_lp = lp.saved; dq_opts.ldz_lp = lp.ld_saved;        // upd-first: dQ into `saved`

    if (order == MIXGCN_ORDER_AGG_FIRST) {
        const int64_t cnt = d->gout_row_count;
        const bool rows_only = (d->flags & MIXGCN_LAYER_OUT_ROWS_ONLY) != 0;   // other rows of G_out / saved are not data
        if (rows_only && !(rmask && cnt > 0)) MIXGCN_FAIL(MIXGCN_EINVAL, "layer_bwd: OUT_ROWS_ONLY needs gout_row_mask and its exact count");
        if (rmask && cnt > 0 && (cnt * 4 < n || rows_only)) {
            // Few non-zero rows: dW, db and dZ from the compacted rows, then a row-sparse aggregation.
            RowSet rs;
            const int64_t lda = (d->d_in + 3) / 4 * 4, ldb = (d->d_out + 3) / 4 * 4;
            MIXGCN_TRY(build_row_set(ctx, n, rmask, cnt, lda, ldb, &rs, s));
            MIXGCN_TRY(launch_gather_rows(ctx, n, cnt, d->d_in, rs.idx, saved, d->ld_saved, rs.a, lda, s));     // Z_T
            MIXGCN_TRY(launch_gather_rows(ctx, n, cnt, d->d_out, rs.idx, G_out, d->ld_out, rs.b, ldb, s));      // dP_T
            MIXGCN_TRY(launch_gemm(ctx, d->precision, 1, 0, d->d_in, d->d_out, cnt, rs.a, lda, rs.b, ldb, dW, ldw, nullptr, 0, s, nullptr, dbias));
            if (!first) {
                MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 1, cnt, d->d_in, d->d_out, rs.b, ldb, W, ldw, rs.a, lda, nullptr, 0, s));
                sp.in_pos = rs.pos;                                                                             // dZ_T is compact
                gin_opts.y_rows = cnt;
                MIXGCN_TRY(launch_spmm(ctx, g, g->bwd, 1, 0, d->d_in, rs.a, lda, G_in, d->ld_in, gin, s, gin_opts));
            }
            return MIXGCN_OK;
        }
        // dW = (A_hat X_in)^T dP ; dZ = dP W^T (over `saved`) ; G_in = A_hat^T dZ
        // dW = (A_hat X_in)^T dP, and db = 1^T dP as its by-product
        GemmLP wlp; wlp.A = lp.saved; wlp.lda = lp.ld_saved; wlp.B = lp.g_out; wlp.ldb = lp.ld_out;
        wlp.a_fp32_missing = (d->flags & MIXGCN_LAYER_SAVED_LP_ONLY) != 0;
        MIXGCN_TRY(launch_gemm(ctx, d->precision, 1, 0, d->d_in, d->d_out, n, saved, d->ld_saved, G_out, d->ld_out, dW,
                               ldw, nullptr, 0, s, &wlp, dbias));
        if (!first) {
            GemmLP zlp; zlp.A = lp.g_out; zlp.lda = lp.ld_out;
            MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 1, n, d->d_in, d->d_out, G_out, d->ld_out, W, ldw, saved,
                                   d->ld_saved, nullptr, 0, s, &zlp));
            MIXGCN_TRY(launch_spmm(ctx, g, g->bwd, 1, 0, d->d_in, saved, d->ld_saved, G_in, d->ld_in, gin, s, gin_opts));
        }
        return MIXGCN_OK;
    }
    // update first: dQ = A_hat^T dZ (into `saved`) ; dW = X_in^T dQ ; G_in = dQ W^T
    // (rows of dQ that received no contribution are zero, and so are those rows of G_in: the mask the
    // aggregation reports is G_in's row mask as well)
    if (d->flags & MIXGCN_LAYER_OUT_ROWS_ONLY) {
        // only the masked rows of G_out are data: the bias gradient sums those rows alone
        const int64_t cnt = d->gout_row_count;
        if (!(rmask && cnt > 0)) MIXGCN_FAIL(MIXGCN_EINVAL, "layer_bwd: OUT_ROWS_ONLY needs gout_row_mask and its exact count");
        if (dbias) {
            RowSet rs;
            const int64_t ldb = (d->d_out + 3) / 4 * 4;
            MIXGCN_TRY(build_row_set(ctx, n, rmask, cnt, 4, ldb, &rs, s));
            MIXGCN_TRY(launch_gather_rows(ctx, n, cnt, d->d_out, rs.idx, G_out, d->ld_out, rs.b, ldb, s));
            MIXGCN_TRY(launch_colsum(ctx, cnt, d->d_out, rs.b, ldb, dbias, s));
        }
    } else if (dbias) {
        MIXGCN_TRY(launch_colsum(ctx, n, d->d_out, G_out, d->ld_out, dbias, s));
    }
    MIXGCN_TRY(launch_spmm(ctx, g, g->bwd, 1, 0, d->d_out, G_out, d->ld_out, saved, d->ld_saved, nullptr, s, dq_opts));
    GemmLP wlp; wlp.A = lp.x_in; wlp.lda = lp.ld_in; wlp.B = lp.saved; wlp.ldb = lp.ld_saved;
    MIXGCN_TRY(launch_gemm(ctx, d->precision, 1, 0, d->d_in, d->d_out, n, X_in, d->ld_in, saved, d->ld_saved, dW, ldw,
                           nullptr, 0, s, &wlp));
    if (!first) {
        GemmLP xlp; xlp.A = lp.saved; xlp.lda = lp.ld_saved; xlp.C = lp.g_in; xlp.ldc = lp.ld_in;
        MIXGCN_TRY(launch_gemm(ctx, d->precision, 0, 1, n, d->d_in, d->d_out, saved, d->ld_saved, W, ldw, G_in, d->ld_in,
                               gin, 0, s, &xlp));
    }
    return MIXGCN_OK;
}
