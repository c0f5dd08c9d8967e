// One whole training iteration (the loop body of Algorithm 2) with host inputs and outputs:
// host -> device copies, all layers forward, loss, backward, Adam, device -> host copies.
// Device buffers come from an arena the context keeps between calls.
#include <new>
#include <vector>

#include "internal.cuh"

using namespace mixgcn;

// Row plans depend on the graph and the train mask only; a training loop calls with the same ones
// every iteration, so the plans of the last call are kept and reused while both are unchanged (the
// mask is compared byte by byte on the device).
struct HostStepCache {
    uint64_t graph_uid = 0;
    int64_t n = 0;
    int levels = 0;
    uint8_t* mask = nullptr;            // device copy of the train mask the plans were made from
    mixgcn_rowplan* plan[2] = {nullptr, nullptr};
};

// Feature prefetch between calls of mixgcn_train_step_host (see mixgcn_train_step_host_prefetch).
struct HostStepPrefetch {
    const float* announced = nullptr;   // host pointer the caller announced for the next call
    const float* in_flight = nullptr;   // host pointer whose copy into X[0] was started by the last call
    float* dst = nullptr;               // where it was copied to
    int64_t n = 0, d0 = 0;
    cudaEvent_t done = nullptr;         // recorded after that copy
};

namespace {

__global__ void mask_differs_kernel(int64_t n, const uint8_t* __restrict__ a, const uint8_t* __restrict__ b, int32_t* differs) {
    bool d = false;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        d |= (a[i] != 0) != (b[i] != 0);
    if (__any_sync(0xFFFFFFFFu, d) && (threadIdx.x & 31) == 0) *differs = 1;
}

void drop_plans(HostStepCache* c) {
    for (int i = 0; i < 2; ++i) { if (c->plan[i]) mixgcn_rowplan_destroy(c->plan[i]); c->plan[i] = nullptr; }
    c->graph_uid = 0; c->levels = 0;
}

inline int64_t round4(int64_t x) { return (x + 3) / 4 * 4; }

struct Carver {
    char* base; int64_t off = 0;
    template <class T> T* take(int64_t count) {
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += ((count * (int64_t)sizeof(T)) + 255) & ~(int64_t)255;
        return p;
    }
};

struct StepLayout {
    std::vector<float*> X, saved, G, W, b, dW, db, mW, vW, mb, vb;
    int32_t* labels; uint8_t* mask; float* loss; int32_t* pred;
    std::vector<uint8_t*> rowmask;   // [L] byte masks the row-sparse backward fills (layer l's input-gradient rows)
    std::vector<mixgcn_layer_desc> desc;
    int64_t bytes;
};

// Pass base == nullptr to size the arena.
mixgcn_status lay_out(char* base, int64_t n, int L, const int32_t* dims, int precision, StepLayout& lo) {
    Carver c{base};
    lo.desc.resize(L);
    std::vector<int64_t> ld(L + 1);
    for (int l = 0; l <= L; ++l) ld[l] = round4(dims[l]);
    for (int l = 0; l < L; ++l) {
        mixgcn_layer_desc& d = lo.desc[l];
        d = mixgcn_layer_desc{};
        d.d_in = dims[l]; d.d_out = dims[l + 1]; d.ld_in = ld[l]; d.ld_out = ld[l + 1]; d.ld_saved = 4;
        d.order = MIXGCN_ORDER_AUTO; d.precision = precision; d.keep_scale = 1.0f; d.in_scale = 1.0f; d.n_chunks = 0;
        d.flags = (l < L - 1 ? MIXGCN_LAYER_RELU : 0u) | (l == 0 ? MIXGCN_LAYER_FIRST : 0u) |
                  (l >= 1 ? MIXGCN_LAYER_GATE_GIN : 0u) | (l < L - 1 ? MIXGCN_LAYER_GOUT_GATED : 0u);
        int32_t order = 0, cols = 0;
        MIXGCN_TRY(mixgcn_layer_plan(&d, &order, &cols));
        d.order = order; d.ld_saved = round4(cols);
    }
    lo.X.resize(L + 1); lo.saved.resize(L); lo.G.assign(L + 1, nullptr);
    for (int l = 0; l <= L; ++l) lo.X[l] = c.take<float>(n * ld[l]);
    for (int l = 0; l < L; ++l) lo.saved[l] = c.take<float>(n * lo.desc[l].ld_saved);
    int64_t wmax = 4;
    for (int l = 1; l < L; ++l) wmax = ld[l] > wmax ? ld[l] : wmax;
    float* pool[2] = {nullptr, nullptr};
    if (L >= 2) pool[0] = c.take<float>(n * wmax);
    if (L >= 3) pool[1] = ld[L] >= wmax ? lo.X[L] : c.take<float>(n * wmax);
    lo.G[L] = lo.X[L];  // the logits' gradient overwrites the logits
    for (int l = L - 1, i = 0; l >= 1; --l, ++i) lo.G[l] = pool[i % 2];
    lo.labels = c.take<int32_t>(n); lo.mask = c.take<uint8_t>(n); lo.loss = c.take<float>(4); lo.pred = c.take<int32_t>(n);
    lo.rowmask.resize(L);
    for (int l = 0; l < L; ++l) lo.rowmask[l] = c.take<uint8_t>(n);
    // sign bitmaps of the hidden activations a dense product writes (agg-first layer below): the backward reads
    // its ReLU gates from them, one bit per element
    for (int l = 1; l < L; ++l) {
        if (lo.desc[l - 1].order != MIXGCN_ORDER_AGG_FIRST) continue;
        const int64_t words = (dims[l] + 31) / 32;
        uint32_t* bits = c.take<uint32_t>(n * words);
        lo.desc[l - 1].x_out_bits = bits; lo.desc[l - 1].ld_out_bits = words;
        lo.desc[l].x_in_bits = bits; lo.desc[l].ld_in_bits = words;
    }
    auto each = [&](std::vector<float*>& v, bool weight) {
        v.resize(L);
        for (int l = 0; l < L; ++l) v[l] = c.take<float>(weight ? (int64_t)dims[l] * dims[l + 1] : dims[l + 1]);
    };
    each(lo.W, true); each(lo.dW, true); each(lo.mW, true); each(lo.vW, true);
    each(lo.b, false); each(lo.db, false); each(lo.mb, false); each(lo.vb, false);
    lo.bytes = c.off;
    return MIXGCN_OK;
}

}  // namespace

namespace mixgcn {
void free_step_cache(mixgcn_ctx* ctx) {
    if (HostStepPrefetch* pf = ctx->step_prefetch) {
        if (pf->done) cudaEventDestroy(pf->done);
        delete pf;
        ctx->step_prefetch = nullptr;
    }
    HostStepCache* c = ctx->step_cache;
    if (!c) return;
    drop_plans(c);
    cudaFree(c->mask);
    delete c;
    ctx->step_cache = nullptr;
}
}  // namespace mixgcn

extern "C" mixgcn_status mixgcn_train_step_host(mixgcn_ctx* ctx, const mixgcn_graph* g, int32_t L,
                                                const int32_t* dims, int32_t precision, const float* X,
                                                const int32_t* labels, const uint8_t* train_mask,
                                                float* const* W, float* const* b, float* const* mW,
                                                float* const* vW, float* const* mb, float* const* vb,
                                                int64_t t, float lr, float beta1, float beta2, float eps,
                                                float* loss, int32_t* pred) {
    if (!ctx || !g || !dims || !X || !labels || !train_mask || !W || !b || !mW || !vW || !mb || !vb || !loss)
        MIXGCN_FAIL(MIXGCN_EINVAL, "train_step_host: null argument");
    if (L < 1 || L > 64) MIXGCN_FAIL(MIXGCN_EINVAL, "train_step_host: need 1 <= L <= 64 (got %d)", L);
    for (int l = 0; l <= L; ++l)
        if (dims[l] <= 0) MIXGCN_FAIL(MIXGCN_EINVAL, "train_step_host: dims[%d] must be positive", l);
    for (int l = 0; l < L; ++l)
        if (!W[l] || !b[l] || !mW[l] || !vW[l] || !mb[l] || !vb[l]) MIXGCN_FAIL(MIXGCN_EINVAL, "train_step_host: null tensor in layer %d", l);
    if (t < 1) MIXGCN_FAIL(MIXGCN_EINVAL, "train_step_host: t must be >= 1");
    if (dims[L] > 4096) MIXGCN_FAIL(MIXGCN_EINVAL, "train_step_host: at most 4096 classes");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    const int64_t n = g->n;
    StepLayout lo;
    MIXGCN_TRY(lay_out(nullptr, n, L, dims, precision, lo));
    HostStepPrefetch* pf = ctx->step_prefetch;
    if (lo.bytes > ctx->arena_bytes) {
        MIXGCN_CUDA(cudaDeviceSynchronize());
        if (pf) pf->in_flight = nullptr;        // the buffer a prefetch went to is gone
        cudaFree(ctx->arena); ctx->arena = nullptr; ctx->arena_bytes = 0;
        void* p = nullptr;
        if (cudaMalloc(&p, (size_t)lo.bytes) != cudaSuccess) {
            cudaGetLastError();
            MIXGCN_FAIL(MIXGCN_ENOMEM, "train_step_host: %lld bytes of device memory could not be allocated", (long long)lo.bytes);
        }
        ctx->arena = p; ctx->arena_bytes = lo.bytes;
        MIXGCN_CUDA(cudaMemset(p, 0, (size_t)lo.bytes));
        MIXGCN_CUDA(cudaDeviceSynchronize());   // the copies below run on a non-blocking stream: the clear must have finished
    }
    MIXGCN_TRY(lay_out(reinterpret_cast<char*>(ctx->arena), n, L, dims, precision, lo));
    cudaStream_t s = ctx->side_stream[0];
    const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;

    // Row sparsity of the backward pass: the loss gradient is non-zero on train rows only, and one
    // aggregation later on their neighbours only (same rule as the device-buffer trainer).  The row
    // plans are kept between calls and reused while the graph and the mask are the same.
    int64_t n_train = 0;
    for (int64_t i = 0; i < n; ++i) n_train += train_mask[i] ? 1 : 0;
    bool rows_only = false;
    MIXGCN_CUDA(cudaMemcpyAsync(lo.mask, train_mask, n * sizeof(uint8_t), H2D, s));
    {
        const double frac = (double)n_train / (double)n, mean_entries = (double)g->nnz / (double)n;
        int levels = frac >= 0.25 ? 0 : (frac * mean_entries < 0.5 ? 2 : 1);
        if (levels > L) levels = L;
        if (n_train == 0) levels = 0;
        if (levels > 0) {
            if (!ctx->step_cache) ctx->step_cache = new (std::nothrow) HostStepCache();
            HostStepCache* c = ctx->step_cache;
            if (!c) MIXGCN_FAIL(MIXGCN_ENOMEM, "train_step_host: host allocation failed");
            bool reuse = c->graph_uid == g->uid && c->n == n && c->levels == levels && c->mask;
            if (reuse) {
                int32_t* flag = reinterpret_cast<int32_t*>(lo.loss) + 1;      // spare words beside the loss scalar
                int32_t differs = 0;
                MIXGCN_CUDA(cudaMemsetAsync(flag, 0, sizeof(int32_t), s));
                mask_differs_kernel<<<(unsigned)(ctx->sm_count * 8), 256, 0, s>>>(n, lo.mask, c->mask, flag);
                MIXGCN_CUDA(cudaMemcpyAsync(&differs, flag, sizeof(int32_t), D2H, s));
                MIXGCN_CUDA(cudaStreamSynchronize(s));
                reuse = differs == 0;
            }
            if (!reuse) {
                drop_plans(c);
                if (c->n != n) { cudaFree(c->mask); c->mask = nullptr; c->n = 0; }
                if (!c->mask) { MIXGCN_CUDA(cudaMalloc((void**)&c->mask, (size_t)n)); c->n = n; }
                MIXGCN_CUDA(cudaStreamSynchronize(s));
                const uint8_t* in_mask = lo.mask;
                for (int i = 0; i < levels; ++i) {
                    MIXGCN_TRY(mixgcn_rowplan_create(ctx, g, 1, in_mask, &c->plan[i]));
                    if (i + 1 < levels) {
                        MIXGCN_TRY(mixgcn_rowplan_export(c->plan[i], nullptr, lo.rowmask[L - 1 - i], s));
                        MIXGCN_CUDA(cudaStreamSynchronize(s));
                        in_mask = lo.rowmask[L - 1 - i];
                    }
                }
                MIXGCN_CUDA(cudaMemcpyAsync(c->mask, lo.mask, (size_t)n, cudaMemcpyDeviceToDevice, s));
                c->graph_uid = g->uid; c->levels = levels;
            }
            for (int i = 0; i < levels; ++i) {
                const int l = L - 1 - i;
                lo.desc[l].gout_plan = c->plan[i];
                lo.desc[l].gout_row_mask = i == 0 ? lo.mask : nullptr;      // the forward's OUT_ROWS_ONLY reads it
                lo.desc[l].gout_row_count = c->plan[i]->in_count;
                if (l > 0 && i + 1 < levels) lo.desc[l].flags |= MIXGCN_LAYER_GIN_ROWS_ONLY;
            }
        }
        // Without `pred` nothing this call returns depends on the last layer's output outside the train
        // rows: compute that layer, the loss and its gradient on the train rows alone.
        rows_only = !pred && levels >= 1 && n_train > 0;
        if (rows_only) lo.desc[L - 1].flags |= MIXGCN_LAYER_OUT_ROWS_ONLY;
    }

    // inputs
    const int64_t d0 = dims[0], ld0 = round4(d0);
    auto copy_features = [&](const float* src, cudaStream_t st) -> cudaError_t {
        if (ld0 == d0) return cudaMemcpyAsync(lo.X[0], src, (size_t)(n * d0) * sizeof(float), H2D, st);
        return cudaMemcpy2DAsync(lo.X[0], ld0 * sizeof(float), src, d0 * sizeof(float), d0 * sizeof(float), (size_t)n, H2D, st);
    };
    if (pf && pf->in_flight == X && pf->dst == lo.X[0] && pf->n == n && pf->d0 == d0) {
        // the previous call already started this copy: wait for it instead of copying again
        MIXGCN_CUDA(cudaStreamWaitEvent(s, pf->done, 0));
    } else {
        if (pf && pf->in_flight) MIXGCN_CUDA(cudaStreamWaitEvent(s, pf->done, 0));   // a stale prefetch still writes X[0]: let it finish first
        MIXGCN_CUDA(copy_features(X, s));
    }
    if (pf) pf->in_flight = nullptr;
    MIXGCN_CUDA(cudaMemcpyAsync(lo.labels, labels, n * sizeof(int32_t), H2D, s));
    for (int l = 0; l < L; ++l) {
        const size_t wb = (size_t)dims[l] * dims[l + 1] * sizeof(float), bb = (size_t)dims[l + 1] * sizeof(float);
        MIXGCN_CUDA(cudaMemcpyAsync(lo.W[l], W[l], wb, H2D, s));
        MIXGCN_CUDA(cudaMemcpyAsync(lo.mW[l], mW[l], wb, H2D, s));
        MIXGCN_CUDA(cudaMemcpyAsync(lo.vW[l], vW[l], wb, H2D, s));
        MIXGCN_CUDA(cudaMemcpyAsync(lo.b[l], b[l], bb, H2D, s));
        MIXGCN_CUDA(cudaMemcpyAsync(lo.mb[l], mb[l], bb, H2D, s));
        MIXGCN_CUDA(cudaMemcpyAsync(lo.vb[l], vb[l], bb, H2D, s));
    }
    // forward, loss, backward, update
    auto after_first_layer = [&]() -> mixgcn_status {
        if (pf && pf->announced && lo.desc[0].order == MIXGCN_ORDER_AGG_FIRST) {
            // In agg-first order nothing after the first layer's forward reads the features again (its
            // backward uses A_hat X from `saved`): the announced features of the NEXT call are copied
            // into X[0] on the second stream while the rest of this iteration runs.
            cudaStream_t s2 = ctx->side_stream[1];
            MIXGCN_CUDA(cudaEventRecord(ctx->fork_ev, s));
            MIXGCN_CUDA(cudaStreamWaitEvent(s2, ctx->fork_ev, 0));
            MIXGCN_CUDA(copy_features(pf->announced, s2));
            MIXGCN_CUDA(cudaEventRecord(pf->done, s2));
            pf->in_flight = pf->announced; pf->dst = lo.X[0]; pf->n = n; pf->d0 = d0;
        }
        return MIXGCN_OK;
    };
    // With predictions wanted for every node the last layer and the loss are one call (the loss is taken where
    // the logits are produced, wherever the kernels allow; rows the backward never reads are left alone).
    const bool one_call = pred != nullptr && !rows_only;
    for (int l = 0; l < (one_call ? L - 1 : L); ++l) {
        MIXGCN_TRY(mixgcn_layer_fwd(ctx, g, &lo.desc[l], lo.X[l], lo.W[l], lo.b[l], nullptr, lo.saved[l], lo.X[l + 1], s));
        if (l == 0) MIXGCN_TRY(after_first_layer());
    }
    {
        const int keep = ctx->loss_train_rows_only;
        mixgcn_status st;
        if (one_call) {
            ctx->loss_train_rows_only = lo.desc[L - 1].gout_plan ? 2 : 0;
            st = mixgcn_layer_fwd_loss(ctx, g, &lo.desc[L - 1], lo.X[L - 1], lo.W[L - 1], lo.b[L - 1], lo.saved[L - 1], lo.X[L],
                                       lo.labels, lo.mask, lo.loss, lo.pred, nullptr, s);
        } else {
            ctx->loss_train_rows_only = rows_only ? 1 : keep;
            st = mixgcn_loss_softmax_xent(ctx, n, dims[L], lo.X[L], round4(dims[L]), lo.labels, lo.mask, lo.loss,
                                          lo.X[L], pred ? lo.pred : nullptr, nullptr, s);
        }
        ctx->loss_train_rows_only = keep;
        MIXGCN_TRY(st);
        if (one_call && L == 1) MIXGCN_TRY(after_first_layer());
    }
    if (pf) pf->announced = nullptr;
    for (int l = L - 1; l >= 0; --l) {
        MIXGCN_TRY(mixgcn_layer_bwd(ctx, g, &lo.desc[l], lo.X[l], lo.saved[l], lo.X[l + 1], nullptr, lo.W[l], lo.G[l + 1],
                                    l > 0 ? lo.G[l] : nullptr, lo.dW[l], lo.db[l], s));
    }
    std::vector<float*> P, M1, M2; std::vector<const float*> Gr; std::vector<int64_t> numel;
    for (int l = 0; l < L; ++l) { P.push_back(lo.W[l]); Gr.push_back(lo.dW[l]); M1.push_back(lo.mW[l]); M2.push_back(lo.vW[l]); numel.push_back((int64_t)dims[l] * dims[l + 1]); }
    for (int l = 0; l < L; ++l) { P.push_back(lo.b[l]); Gr.push_back(lo.db[l]); M1.push_back(lo.mb[l]); M2.push_back(lo.vb[l]); numel.push_back(dims[l + 1]); }
    MIXGCN_TRY(mixgcn_adam_step(ctx, 2 * L, P.data(), Gr.data(), M1.data(), M2.data(), numel.data(), t, lr, beta1, beta2, eps, s));
    // results
    MIXGCN_CUDA(cudaMemcpyAsync(loss, lo.loss, sizeof(float), D2H, s));
    if (pred) MIXGCN_CUDA(cudaMemcpyAsync(pred, lo.pred, n * sizeof(int32_t), D2H, s));
    for (int l = 0; l < L; ++l) {
        const size_t wb = (size_t)dims[l] * dims[l + 1] * sizeof(float), bb = (size_t)dims[l + 1] * sizeof(float);
        MIXGCN_CUDA(cudaMemcpyAsync(W[l], lo.W[l], wb, D2H, s));
        MIXGCN_CUDA(cudaMemcpyAsync(mW[l], lo.mW[l], wb, D2H, s));
        MIXGCN_CUDA(cudaMemcpyAsync(vW[l], lo.vW[l], wb, D2H, s));
        MIXGCN_CUDA(cudaMemcpyAsync(b[l], lo.b[l], bb, D2H, s));
        MIXGCN_CUDA(cudaMemcpyAsync(mb[l], lo.mb[l], bb, D2H, s));
        MIXGCN_CUDA(cudaMemcpyAsync(vb[l], lo.vb[l], bb, D2H, s));
    }
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_train_step_host_prefetch(mixgcn_ctx* ctx, const float* X_next) {
    if (!ctx) MIXGCN_FAIL(MIXGCN_EINVAL, "train_step_host_prefetch: null ctx");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    if (!ctx->step_prefetch) {
        HostStepPrefetch* pf = new (std::nothrow) HostStepPrefetch();
        if (!pf) MIXGCN_FAIL(MIXGCN_ENOMEM, "train_step_host_prefetch: host allocation failed");
        if (cudaEventCreateWithFlags(&pf->done, cudaEventDisableTiming) != cudaSuccess) {
            delete pf;
            MIXGCN_FAIL(MIXGCN_ECUDA, "train_step_host_prefetch: event creation failed");
        }
        ctx->step_prefetch = pf;
    }
    ctx->step_prefetch->announced = X_next;
    return MIXGCN_OK;
}
