// Row plans for the row-sparse backward pass.  Which rows of a gradient are non-zero depends on the
// graph and the train mask only (the loss gradient lives on train rows, one aggregation later on
// their neighbours), so everything that follows from it is computed once: the list of kept rows and
// the CSR of A_hat^T restricted to the kept columns, renumbered to positions in the compacted input,
// with its own aggregation schedule.  A row-sparse aggregation is then the ordinary kernel on a
// smaller matrix and a compact input: the dense sum with its exactly-zero terms left out, entries
// in the same order.  (The paper's sampled SpMM, Eq. 4, skips work by a mask on the output; here the
// mask is on the operand's rows and the skipping is done ahead of time.)
#include <cub/cub.cuh>
#include <thrust/iterator/counting_iterator.h>

#include <new>

#include "internal.cuh"

using namespace mixgcn;

namespace {

struct DevMem {
    void* p = nullptr;
    ~DevMem() { if (p) cudaFree(p); }
    template <class T> T* as() { return reinterpret_cast<T*>(p); }
};

__global__ void pos_fill_kernel(int64_t count, const int32_t* __restrict__ idx, int32_t* __restrict__ pos) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) pos[idx[i]] = (int32_t)i;
}

// kept entries per row (one warp per row); out_mask[u] = 1 iff the row keeps at least one entry
__global__ void kept_count_kernel(int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                  const uint8_t* __restrict__ mask, int64_t* __restrict__ cnt, uint8_t* __restrict__ out_mask) {
    const int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (u >= n) return;
    const int64_t b = rowptr[u], e = rowptr[u + 1];
    int c = 0;
    for (int64_t i = b + lane; i < e; i += 32) c += mask[col[i]] ? 1 : 0;
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
    if (lane == 0) { cnt[u] = c; out_mask[u] = c > 0 ? 1 : 0; }
}

// number of non-zero bytes (integer sum: order-free)
__global__ void count_nonzero_kernel(int64_t n, const uint8_t* __restrict__ m, unsigned long long* out) {
    unsigned int c = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        c += m[i] ? 1u : 0u;
    for (int o = 16; o > 0; o >>= 1) c += __shfl_down_sync(0xFFFFFFFFu, c, o);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(out, (unsigned long long)c);
}

// kept entries of a row, in entry order, with column ids renumbered through pos
__global__ void kept_fill_kernel(int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                 const float* __restrict__ val, const uint8_t* __restrict__ mask,
                                 const int32_t* __restrict__ pos, const int64_t* __restrict__ rowptr2,
                                 int32_t* __restrict__ col2, float* __restrict__ val2) {
    const int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (u >= n) return;
    const int64_t b = rowptr[u], e = rowptr[u + 1];
    int64_t w = rowptr2[u];
    if (rowptr2[u + 1] == w) return;
    for (int64_t i0 = b; i0 < e; i0 += 32) {
        const int64_t i = i0 + lane;
        int c = -1;
        if (i < e) { const int cc = col[i]; if (mask[cc]) c = cc; }
        const unsigned keep = __ballot_sync(0xFFFFFFFFu, c >= 0);
        if (c >= 0) {
            const int64_t at = w + __popc(keep & ((1u << lane) - 1u));
            col2[at] = pos[c];
            val2[at] = val[i];
        }
        w += __popc(keep);
    }
}

}  // namespace

extern "C" mixgcn_status mixgcn_rowplan_destroy(mixgcn_rowplan* p) {
    if (!p) return MIXGCN_OK;
    cudaSetDevice(p->device);
    cudaDeviceSynchronize();
    cudaFree(p->idx);
    cudaFree(p->out_mask);
    release_view(p->view);
    delete p;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_rowplan_create(mixgcn_ctx* ctx, const mixgcn_graph* g, int transposed,
                                               const uint8_t* in_row_mask, mixgcn_rowplan** out) {
    if (!ctx || !g || !in_row_mask || !out) MIXGCN_FAIL(MIXGCN_EINVAL, "rowplan_create: null argument");
    *out = nullptr;
    if (g->ctx != ctx) MIXGCN_FAIL(MIXGCN_EINVAL, "rowplan_create: the graph belongs to another context");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    MIXGCN_CUDA(cudaDeviceSynchronize());   // the mask may have been written on any stream
    const int64_t n = g->n;
    const CsrView& A = transposed ? g->bwd : g->fwd;
    cudaStream_t s = nullptr;
    LaunchScope scope(ctx, PH_GRAPH, s, 8);
    mixgcn_rowplan* p = new (std::nothrow) mixgcn_rowplan();
    if (!p) MIXGCN_FAIL(MIXGCN_ENOMEM, "rowplan_create: host allocation failed");
    p->ctx = ctx; p->device = ctx->device; p->g = g; p->transposed = transposed ? 1 : 0; p->n = n;
    struct Guard { mixgcn_rowplan* p; ~Guard() { if (p) mixgcn_rowplan_destroy(p); } } guard{p};

    // kept rows, ascending, and their positions
    DevMem sel, tmp, pos, cnt;
    size_t tb = 0;
    thrust::counting_iterator<int32_t> ids(0);
    MIXGCN_CUDA(cudaMalloc((void**)&p->idx, (size_t)(n > 0 ? n : 1) * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMalloc(&sel.p, sizeof(int64_t)));
    MIXGCN_CUDA(cub::DeviceSelect::Flagged(nullptr, tb, ids, in_row_mask, p->idx, sel.as<int64_t>(), n, s));
    MIXGCN_CUDA(cudaMalloc(&tmp.p, tb ? tb : 1));
    MIXGCN_CUDA(cub::DeviceSelect::Flagged(tmp.p, tb, ids, in_row_mask, p->idx, sel.as<int64_t>(), n, s));
    int64_t in_count = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&in_count, sel.p, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    p->in_count = in_count;
    MIXGCN_CUDA(cudaMalloc(&pos.p, (size_t)(n > 0 ? n : 1) * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMemsetAsync(pos.p, 0xFF, (size_t)n * sizeof(int32_t), s));
    if (in_count > 0)
        pos_fill_kernel<<<(unsigned)((in_count + 255) / 256), 256, 0, s>>>(in_count, p->idx, pos.as<int32_t>());

    // restricted CSR: per-row kept counts -> row pointers -> entries
    CsrView& V = p->view;
    V = CsrView{};
    MIXGCN_CUDA(cudaMalloc((void**)&p->out_mask, (size_t)(n > 0 ? n : 1)));
    MIXGCN_CUDA(cudaMalloc(&cnt.p, (size_t)(n + 1) * sizeof(int64_t)));
    MIXGCN_CUDA(cudaMemsetAsync(cnt.p, 0, (size_t)(n + 1) * sizeof(int64_t), s));
    MIXGCN_CUDA(cudaMalloc((void**)&V.rowptr, (size_t)(n + 1) * sizeof(int64_t)));
    const unsigned row_blocks = (unsigned)((n * 32 + 255) / 256);
    if (n > 0) kept_count_kernel<<<row_blocks, 256, 0, s>>>(n, A.rowptr, A.col, in_row_mask, cnt.as<int64_t>(), p->out_mask);
    DevMem tmp2;
    size_t tb2 = 0;
    MIXGCN_CUDA(cub::DeviceScan::ExclusiveSum(nullptr, tb2, cnt.as<int64_t>(), V.rowptr, n + 1, s));
    MIXGCN_CUDA(cudaMalloc(&tmp2.p, tb2 ? tb2 : 1));
    MIXGCN_CUDA(cub::DeviceScan::ExclusiveSum(tmp2.p, tb2, cnt.as<int64_t>(), V.rowptr, n + 1, s));
    int64_t nnz2 = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&nnz2, V.rowptr + n, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
    // rows with a kept entry
    DevMem oc;
    MIXGCN_CUDA(cudaMalloc(&oc.p, sizeof(unsigned long long)));
    MIXGCN_CUDA(cudaMemsetAsync(oc.p, 0, sizeof(unsigned long long), s));
    if (n > 0) {
        int64_t cb = (n + 255) / 256;
        if (cb > (int64_t)ctx->sm_count * 16) cb = (int64_t)ctx->sm_count * 16;
        count_nonzero_kernel<<<(unsigned)cb, 256, 0, s>>>(n, p->out_mask, oc.as<unsigned long long>());
    }
    int64_t out_count = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&out_count, oc.p, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    p->nnz = nnz2; p->out_count = out_count;
    MIXGCN_CUDA(cudaMalloc((void**)&V.col, (size_t)(nnz2 > 0 ? nnz2 : 1) * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMalloc((void**)&V.val, (size_t)(nnz2 > 0 ? nnz2 : 1) * sizeof(float)));
    if (n > 0 && nnz2 > 0)
        kept_fill_kernel<<<row_blocks, 256, 0, s>>>(n, A.rowptr, A.col, A.val, in_row_mask, pos.as<int32_t>(), V.rowptr, V.col, V.val);
    MIXGCN_CUDA(cudaGetLastError());
    MIXGCN_TRY(build_view_schedule(in_count > 0 ? in_count : 1, n, V, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    guard.p = nullptr;
    *out = p;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_rowplan_info(const mixgcn_rowplan* p, int64_t* in_count, int64_t* out_count,
                                             int64_t* nnz) {
    if (!p) MIXGCN_FAIL(MIXGCN_EINVAL, "rowplan_info: null plan");
    if (in_count) *in_count = p->in_count;
    if (out_count) *out_count = p->out_count;
    if (nnz) *nnz = p->nnz;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_rowplan_export(const mixgcn_rowplan* p, int32_t* in_rows, uint8_t* out_row_mask,
                                               void* stream) {
    if (!p) MIXGCN_FAIL(MIXGCN_EINVAL, "rowplan_export: null plan");
    MIXGCN_CUDA(cudaSetDevice(p->device));
    cudaStream_t s = (cudaStream_t)stream;
    if (in_rows && p->in_count > 0)
        MIXGCN_CUDA(cudaMemcpyAsync(in_rows, p->idx, (size_t)p->in_count * sizeof(int32_t), cudaMemcpyDeviceToDevice, s));
    if (out_row_mask && p->n > 0)
        MIXGCN_CUDA(cudaMemcpyAsync(out_row_mask, p->out_mask, (size_t)p->n, cudaMemcpyDeviceToDevice, s));
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_spmm_rowplan(mixgcn_ctx* ctx, const mixgcn_rowplan* p, int32_t w, const float* Yc,
                                             int64_t ldy, float* Z, int64_t ldz, const mixgcn_epilogue* epi,
                                             int32_t rows_only, void* stream) {
    if (!ctx || !p || !Z || (!Yc && p->in_count > 0)) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_rowplan: null argument");
    if (p->ctx != ctx) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_rowplan: the plan belongs to another context");
    if (w <= 0) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_rowplan: w must be positive (got %d)", w);
    if (ldy < w || ldz < w || (ldy & 3) || (ldz & 3))
        MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_rowplan: leading dimensions must be multiples of 4 and >= w (ldy=%lld ldz=%lld w=%d)",
                    (long long)ldy, (long long)ldz, w);
    if (!aligned16(Yc) || !aligned16(Z)) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_rowplan: Yc and Z must be 16-byte aligned");
    if (Yc == Z) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_rowplan: Yc and Z must not overlap");
    if (epi && epi->gate && epi->ld_gate < w) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_rowplan: gate leading dimension < w");
    if (epi && epi->residual && (epi->ld_residual < w || epi->residual == Z)) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_rowplan: residual needs ld_residual >= w and must not be the output");
    if (epi && epi->residual && rows_only) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "spmm_rowplan: rows_only cannot be combined with a residual (rows without a kept entry are not zero then)");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    // rows of the restricted matrix are scheduled longest first, so its non-empty rows are the first out_count
    SpmmOpts opts;
    opts.phase = PH_SPMM_SPARSE;
    opts.row_limit = rows_only ? p->out_count : -1;
    opts.y_rows = p->in_count; opts.nnz = p->nnz;
    return launch_spmm(ctx, p->g, p->view, 1, 0, w, Yc, ldy, Z, ldz, epi, (cudaStream_t)stream, opts);
}
