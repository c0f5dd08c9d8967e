// Node reordering for the fine-grain pipeline (Section 3.2.2 of the paper): graph bandwidth
// b = max over edges of p_v - p_u, the reverse Cuthill-McKee order that reduces it, the stage count
// ceil(2n / (n - b)) of Proposition 3.5, and a relabelled copy of a graph.  As in the paper the
// ordering itself is a host (C++) preprocessing step -- a breadth-first search; the bandwidth of an
// order and the relabelling run on the device.
#include <algorithm>
#include <new>
#include <vector>

#include "internal.cuh"

using namespace mixgcn;

namespace {

__global__ void bandwidth_kernel(int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                 const int32_t* __restrict__ pos, unsigned long long* out) {
    const int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    long long best = 0;
    if (u < n) {
        const long long pu = pos ? pos[u] : u;
        for (int64_t i = rowptr[u] + lane; i < rowptr[u + 1]; i += 32) {
            const long long pv = pos ? pos[col[i]] : col[i];
            if (pv - pu > best) best = pv - pu;
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const long long other = __shfl_xor_sync(0xFFFFFFFFu, best, o);
        if (other > best) best = other;
    }
    if (lane == 0 && best > 0) atomicMax(out, (unsigned long long)best);   // integer maximum: order-free
}

// edges (pos[u], pos[v]) of every stored off-diagonal entry
__global__ void relabel_edges_kernel(int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                     const int32_t* __restrict__ pos, int32_t* __restrict__ src, int32_t* __restrict__ dst) {
    const int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (u >= n) return;
    const int32_t pu = pos[u];
    for (int64_t i = rowptr[u] + lane; i < rowptr[u + 1]; i += 32) { src[i] = pu; dst[i] = pos[col[i]]; }
}

struct DevMem {
    void* p = nullptr;
    ~DevMem() { if (p) cudaFree(p); }
};

mixgcn_status check_order(int64_t n, const int32_t* order, std::vector<int32_t>& pos) {
    pos.assign((size_t)n, -1);
    for (int64_t k = 0; k < n; ++k) {
        const int32_t u = order[k];
        if (u < 0 || u >= n || pos[(size_t)u] != -1) MIXGCN_FAIL(MIXGCN_EINVAL, "order is not a permutation of [0, n)");
        pos[(size_t)u] = (int32_t)k;
    }
    return MIXGCN_OK;
}

}  // namespace

extern "C" mixgcn_status mixgcn_pipeline_stages(int64_t n, int64_t b, int64_t* stages) {
    if (!stages || n <= 0 || b < 0) MIXGCN_FAIL(MIXGCN_EINVAL, "pipeline_stages: bad argument");
    if (b >= n) MIXGCN_FAIL(MIXGCN_EINVAL, "pipeline_stages: bandwidth %lld leaves no independent batch (n = %lld)", (long long)b, (long long)n);
    *stages = (2 * n + (n - b) - 1) / (n - b);
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_graph_bandwidth(const mixgcn_graph* g, const int32_t* order, int64_t* bandwidth) {
    if (!g || !bandwidth) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_bandwidth: null argument");
    MIXGCN_CUDA(cudaSetDevice(g->ctx->device));
    const int64_t n = g->n;
    DevMem dpos, dout;
    if (order) {
        std::vector<int32_t> pos;
        MIXGCN_TRY(check_order(n, order, pos));
        MIXGCN_CUDA(cudaMalloc(&dpos.p, n * sizeof(int32_t)));
        MIXGCN_CUDA(cudaMemcpy(dpos.p, pos.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice));
    }
    MIXGCN_CUDA(cudaMalloc(&dout.p, sizeof(unsigned long long)));
    MIXGCN_CUDA(cudaMemset(dout.p, 0, sizeof(unsigned long long)));
    {
        LaunchScope scope(g->ctx, PH_GRAPH, nullptr);
        bandwidth_kernel<<<(unsigned)((n * 32 + 255) / 256), 256>>>(n, g->fwd.rowptr, g->fwd.col,
                                                                   reinterpret_cast<const int32_t*>(dpos.p),
                                                                   reinterpret_cast<unsigned long long*>(dout.p));
    }
    unsigned long long b = 0;
    MIXGCN_CUDA(cudaMemcpy(&b, dout.p, sizeof(b), cudaMemcpyDeviceToHost));
    *bandwidth = (int64_t)b;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_graph_rcm(const mixgcn_graph* g, int32_t* order) {
    if (!g || !order) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_rcm: null argument");
    if (!g->symmetric) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "graph_rcm: the stored matrix must be symmetric");
    MIXGCN_CUDA(cudaSetDevice(g->ctx->device));
    MIXGCN_CUDA(cudaDeviceSynchronize());
    const int64_t n = g->n, nnz = g->nnz;
    std::vector<int64_t> rowptr;
    std::vector<int32_t> col, by_len, nb;
    std::vector<uint8_t> seen;
    try {
        rowptr.resize((size_t)n + 1); col.resize((size_t)(nnz > 0 ? nnz : 1)); by_len.resize((size_t)n); seen.assign((size_t)n, 0);
    } catch (const std::bad_alloc&) {
        MIXGCN_FAIL(MIXGCN_ENOMEM, "graph_rcm: host allocation failed");
    }
    MIXGCN_CUDA(cudaMemcpy(rowptr.data(), g->fwd.rowptr, (n + 1) * sizeof(int64_t), cudaMemcpyDeviceToHost));
    if (nnz) MIXGCN_CUDA(cudaMemcpy(col.data(), g->fwd.col, nnz * sizeof(int32_t), cudaMemcpyDeviceToHost));
    auto len = [&](int32_t u) { return rowptr[(size_t)u + 1] - rowptr[(size_t)u]; };
    // start candidates: nodes by (entry count, id)
    for (int64_t u = 0; u < n; ++u) by_len[(size_t)u] = (int32_t)u;
    std::stable_sort(by_len.begin(), by_len.end(), [&](int32_t a, int32_t b) { return len(a) < len(b); });
    int64_t head = 0, tail = 0, next_start = 0;
    while (tail < n) {
        while (seen[(size_t)by_len[(size_t)next_start]]) ++next_start;
        const int32_t s = by_len[(size_t)next_start];
        seen[(size_t)s] = 1; order[tail++] = s;
        while (head < tail) {
            const int32_t x = order[head++];
            nb.clear();
            for (int64_t i = rowptr[(size_t)x]; i < rowptr[(size_t)x + 1]; ++i) {
                const int32_t y = col[(size_t)i];
                if (!seen[(size_t)y]) { seen[(size_t)y] = 1; nb.push_back(y); }
            }
            // unvisited neighbours by increasing entry count; the CSR row is in ascending id, so a stable
            // sort keeps the lower id first among equals
            std::stable_sort(nb.begin(), nb.end(), [&](int32_t a, int32_t b) { return len(a) < len(b); });
            for (int32_t y : nb) order[tail++] = y;
        }
    }
    std::reverse(order, order + n);
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_graph_create_permuted(mixgcn_ctx* ctx, const mixgcn_graph* g, const int32_t* order,
                                                      mixgcn_graph** out) {
    if (!ctx || !g || !order || !out) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_create_permuted: null argument");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    const int64_t n = g->n, nnz = g->nnz;
    if (g->has_diagonal == 2) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "graph_create_permuted: only some rows store their diagonal entry");
    std::vector<int32_t> pos;
    MIXGCN_TRY(check_order(n, order, pos));
    DevMem dpos, dsrc, ddst;
    MIXGCN_CUDA(cudaMalloc(&dpos.p, n * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMalloc(&dsrc.p, (nnz > 0 ? nnz : 1) * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMalloc(&ddst.p, (nnz > 0 ? nnz : 1) * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMemcpy(dpos.p, pos.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice));
    {
        LaunchScope scope(ctx, PH_GRAPH, nullptr);
        relabel_edges_kernel<<<(unsigned)((n * 32 + 255) / 256), 256>>>(n, g->fwd.rowptr, g->fwd.col,
                                                                       reinterpret_cast<const int32_t*>(dpos.p),
                                                                       reinterpret_cast<int32_t*>(dsrc.p),
                                                                       reinterpret_cast<int32_t*>(ddst.p));
    }
    MIXGCN_CUDA(cudaDeviceSynchronize());
    // Every stored entry is carried over; the diagonal (if the source has one) comes back through ADD_SELF_LOOPS.
    return mixgcn_graph_create(ctx, n, nnz, reinterpret_cast<const int32_t*>(dsrc.p), reinterpret_cast<const int32_t*>(ddst.p),
                               MIXGCN_GRAPH_EDGES_ON_DEVICE | (g->has_diagonal == 1 ? MIXGCN_GRAPH_ADD_SELF_LOOPS : 0u) |
                                   (g->norm == 1 ? MIXGCN_GRAPH_NORM_ROW : (g->norm == 2 ? MIXGCN_GRAPH_NORM_NONE : 0u)), out);
}
