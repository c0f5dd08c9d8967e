// Node reordering for the fine-grain pipeline (Section 3.2.2 of the paper): graph bandwidth
// b = max over edges of p_v - p_u, the reverse Cuthill-McKee order that reduces it, the stage count
// ceil(2n / (n - b)) of Proposition 3.5, and a relabelled copy of a graph.  Everything runs on the
// device.  The ordering is a level-synchronous breadth-first search: a level's nodes are claimed by
// integer atomics (order-free), each with the position of its earliest-placed neighbour in the level
// above, and are then sorted by (that position, entry count, id) -- exactly the sequence in which a
// one-node-at-a-time Cuthill-McKee queue would have appended them.
#include <cub/cub.cuh>

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

namespace {

constexpr int32_t RCM_UNSEEN = -1;

// entries of row u other than the diagonal
__global__ void rcm_init_kernel(int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                int32_t* __restrict__ len, int32_t* __restrict__ ids, uint8_t* __restrict__ lonely,
                                int32_t* __restrict__ level_of, int32_t* __restrict__ parent) {
    const int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= n) return;
    const int64_t b = rowptr[u], e = rowptr[u + 1];
    int64_t off = e - b;
    for (int64_t i = b; i < e; ++i) if (col[i] == u) --off;
    len[u] = (int32_t)(e - b);
    ids[u] = (int32_t)u;
    lonely[u] = off == 0 ? 1 : 0;
    level_of[u] = RCM_UNSEEN;
    parent[u] = 0x7FFFFFFF;
}

// nodes without neighbours have the fewest entries of all and reach nothing: a one-at-a-time search
// places all of them first, in ascending id
__global__ void rcm_mark_placed_kernel(int64_t count, const int32_t* __restrict__ order, int32_t* __restrict__ level_of) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) level_of[order[i]] = 0;
}

// One block.  Advances *cursor over `by_len` (nodes by entry count, then id) to the first node not yet
// placed, places it at order[tail] and claims it for level `level`.
__global__ void rcm_next_start_kernel(int64_t n, const int32_t* __restrict__ by_len, int32_t* __restrict__ level_of,
                                      int64_t* cursor, int32_t* __restrict__ order, int64_t tail, int32_t level) {
    __shared__ long long found;
    long long at = *cursor;
    for (;;) {
        if (threadIdx.x == 0) found = (long long)n;
        __syncthreads();
        const long long i = at + threadIdx.x;
        if (i < n && level_of[by_len[i]] == RCM_UNSEEN) atomicMin(&found, i);
        __syncthreads();
        const long long f = found;
        __syncthreads();
        if (f < n || at + blockDim.x >= n) {
            if (threadIdx.x == 0) {
                *cursor = f < n ? f + 1 : (long long)n;
                if (f < n) { const int32_t s = by_len[f]; level_of[s] = level; order[tail] = s; }
            }
            return;
        }
        at += blockDim.x;
    }
}

// One warp per node of the current level (order[begin + i], i.e. the node at position begin + i): every
// neighbour not placed before this level is claimed for the next one (first claimant appends it to
// `cand`) and remembers the lowest position among its neighbours in the current level.
__global__ void rcm_expand_kernel(int64_t begin, int64_t count, const int32_t* __restrict__ order,
                                  const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                  int32_t* __restrict__ level_of, int32_t* __restrict__ parent, int32_t next_level,
                                  int32_t* __restrict__ cand, unsigned long long* __restrict__ n_cand) {
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (i >= count) return;
    const int32_t x = order[begin + i];
    const int32_t px = (int32_t)(begin + i);
    for (int64_t e = rowptr[x] + lane; e < rowptr[x + 1]; e += 32) {
        const int32_t y = col[e];
        int32_t st = level_of[y];
        if (st == RCM_UNSEEN) {
            st = atomicCAS(level_of + y, RCM_UNSEEN, next_level);
            if (st == RCM_UNSEEN) { cand[atomicAdd(n_cand, 1ull)] = y; st = next_level; }
        }
        if (st == next_level) atomicMin(parent + y, px);
    }
}

__global__ void rcm_keys_kernel(int64_t count, const int32_t* __restrict__ ids, const int32_t* __restrict__ parent,
                                const int32_t* __restrict__ len, uint64_t* __restrict__ keys) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) keys[i] = ((uint64_t)(uint32_t)parent[ids[i]] << 32) | (uint32_t)len[ids[i]];
}

__global__ void rcm_reverse_kernel(int64_t n, const int32_t* __restrict__ in, int32_t* __restrict__ out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = in[n - 1 - i];
}

}  // namespace

extern "C" mixgcn_status mixgcn_graph_rcm(const mixgcn_graph* g, int32_t* order) {
    if (!g || !order) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_rcm: null argument");
    if (!g->symmetric) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "graph_rcm: the stored matrix must be symmetric");
    MIXGCN_CUDA(cudaSetDevice(g->ctx->device));
    MIXGCN_CUDA(cudaDeviceSynchronize());
    const int64_t n = g->n;
    const int64_t* rowptr = g->fwd.rowptr;
    const int32_t* col = g->fwd.col;
    auto up = [](int64_t x) { return (x + 255) & ~(int64_t)255; };
    // temporary storage of the three library sorts / selections (the largest input is n)
    size_t t_sel = 0, t_len = 0, t_id = 0, t_key = 0;
    MIXGCN_CUDA(cub::DeviceSelect::Flagged(nullptr, t_sel, (int32_t*)nullptr, (uint8_t*)nullptr, (int32_t*)nullptr, (int64_t*)nullptr, n));
    MIXGCN_CUDA(cub::DeviceRadixSort::SortPairs(nullptr, t_len, (int32_t*)nullptr, (int32_t*)nullptr, (int32_t*)nullptr, (int32_t*)nullptr, n));
    MIXGCN_CUDA(cub::DeviceRadixSort::SortKeys(nullptr, t_id, (int32_t*)nullptr, (int32_t*)nullptr, n));
    MIXGCN_CUDA(cub::DeviceRadixSort::SortPairs(nullptr, t_key, (uint64_t*)nullptr, (uint64_t*)nullptr, (int32_t*)nullptr, (int32_t*)nullptr, n));
    const int64_t t_max = (int64_t)std::max(std::max(t_sel, t_len), std::max(t_id, t_key));
    const int64_t o_len = 0, o_ids = o_len + up(n * 4), o_lonely = o_ids + up(n * 4), o_level = o_lonely + up(n),
                  o_parent = o_level + up(n * 4), o_bylen = o_parent + up(n * 4), o_lensorted = o_bylen + up(n * 4),
                  o_order = o_lensorted + up(n * 4), o_cand = o_order + up(n * 4), o_cand2 = o_cand + up(n * 4),
                  o_keys = o_cand2 + up(n * 4), o_keys2 = o_keys + up(n * 8), o_scalars = o_keys2 + up(n * 8),
                  o_tmp = o_scalars + 256, total = o_tmp + up(t_max);
    DevMem mem;
    if (cudaMalloc(&mem.p, (size_t)total) != cudaSuccess) {
        cudaGetLastError();
        MIXGCN_FAIL(MIXGCN_ENOMEM, "graph_rcm: %lld bytes of device scratch could not be allocated", (long long)total);
    }
    char* base = reinterpret_cast<char*>(mem.p);
    int32_t* len = reinterpret_cast<int32_t*>(base + o_len);
    int32_t* ids = reinterpret_cast<int32_t*>(base + o_ids);
    uint8_t* lonely = reinterpret_cast<uint8_t*>(base + o_lonely);
    int32_t* level_of = reinterpret_cast<int32_t*>(base + o_level);
    int32_t* parent = reinterpret_cast<int32_t*>(base + o_parent);
    int32_t* by_len = reinterpret_cast<int32_t*>(base + o_bylen);
    int32_t* len_sorted = reinterpret_cast<int32_t*>(base + o_lensorted);
    int32_t* ord = reinterpret_cast<int32_t*>(base + o_order);
    int32_t* cand = reinterpret_cast<int32_t*>(base + o_cand);
    int32_t* cand2 = reinterpret_cast<int32_t*>(base + o_cand2);
    uint64_t* keys = reinterpret_cast<uint64_t*>(base + o_keys);
    uint64_t* keys2 = reinterpret_cast<uint64_t*>(base + o_keys2);
    int64_t* d_selected = reinterpret_cast<int64_t*>(base + o_scalars);
    int64_t* d_cursor = d_selected + 1;
    unsigned long long* d_ncand = reinterpret_cast<unsigned long long*>(d_selected + 2);
    void* tmp = base + o_tmp;
    size_t tb;
    cudaStream_t s = nullptr;
    const unsigned nb = (unsigned)((n + 255) / 256);

    LaunchScope scope(g->ctx, PH_GRAPH, s);
    rcm_init_kernel<<<nb, 256, 0, s>>>(n, rowptr, col, len, ids, lonely, level_of, parent);
    // start candidates: nodes by (entry count, id) -- a stable sort of the ascending ids by entry count
    tb = t_len;
    MIXGCN_CUDA(cub::DeviceRadixSort::SortPairs(tmp, tb, len, len_sorted, ids, by_len, n, 0, 32, s));
    // nodes without neighbours first, in ascending id
    tb = t_sel;
    MIXGCN_CUDA(cub::DeviceSelect::Flagged(tmp, tb, ids, lonely, ord, d_selected, n, s));
    int64_t tail = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&tail, d_selected, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaMemsetAsync(d_cursor, 0, sizeof(int64_t), s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    if (tail > 0) rcm_mark_placed_kernel<<<(unsigned)((tail + 255) / 256), 256, 0, s>>>(tail, ord, level_of);

    int32_t level = 1;
    int64_t begin = tail, count = 0;      // the current level is ord[begin, begin + count)
    while (tail < n) {
        if (count == 0) {
            // a new component starts from the unplaced node of fewest entries (lowest id on ties)
            rcm_next_start_kernel<<<1, 1024, 0, s>>>(n, by_len, level_of, d_cursor, ord, tail, level);
            begin = tail; count = 1; tail += 1;
            ++level;
            if (level == 0x7FFFFFF0) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "graph_rcm: too many levels");
            continue;
        }
        MIXGCN_CUDA(cudaMemsetAsync(d_ncand, 0, sizeof(unsigned long long), s));
        rcm_expand_kernel<<<(unsigned)((count * 32 + 255) / 256), 256, 0, s>>>(begin, count, ord, rowptr, col, level_of, parent,
                                                                                level, cand, d_ncand);
        unsigned long long m = 0;
        MIXGCN_CUDA(cudaMemcpyAsync(&m, d_ncand, sizeof(m), cudaMemcpyDeviceToHost, s));
        MIXGCN_CUDA(cudaStreamSynchronize(s));
        if (m > 0) {
            // (position of the earliest-placed neighbour, entry count, id): ids ascending first, then a
            // stable sort by the 64-bit (position, count) key
            const int64_t mm = (int64_t)m;
            tb = t_id;
            MIXGCN_CUDA(cub::DeviceRadixSort::SortKeys(tmp, tb, cand, cand2, mm, 0, 32, s));
            rcm_keys_kernel<<<(unsigned)((mm + 255) / 256), 256, 0, s>>>(mm, cand2, parent, len, keys);
            tb = t_key;
            MIXGCN_CUDA(cub::DeviceRadixSort::SortPairs(tmp, tb, keys, keys2, cand2, ord + tail, mm, 0, 64, s));
        }
        begin = tail; count = (int64_t)m; tail += (int64_t)m;
        ++level;
    }
    // reverse, then to the caller's host array
    rcm_reverse_kernel<<<nb, 256, 0, s>>>(n, ord, cand);
    MIXGCN_CUDA(cudaGetLastError());
    MIXGCN_CUDA(cudaMemcpy(order, cand, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
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
