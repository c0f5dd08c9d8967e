// Graph construction on the device: edge list -> A + I in CSR -> symmetric normalisation
// A_hat = D^-1/2 (A+I) D^-1/2 (Section 2.1 of the paper) -> CSR of the transpose (aliased when
// symmetric) -> degree-sorted row schedule.  Sorting, run-length and selection steps use CUB
// device primitives; everything else is a kernel in this file.
#include <cub/cub.cuh>

#include <new>

#include "internal.cuh"

using namespace mixgcn;

#include <atomic>

namespace {

uint64_t next_graph_uid() {
    static std::atomic<uint64_t> counter{0};
    return ++counter;
}

constexpr int TPB = 256;
inline unsigned blocks_for(int64_t n) { return (unsigned)((n + TPB - 1) / TPB); }

// flag bits written by validation kernels
enum { F_BAD_ID = 1, F_NOT_SYMMETRIC = 2, F_BAD_ROWPTR = 4, F_UNSORTED = 8 };

__global__ void make_keys_kernel(int64_t n, int64_t m, const int32_t* __restrict__ src,
                                 const int32_t* __restrict__ dst, int sym, int self_loops,
                                 uint64_t sentinel, uint64_t* __restrict__ keys, int32_t* flags) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) {
        int32_t u = src[i], v = dst[i];
        bool bad = u < 0 || v < 0 || u >= n || v >= n;
        if (bad) atomicOr(flags, F_BAD_ID);
        bool drop = bad || u == v;
        keys[i] = drop ? sentinel : (((uint64_t)(uint32_t)u << 32) | (uint32_t)v);
        if (sym) keys[m + i] = drop ? sentinel : (((uint64_t)(uint32_t)v << 32) | (uint32_t)u);
    }
    if (self_loops && i < n) {
        int64_t base = sym ? 2 * m : m;
        keys[base + i] = ((uint64_t)i << 32) | (uint64_t)i;
    }
}

// rowptr[q] = first position whose row id is >= q, from the sorted unique keys.
__global__ void rowptr_from_keys_kernel(int64_t n, int64_t nnz, const uint64_t* __restrict__ keys,
                                        int64_t* __restrict__ rowptr, int32_t* __restrict__ col) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nnz) {
        int64_t r = (int64_t)(keys[i] >> 32);
        int64_t rp = i == 0 ? -1 : (int64_t)(keys[i - 1] >> 32);
        for (int64_t q = rp + 1; q <= r; ++q) rowptr[q] = i;
        col[i] = (int32_t)(uint32_t)(keys[i] & 0xFFFFFFFFull);
    } else if (i == nnz) {
        int64_t last = nnz == 0 ? -1 : (int64_t)(keys[nnz - 1] >> 32);
        for (int64_t q = last + 1; q <= n; ++q) rowptr[q] = nnz;
    }
}

__global__ void degree_kernel(int64_t n, const int64_t* __restrict__ rowptr, int32_t* __restrict__ deg,
                              float* __restrict__ dinv) {
    int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= n) return;
    int32_t d = (int32_t)(rowptr[u + 1] - rowptr[u]);
    deg[u] = d;
    // dinv = 1/sqrt(deg): IEEE square root, then IEEE reciprocal, each rounded to fp32.
    dinv[u] = d > 0 ? __frcp_rn(__fsqrt_rn((float)d)) : 0.0f;
}

// One warp per row.  norm 0: val_uv = dinv_u * dinv_v (Section 2.1); 1: 1 / (entries in row u), the row
// mean (GraphSAGE's mean aggregator); 2: 1, the plain sum (GIN's sum aggregator).
__global__ void values_kernel(int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                              const float* __restrict__ dinv, int norm, float* __restrict__ val) {
    int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (u >= n) return;
    const int64_t b = rowptr[u], e = rowptr[u + 1];
    if (norm == 0) {
        float du = dinv[u];
        for (int64_t i = b + lane; i < e; i += 32) val[i] = __fmul_rn(du, dinv[col[i]]);
    } else {
        const float v = norm == 1 ? __frcp_rn((float)(e - b)) : 1.0f;   // IEEE reciprocal of the entry count
        for (int64_t i = b + lane; i < e; i += 32) val[i] = v;
    }
}

// For every stored (u,v), u != v, look v's row up for u.
__global__ void symmetry_kernel(int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                int32_t* flags) {
    int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (u >= n) return;
    for (int64_t i = rowptr[u] + lane; i < rowptr[u + 1]; i += 32) {
        int32_t v = col[i];
        if (v == u) continue;
        int64_t lo = rowptr[v], hi = rowptr[v + 1];
        bool found = false;
        while (lo < hi) {
            int64_t mid = (lo + hi) >> 1;
            int32_t c = col[mid];
            if (c == (int32_t)u) { found = true; break; }
            if (c < (int32_t)u) lo = mid + 1; else hi = mid;
        }
        if (!found) { atomicOr(flags, F_NOT_SYMMETRIC); return; }
    }
}

// Rows that store their own diagonal entry (binary search of u in row u).
__global__ void diagonal_count_kernel(int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                      unsigned long long* count) {
    const int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    bool has = false;
    if (u < n) {
        int64_t lo = rowptr[u], hi = rowptr[u + 1];
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            const int32_t c = col[mid];
            if (c == (int32_t)u) { has = true; break; }
            if (c < (int32_t)u) lo = mid + 1; else hi = mid;
        }
    }
    const unsigned b = __ballot_sync(0xFFFFFFFFu, has);
    if ((threadIdx.x & 31) == 0 && b) atomicAdd(count, (unsigned long long)__popc(b));
}

__global__ void transpose_keys_kernel(int64_t n, const int64_t* __restrict__ rowptr,
                                      const int32_t* __restrict__ col, uint64_t* __restrict__ keys) {
    int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (u >= n) return;
    for (int64_t i = rowptr[u] + lane; i < rowptr[u + 1]; i += 32)
        keys[i] = ((uint64_t)(uint32_t)col[i] << 32) | (uint32_t)u;
}

__global__ void schedule_keys_kernel(int64_t row0, int64_t n_rows, const int64_t* __restrict__ rowptr,
                                     uint64_t* __restrict__ keys) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_rows) return;
    const int64_t u = row0 + i;
    uint64_t d = (uint64_t)(rowptr[u + 1] - rowptr[u]);
    keys[i] = ((0x7FFFFFFFull - d) << 32) | (uint64_t)u;  // descending entries, ascending id
}

// perm from the sorted keys; counts[0] = rows longer than SPMM_SEG, counts[1..3] = rows longer than
// SPMM_PACK_DEG[0..2] (one atomic per warp and counter; integers, so order does not matter).
__global__ void schedule_finish_kernel(int64_t n, const uint64_t* __restrict__ keys, int32_t* __restrict__ perm,
                                       unsigned long long* counts) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t d = -1;
    if (i < n) {
        perm[i] = (int32_t)(uint32_t)(keys[i] & 0xFFFFFFFFull);
        d = (int64_t)(0x7FFFFFFFull - (keys[i] >> 32));
    }
    const int thr[4] = {SPMM_SEG, SPMM_PACK_DEG[0], SPMM_PACK_DEG[1], SPMM_PACK_DEG[2]};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        unsigned b = __ballot_sync(0xFFFFFFFFu, d > thr[q]);
        if ((threadIdx.x & 31) == 0 && b) atomicAdd(counts + q, (unsigned long long)__popc(b));
    }
}

// Long rows are cut at dyadic column-block boundaries (and every SPMM_SEG entries): a row with d
// entries uses 2^k blocks, the largest k <= SPMM_MAX_LOG_BLOCKS with d / 2^k >= SPMM_BLK_MIN_ENTRIES.
__device__ __forceinline__ int row_log_blocks(int64_t d) {
    int k = 0;
    while (k < SPMM_MAX_LOG_BLOCKS && (d >> (k + 1)) >= SPMM_BLK_MIN_ENTRIES) ++k;
    return k;
}

__global__ void blk_count_kernel(int64_t n_long, const int32_t* __restrict__ perm, const int64_t* __restrict__ rowptr,
                                 int64_t* __restrict__ nblk) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i > n_long) return;
    if (i == n_long) { nblk[i] = 0; return; }
    const int64_t u = perm[i];
    nblk[i] = (int64_t)1 << row_log_blocks(rowptr[u + 1] - rowptr[u]);
}

__device__ __forceinline__ int64_t lower_bound_col(const int32_t* __restrict__ col, int64_t lo, int64_t hi, int64_t key) {
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if ((int64_t)col[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// largest i with off[i] <= t  (off is ascending, off[0] = 0, off[count] > t)
__device__ __forceinline__ int64_t owner_of(const int64_t* __restrict__ off, int64_t count, int64_t t) {
    int64_t lo = 0, hi = count;
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (off[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// One thread per (long row, column block) pair: the entries of the row inside the block and how many
// segments they need.
__global__ void pair_segments_kernel(int64_t n, int64_t n_long, int64_t total_pairs, const int32_t* __restrict__ perm,
                                     const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                     const int64_t* __restrict__ blk_off, int64_t* __restrict__ pair_lo,
                                     int64_t* __restrict__ pair_cnt, int64_t* __restrict__ pair_segs) {
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t > total_pairs) return;
    if (t == total_pairs) { pair_segs[t] = 0; return; }
    const int64_t i = owner_of(blk_off, n_long, t);
    const int64_t b = t - blk_off[i], nb = blk_off[i + 1] - blk_off[i];
    const int64_t u = perm[i];
    const int64_t rb = rowptr[u], re = rowptr[u + 1];
    const int64_t width = (n + nb - 1) / nb;
    const int64_t lo = lower_bound_col(col, rb, re, b * width);
    const int64_t hi = lower_bound_col(col, lo, re, (b + 1) * width);
    pair_lo[t] = lo;
    pair_cnt[t] = hi - lo;
    pair_segs[t] = (hi - lo + SPMM_SEG - 1) / SPMM_SEG;
}

__global__ void seg_fill_kernel(int64_t n_long, int64_t total_pairs, const int32_t* __restrict__ col,
                                const int64_t* __restrict__ blk_off, const int64_t* __restrict__ pair_lo,
                                const int64_t* __restrict__ pair_cnt, const int64_t* __restrict__ pair_seg_off,
                                SpmmRec* __restrict__ rec_tmp, uint32_t* __restrict__ keys, uint32_t* __restrict__ ids,
                                int64_t* __restrict__ seg_off) {
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total_pairs) return;
    const int64_t i = owner_of(blk_off, n_long, t);
    if (t == blk_off[i]) seg_off[i] = pair_seg_off[t];
    if (t == total_pairs - 1) seg_off[n_long] = pair_seg_off[total_pairs];
    int64_t q = pair_seg_off[t];
    const int64_t lo = pair_lo[t], hi = lo + pair_cnt[t];
    for (int64_t pos = lo; pos < hi; pos += SPMM_SEG, ++q) {
        SpmmRec x; x.begin = pos; x.len = (int32_t)((hi - pos) < SPMM_SEG ? (hi - pos) : SPMM_SEG); x.row = (int32_t)i;
        rec_tmp[q] = x;
        keys[q] = (uint32_t)col[pos];      // segments run in order of their first column
        ids[q] = (uint32_t)q;
    }
}

__global__ void seg_place_kernel(int64_t total_segs, const uint32_t* __restrict__ order, const SpmmRec* __restrict__ rec_tmp,
                                 SpmmRec* __restrict__ rec, int64_t* __restrict__ seg_pos) {
    int64_t pos = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (pos >= total_segs) return;
    const uint32_t q = order[pos];
    rec[pos] = rec_tmp[q];
    seg_pos[q] = pos;
}

// Ordinary rows: one record each, in perm order, after the segment records.
__global__ void fill_records_kernel(int64_t n, int64_t n_long, int64_t total_segs, const int32_t* __restrict__ perm,
                                    const int64_t* __restrict__ rowptr, SpmmRec* __restrict__ rec) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n || i < n_long) return;
    const int64_t u = perm[i];
    SpmmRec x; x.begin = rowptr[u]; x.len = (int32_t)(rowptr[u + 1] - rowptr[u]); x.row = (int32_t)u;
    rec[total_segs + (i - n_long)] = x;
}

__global__ void validate_csr_kernel(int64_t n, int64_t nnz, const int64_t* __restrict__ rowptr,
                                    const int32_t* __restrict__ col, int32_t* flags) {
    int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= n) return;
    int64_t b = rowptr[u], e = rowptr[u + 1];
    if ((u == 0 && b != 0) || b < 0 || e < b || e > nnz) { atomicOr(flags, F_BAD_ROWPTR); return; }
    if (e - b > 0x7FFFFFFFll) { atomicOr(flags, F_BAD_ROWPTR); return; }
    for (int64_t i = b; i < e; ++i) {
        int32_t c = col[i];
        if (c < 0 || c >= n) { atomicOr(flags, F_BAD_ID); return; }
        if (i > b && col[i - 1] >= c) { atomicOr(flags, F_UNSORTED); return; }
    }
}

struct DevBuf {  // frees on scope exit
    void* p = nullptr;
    ~DevBuf() { if (p) cudaFree(p); }
    template <class T> T* as() { return reinterpret_cast<T*>(p); }
};

int bits_for(uint64_t x) { int b = 0; while (x) { ++b; x >>= 1; } return b; }

void free_schedule(SpmmSchedule& v) {
    cudaFree(v.perm); cudaFree(v.rec); cudaFree(v.seg_off); cudaFree(v.seg_pos);
    v = SpmmSchedule{};
}

void free_view(CsrView& v) {
    cudaFree(v.rowptr); cudaFree(v.col); cudaFree(v.val);
    free_schedule(v.full);
    for (int k = 0; k < v.n_chunk; ++k) free_schedule(v.chunk[k]);
    delete[] v.chunk;
    v = CsrView{};
}

// Schedule of rows [row0, row0 + n) of the CSR (rowptr, col) of a matrix with n_total columns.
mixgcn_status build_schedule(int64_t n_total, const int64_t* rowptr, const int32_t* col, int64_t row0, int64_t n,
                             SpmmSchedule& v, cudaStream_t s) {
    v = SpmmSchedule{};
    v.row0 = row0; v.n_rows = n;
    if (n <= 0) return MIXGCN_OK;
    DevBuf k0, k1, tmp, hub;
    MIXGCN_CUDA(cudaMalloc(&k0.p, n * sizeof(uint64_t)));
    MIXGCN_CUDA(cudaMalloc(&k1.p, n * sizeof(uint64_t)));
    MIXGCN_CUDA(cudaMalloc(&hub.p, 4 * sizeof(unsigned long long)));
    MIXGCN_CUDA(cudaMemsetAsync(hub.p, 0, 4 * sizeof(unsigned long long), s));
    MIXGCN_CUDA(cudaMalloc((void**)&v.perm, n * sizeof(int32_t)));
    schedule_keys_kernel<<<blocks_for(n), TPB, 0, s>>>(row0, n, rowptr, k0.as<uint64_t>());
    size_t tb = 0;
    MIXGCN_CUDA(cub::DeviceRadixSort::SortKeys(nullptr, tb, k0.as<uint64_t>(), k1.as<uint64_t>(), n, 0, 64, s));
    MIXGCN_CUDA(cudaMalloc(&tmp.p, tb ? tb : 1));
    MIXGCN_CUDA(cub::DeviceRadixSort::SortKeys(tmp.p, tb, k0.as<uint64_t>(), k1.as<uint64_t>(), n, 0, 64, s));
    schedule_finish_kernel<<<blocks_for(n), TPB, 0, s>>>(n, k1.as<uint64_t>(), v.perm, hub.as<unsigned long long>());
    unsigned long long h[4] = {0, 0, 0, 0};
    uint64_t first = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(h, hub.p, sizeof(h), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaMemcpyAsync(&first, k1.p, sizeof(first), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    v.n_long = (int64_t)h[0];
    for (int q = 0; q < 3; ++q) v.rows_above[q] = (int64_t)h[q + 1];
    v.max_deg = (int32_t)(0x7FFFFFFFull - (first >> 32));
    // long rows -> (row, column block) pairs -> segments, ordered by their first column
    const int64_t nl = v.n_long;
    DevBuf nblk, blk_off, tmp2;
    MIXGCN_CUDA(cudaMalloc(&nblk.p, (nl + 1) * sizeof(int64_t)));
    MIXGCN_CUDA(cudaMalloc(&blk_off.p, (nl + 1) * sizeof(int64_t)));
    MIXGCN_CUDA(cudaMalloc((void**)&v.seg_off, (nl + 1) * sizeof(int64_t)));
    MIXGCN_CUDA(cudaMemsetAsync(v.seg_off, 0, (nl + 1) * sizeof(int64_t), s));
    blk_count_kernel<<<blocks_for(nl + 1), TPB, 0, s>>>(nl, v.perm, rowptr, nblk.as<int64_t>());
    size_t tb2 = 0;
    MIXGCN_CUDA(cub::DeviceScan::ExclusiveSum(nullptr, tb2, nblk.as<int64_t>(), blk_off.as<int64_t>(), nl + 1, s));
    MIXGCN_CUDA(cudaMalloc(&tmp2.p, tb2 ? tb2 : 1));
    MIXGCN_CUDA(cub::DeviceScan::ExclusiveSum(tmp2.p, tb2, nblk.as<int64_t>(), blk_off.as<int64_t>(), nl + 1, s));
    int64_t total_pairs = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&total_pairs, blk_off.as<int64_t>() + nl, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    int64_t total = 0;
    DevBuf pair_lo, pair_cnt, pair_segs, pair_seg_off, tmp3, rec_tmp, keys0, keys1, ids0, ids1, tmp4;
    if (total_pairs > 0) {
        MIXGCN_CUDA(cudaMalloc(&pair_lo.p, total_pairs * sizeof(int64_t)));
        MIXGCN_CUDA(cudaMalloc(&pair_cnt.p, total_pairs * sizeof(int64_t)));
        MIXGCN_CUDA(cudaMalloc(&pair_segs.p, (total_pairs + 1) * sizeof(int64_t)));
        MIXGCN_CUDA(cudaMalloc(&pair_seg_off.p, (total_pairs + 1) * sizeof(int64_t)));
        pair_segments_kernel<<<blocks_for(total_pairs + 1), TPB, 0, s>>>(n_total, nl, total_pairs, v.perm, rowptr, col,
                                                                        blk_off.as<int64_t>(), pair_lo.as<int64_t>(),
                                                                        pair_cnt.as<int64_t>(), pair_segs.as<int64_t>());
        size_t tb3 = 0;
        MIXGCN_CUDA(cub::DeviceScan::ExclusiveSum(nullptr, tb3, pair_segs.as<int64_t>(), pair_seg_off.as<int64_t>(), total_pairs + 1, s));
        MIXGCN_CUDA(cudaMalloc(&tmp3.p, tb3 ? tb3 : 1));
        MIXGCN_CUDA(cub::DeviceScan::ExclusiveSum(tmp3.p, tb3, pair_segs.as<int64_t>(), pair_seg_off.as<int64_t>(), total_pairs + 1, s));
        MIXGCN_CUDA(cudaMemcpyAsync(&total, pair_seg_off.as<int64_t>() + total_pairs, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
        MIXGCN_CUDA(cudaStreamSynchronize(s));
    }
    if (total >= 0xFFFFFFFFll) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "graph schedule: too many long-row segments (%lld)", (long long)total);
    v.total_segs = total;
    MIXGCN_CUDA(cudaMalloc((void**)&v.rec, (size_t)(total + n - nl + 1) * sizeof(SpmmRec)));
    MIXGCN_CUDA(cudaMalloc((void**)&v.seg_pos, (size_t)(total + 1) * sizeof(int64_t)));
    if (total > 0) {
        MIXGCN_CUDA(cudaMalloc(&rec_tmp.p, total * sizeof(SpmmRec)));
        MIXGCN_CUDA(cudaMalloc(&keys0.p, total * sizeof(uint32_t)));
        MIXGCN_CUDA(cudaMalloc(&keys1.p, total * sizeof(uint32_t)));
        MIXGCN_CUDA(cudaMalloc(&ids0.p, total * sizeof(uint32_t)));
        MIXGCN_CUDA(cudaMalloc(&ids1.p, total * sizeof(uint32_t)));
        seg_fill_kernel<<<blocks_for(total_pairs), TPB, 0, s>>>(nl, total_pairs, col, blk_off.as<int64_t>(), pair_lo.as<int64_t>(),
                                                               pair_cnt.as<int64_t>(), pair_seg_off.as<int64_t>(),
                                                               rec_tmp.as<SpmmRec>(), keys0.as<uint32_t>(), ids0.as<uint32_t>(),
                                                               v.seg_off);
        size_t tb4 = 0;
        MIXGCN_CUDA(cub::DeviceRadixSort::SortPairs(nullptr, tb4, keys0.as<uint32_t>(), keys1.as<uint32_t>(), ids0.as<uint32_t>(),
                                                    ids1.as<uint32_t>(), total, 0, 32, s));
        MIXGCN_CUDA(cudaMalloc(&tmp4.p, tb4 ? tb4 : 1));
        MIXGCN_CUDA(cub::DeviceRadixSort::SortPairs(tmp4.p, tb4, keys0.as<uint32_t>(), keys1.as<uint32_t>(), ids0.as<uint32_t>(),
                                                    ids1.as<uint32_t>(), total, 0, 32, s));
        seg_place_kernel<<<blocks_for(total), TPB, 0, s>>>(total, ids1.as<uint32_t>(), rec_tmp.as<SpmmRec>(), v.rec, v.seg_pos);
    }
    fill_records_kernel<<<blocks_for(n), TPB, 0, s>>>(n, nl, total, v.perm, rowptr, v.rec);
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

// Everything after rowptr/col exist: degrees, values, symmetry, transpose, schedules.
mixgcn_status finish_graph(mixgcn_graph* g, cudaStream_t s) {
    const int64_t n = g->n, nnz = g->nnz;
    CsrView& A = g->fwd;
    DevBuf flags;
    MIXGCN_CUDA(cudaMalloc(&flags.p, sizeof(int32_t)));
    MIXGCN_CUDA(cudaMemsetAsync(flags.p, 0, sizeof(int32_t), s));
    MIXGCN_CUDA(cudaMalloc((void**)&g->deg, n * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMalloc((void**)&g->dinv, n * sizeof(float)));
    MIXGCN_CUDA(cudaMalloc((void**)&A.val, (nnz > 0 ? nnz : 1) * sizeof(float)));
    degree_kernel<<<blocks_for(n), TPB, 0, s>>>(n, A.rowptr, g->deg, g->dinv);
    values_kernel<<<blocks_for(n * 32), TPB, 0, s>>>(n, A.rowptr, A.col, g->dinv, g->norm, A.val);
    symmetry_kernel<<<blocks_for(n * 32), TPB, 0, s>>>(n, A.rowptr, A.col, flags.as<int32_t>());
    int32_t hf = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&hf, flags.p, sizeof(hf), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    g->symmetric = (hf & F_NOT_SYMMETRIC) ? 0 : 1;
    {
        DevBuf dc;
        MIXGCN_CUDA(cudaMalloc(&dc.p, sizeof(unsigned long long)));
        MIXGCN_CUDA(cudaMemsetAsync(dc.p, 0, sizeof(unsigned long long), s));
        diagonal_count_kernel<<<blocks_for(n), TPB, 0, s>>>(n, A.rowptr, A.col, dc.as<unsigned long long>());
        unsigned long long hd = 0;
        MIXGCN_CUDA(cudaMemcpyAsync(&hd, dc.p, sizeof(hd), cudaMemcpyDeviceToHost, s));
        MIXGCN_CUDA(cudaStreamSynchronize(s));
        g->has_diagonal = hd == (unsigned long long)n ? 1 : (hd == 0 ? 0 : 2);
    }
    MIXGCN_TRY(build_schedule(n, A.rowptr, A.col, 0, n, A.full, s));
    g->bwd_is_fwd = (g->symmetric && g->norm != 1) ? 1 : 0;   // row-mean values are not symmetric: A_hat^T needs its own copy
    if (g->bwd_is_fwd) {
        g->bwd = A;  // alias: the same index serves the backward aggregation
        return MIXGCN_OK;
    }
    // Transposed structure: sort (col,row) keys carrying the value.
    CsrView& T = g->bwd;
    DevBuf k0, k1, v1, tmp;
    const int64_t cap = nnz > 0 ? nnz : 1;
    MIXGCN_CUDA(cudaMalloc(&k0.p, cap * sizeof(uint64_t)));
    MIXGCN_CUDA(cudaMalloc(&k1.p, cap * sizeof(uint64_t)));
    MIXGCN_CUDA(cudaMalloc((void**)&T.val, cap * sizeof(float)));
    MIXGCN_CUDA(cudaMalloc((void**)&T.rowptr, (n + 1) * sizeof(int64_t)));
    MIXGCN_CUDA(cudaMalloc((void**)&T.col, cap * sizeof(int32_t)));
    transpose_keys_kernel<<<blocks_for(n * 32), TPB, 0, s>>>(n, A.rowptr, A.col, k0.as<uint64_t>());
    size_t tb = 0;
    const int end_bit = 32 + bits_for((uint64_t)n);
    MIXGCN_CUDA(cub::DeviceRadixSort::SortPairs(nullptr, tb, k0.as<uint64_t>(), k1.as<uint64_t>(), A.val, T.val,
                                                nnz, 0, end_bit, s));
    MIXGCN_CUDA(cudaMalloc(&tmp.p, tb ? tb : 1));
    MIXGCN_CUDA(cub::DeviceRadixSort::SortPairs(tmp.p, tb, k0.as<uint64_t>(), k1.as<uint64_t>(), A.val, T.val,
                                                nnz, 0, end_bit, s));
    rowptr_from_keys_kernel<<<blocks_for(nnz + 1), TPB, 0, s>>>(n, nnz, k1.as<uint64_t>(), T.rowptr, T.col);
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    MIXGCN_TRY(build_schedule(n, T.rowptr, T.col, 0, n, T.full, s));
    return MIXGCN_OK;
}

mixgcn_status check_common(mixgcn_ctx* ctx, int64_t n, mixgcn_graph** out) {
    if (!ctx || !out) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_create: null ctx or out");
    if (n <= 0) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_create: n must be positive (got %lld)", (long long)n);
    if (n >= 0x7FFFFFFFll) MIXGCN_FAIL(MIXGCN_EBADGRAPH, "graph_create: n = %lld does not fit int32 ids", (long long)n);
    return MIXGCN_OK;
}

}  // namespace

namespace mixgcn {

mixgcn_status build_view_schedule(int64_t n_cols, int64_t n, CsrView& v, cudaStream_t s) {
    return build_schedule(n_cols, v.rowptr, v.col, 0, n, v.full, s);
}

void release_view(CsrView& v) { free_view(v); }

mixgcn_status ensure_chunk_schedules(const mixgcn_graph* g, const CsrView& A_const, int chunks) {
    // a cache inside the graph object; a symmetric graph keeps one set (in fwd) and mirrors it into the alias
    CsrView& A = const_cast<CsrView&>(g->bwd_is_fwd ? g->fwd : A_const);
    if (chunks <= 1 || A.n_chunk == chunks) return MIXGCN_OK;
    MIXGCN_CUDA(cudaDeviceSynchronize());         // earlier launches may still read the schedules being replaced
    for (int k = 0; k < A.n_chunk; ++k) free_schedule(A.chunk[k]);
    delete[] A.chunk;
    A.chunk = nullptr; A.n_chunk = 0;
    SpmmSchedule* sc = new (std::nothrow) SpmmSchedule[chunks]();
    if (!sc) MIXGCN_FAIL(MIXGCN_ENOMEM, "chunk schedules: host allocation failed");
    cudaStream_t s = g->ctx->side_stream[0];
    for (int k = 0; k < chunks; ++k) {
        const int64_t r0 = (g->n * (int64_t)k) / chunks, r1 = (g->n * (int64_t)(k + 1)) / chunks;
        mixgcn_status st = build_schedule(g->n, A.rowptr, A.col, r0, r1 - r0, sc[k], s);
        if (st != MIXGCN_OK) {
            for (int q = 0; q <= k; ++q) free_schedule(sc[q]);
            delete[] sc;
            return st;
        }
    }
    A.chunk = sc; A.n_chunk = chunks;
    if (g->bwd_is_fwd) const_cast<mixgcn_graph*>(g)->bwd = g->fwd;   // keep the alias in step
    return MIXGCN_OK;
}

}  // namespace mixgcn

extern "C" mixgcn_status mixgcn_graph_destroy(mixgcn_graph* g) {
    if (!g) return MIXGCN_OK;
    cudaSetDevice(g->device);
    if (!g->bwd_is_fwd) free_view(g->bwd);
    free_view(g->fwd);
    cudaFree(g->deg);
    cudaFree(g->dinv);
    delete g;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_graph_create(mixgcn_ctx* ctx, int64_t n, int64_t m, const int32_t* src,
                                             const int32_t* dst, uint32_t flags, mixgcn_graph** out) {
    MIXGCN_TRY(check_common(ctx, n, out));
    if (m < 0 || (m > 0 && (!src || !dst))) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_create: bad edge list (m=%lld)", (long long)m);
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t s = ctx->side_stream[0];
    if ((flags & MIXGCN_GRAPH_NORM_ROW) && (flags & MIXGCN_GRAPH_NORM_NONE)) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_create: NORM_ROW and NORM_NONE exclude each other");
    const int sym = (flags & MIXGCN_GRAPH_SYMMETRISE) != 0, self = (flags & MIXGCN_GRAPH_ADD_SELF_LOOPS) != 0;
    const int64_t total = m * (sym ? 2 : 1) + (self ? n : 0);

    mixgcn_graph* g = new (std::nothrow) mixgcn_graph();
    if (g) g->uid = next_graph_uid();
    if (!g) MIXGCN_FAIL(MIXGCN_ENOMEM, "graph_create: host allocation failed");
    g->ctx = ctx; g->device = ctx->device; g->n = n; g->nnz = 0; g->symmetric = 1; g->bwd_is_fwd = 1;
    g->norm = (flags & MIXGCN_GRAPH_NORM_ROW) ? 1 : ((flags & MIXGCN_GRAPH_NORM_NONE) ? 2 : 0);
    struct Guard { mixgcn_graph* g; bool keep = false; ~Guard() { if (!keep) { g->bwd_is_fwd = g->bwd.rowptr == g->fwd.rowptr; mixgcn_graph_destroy(g); } } } guard{g};
    LaunchScope scope(ctx, PH_GRAPH, s, 12);

    DevBuf dsrc, ddst, k0, k1, tmp, fl, cnt;
    const int32_t *ps = src, *pd = dst;
    if (!(flags & MIXGCN_GRAPH_EDGES_ON_DEVICE) && m > 0) {
        MIXGCN_CUDA(cudaMalloc(&dsrc.p, m * sizeof(int32_t)));
        MIXGCN_CUDA(cudaMalloc(&ddst.p, m * sizeof(int32_t)));
        MIXGCN_CUDA(cudaMemcpyAsync(dsrc.p, src, m * sizeof(int32_t), cudaMemcpyHostToDevice, s));
        MIXGCN_CUDA(cudaMemcpyAsync(ddst.p, dst, m * sizeof(int32_t), cudaMemcpyHostToDevice, s));
        ps = dsrc.as<int32_t>(); pd = ddst.as<int32_t>();
    }
    const int64_t cap = total > 0 ? total : 1;
    MIXGCN_CUDA(cudaMalloc(&k0.p, cap * sizeof(uint64_t)));
    MIXGCN_CUDA(cudaMalloc(&k1.p, cap * sizeof(uint64_t)));
    MIXGCN_CUDA(cudaMalloc(&fl.p, sizeof(int32_t)));
    MIXGCN_CUDA(cudaMalloc(&cnt.p, sizeof(int64_t)));
    MIXGCN_CUDA(cudaMemsetAsync(fl.p, 0, sizeof(int32_t), s));
    const uint64_t sentinel = (uint64_t)n << 32;  // sorts after every valid key
    {
        int64_t work = m > n ? m : n;
        make_keys_kernel<<<blocks_for(work > 0 ? work : 1), TPB, 0, s>>>(n, m, ps, pd, sym, self, sentinel,
                                                                        k0.as<uint64_t>(), fl.as<int32_t>());
    }
    const int end_bit = 32 + bits_for((uint64_t)n);
    size_t tb_sort = 0, tb_uniq = 0;
    MIXGCN_CUDA(cub::DeviceRadixSort::SortKeys(nullptr, tb_sort, k0.as<uint64_t>(), k1.as<uint64_t>(), total, 0, end_bit, s));
    MIXGCN_CUDA(cub::DeviceSelect::Unique(nullptr, tb_uniq, k1.as<uint64_t>(), k0.as<uint64_t>(), cnt.as<int64_t>(), total, s));
    size_t tb = tb_sort > tb_uniq ? tb_sort : tb_uniq;
    MIXGCN_CUDA(cudaMalloc(&tmp.p, tb ? tb : 1));
    MIXGCN_CUDA(cub::DeviceRadixSort::SortKeys(tmp.p, tb, k0.as<uint64_t>(), k1.as<uint64_t>(), total, 0, end_bit, s));
    // edge arrays are no longer needed
    MIXGCN_CUDA(cub::DeviceSelect::Unique(tmp.p, tb, k1.as<uint64_t>(), k0.as<uint64_t>(), cnt.as<int64_t>(), total, s));
    int64_t n_unique = 0;
    int32_t hf = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&n_unique, cnt.p, sizeof(int64_t), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaMemcpyAsync(&hf, fl.p, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    if (hf & F_BAD_ID) MIXGCN_FAIL(MIXGCN_EBADGRAPH, "graph_create: a node id lies outside [0, %lld)", (long long)n);
    if (total == 0) n_unique = 0;
    if (n_unique > 0) {
        uint64_t last = 0;
        MIXGCN_CUDA(cudaMemcpy(&last, k0.as<uint64_t>() + (n_unique - 1), sizeof(last), cudaMemcpyDeviceToHost));
        if (last == sentinel) --n_unique;
    }
    g->nnz = n_unique;
    cudaFree(k1.p); k1.p = nullptr;
    cudaFree(tmp.p); tmp.p = nullptr;
    MIXGCN_CUDA(cudaMalloc((void**)&g->fwd.rowptr, (n + 1) * sizeof(int64_t)));
    MIXGCN_CUDA(cudaMalloc((void**)&g->fwd.col, (n_unique > 0 ? n_unique : 1) * sizeof(int32_t)));
    rowptr_from_keys_kernel<<<blocks_for(n_unique + 1), TPB, 0, s>>>(n, n_unique, k0.as<uint64_t>(), g->fwd.rowptr, g->fwd.col);
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    cudaFree(k0.p); k0.p = nullptr;
    MIXGCN_TRY(finish_graph(g, s));
    MIXGCN_CUDA(cudaGetLastError());
    guard.keep = true;
    *out = g;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_graph_create_from_csr(mixgcn_ctx* ctx, int64_t n, const int64_t* rowptr,
                                                      const int32_t* col, uint32_t flags, mixgcn_graph** out) {
    MIXGCN_TRY(check_common(ctx, n, out));
    if (!rowptr) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_create_from_csr: null rowptr");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t s = ctx->side_stream[0];
    const bool on_dev = (flags & MIXGCN_GRAPH_EDGES_ON_DEVICE) != 0;
    const cudaMemcpyKind kind = on_dev ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    int64_t nnz = 0;
    MIXGCN_CUDA(cudaMemcpy(&nnz, rowptr + n, sizeof(int64_t), on_dev ? cudaMemcpyDeviceToHost : cudaMemcpyHostToHost));
    if (nnz < 0) MIXGCN_FAIL(MIXGCN_EBADGRAPH, "graph_create_from_csr: rowptr[n] is negative");
    if (nnz > 0 && !col) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_create_from_csr: null col");

    mixgcn_graph* g = new (std::nothrow) mixgcn_graph();
    if (g) g->uid = next_graph_uid();
    if (!g) MIXGCN_FAIL(MIXGCN_ENOMEM, "graph_create_from_csr: host allocation failed");
    g->ctx = ctx; g->device = ctx->device; g->n = n; g->nnz = nnz; g->symmetric = 1; g->bwd_is_fwd = 1;
    g->norm = (flags & MIXGCN_GRAPH_NORM_ROW) ? 1 : ((flags & MIXGCN_GRAPH_NORM_NONE) ? 2 : 0);
    struct Guard { mixgcn_graph* g; bool keep = false; ~Guard() { if (!keep) { g->bwd_is_fwd = g->bwd.rowptr == g->fwd.rowptr; mixgcn_graph_destroy(g); } } } guard{g};
    LaunchScope scope(ctx, PH_GRAPH, s, 8);
    DevBuf fl;
    MIXGCN_CUDA(cudaMalloc(&fl.p, sizeof(int32_t)));
    MIXGCN_CUDA(cudaMemsetAsync(fl.p, 0, sizeof(int32_t), s));
    MIXGCN_CUDA(cudaMalloc((void**)&g->fwd.rowptr, (n + 1) * sizeof(int64_t)));
    MIXGCN_CUDA(cudaMalloc((void**)&g->fwd.col, (nnz > 0 ? nnz : 1) * sizeof(int32_t)));
    MIXGCN_CUDA(cudaMemcpyAsync(g->fwd.rowptr, rowptr, (n + 1) * sizeof(int64_t), kind, s));
    if (nnz > 0) MIXGCN_CUDA(cudaMemcpyAsync(g->fwd.col, col, nnz * sizeof(int32_t), kind, s));
    // rowptr must be validated before col is indexed with it: first monotonicity on the host side
    // of the device array (cheap kernel), then the per-row column checks.
    validate_csr_kernel<<<blocks_for(n), TPB, 0, s>>>(n, nnz, g->fwd.rowptr, g->fwd.col, fl.as<int32_t>());
    int32_t hf = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&hf, fl.p, sizeof(hf), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    if (hf & F_BAD_ROWPTR) MIXGCN_FAIL(MIXGCN_EBADGRAPH, "graph_create_from_csr: rowptr is not monotone from 0");
    if (hf & F_BAD_ID) MIXGCN_FAIL(MIXGCN_EBADGRAPH, "graph_create_from_csr: a column id lies outside [0, %lld)", (long long)n);
    if (hf & F_UNSORTED) MIXGCN_FAIL(MIXGCN_EBADGRAPH, "graph_create_from_csr: columns are not strictly ascending in a row");
    MIXGCN_TRY(finish_graph(g, s));
    MIXGCN_CUDA(cudaGetLastError());
    guard.keep = true;
    *out = g;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_graph_info(const mixgcn_graph* g, int64_t* n, int64_t* nnz, int32_t* max_deg,
                                           int32_t* symmetric) {
    if (!g) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_info: null graph");
    if (n) *n = g->n;
    if (nnz) *nnz = g->nnz;
    if (max_deg) *max_deg = g->fwd.full.max_deg;
    if (symmetric) *symmetric = g->symmetric;
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_graph_export(const mixgcn_graph* g, int transposed, int64_t* rowptr, int32_t* col,
                                             float* val, int32_t* deg, float* dinv) {
    if (!g) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_export: null graph");
    MIXGCN_CUDA(cudaSetDevice(g->ctx->device));
    MIXGCN_CUDA(cudaDeviceSynchronize());
    const CsrView& v = transposed ? g->bwd : g->fwd;
    if (rowptr) MIXGCN_CUDA(cudaMemcpy(rowptr, v.rowptr, (g->n + 1) * sizeof(int64_t), cudaMemcpyDeviceToHost));
    if (col && g->nnz) MIXGCN_CUDA(cudaMemcpy(col, v.col, g->nnz * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (val && g->nnz) MIXGCN_CUDA(cudaMemcpy(val, v.val, g->nnz * sizeof(float), cudaMemcpyDeviceToHost));
    if (deg) MIXGCN_CUDA(cudaMemcpy(deg, g->deg, g->n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (dinv) MIXGCN_CUDA(cudaMemcpy(dinv, g->dinv, g->n * sizeof(float), cudaMemcpyDeviceToHost));
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_graph_export_schedule(const mixgcn_graph* g, int transposed, int32_t* perm) {
    if (!g || !perm) MIXGCN_FAIL(MIXGCN_EINVAL, "graph_export_schedule: null argument");
    MIXGCN_CUDA(cudaSetDevice(g->ctx->device));
    MIXGCN_CUDA(cudaDeviceSynchronize());
    const CsrView& v = transposed ? g->bwd : g->fwd;
    MIXGCN_CUDA(cudaMemcpy(perm, v.full.perm, g->n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    return MIXGCN_OK;
}
