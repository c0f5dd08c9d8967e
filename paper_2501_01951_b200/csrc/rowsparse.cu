// Helpers of the row-sparse backward pass: when the gradient that enters a layer has only a few
// non-zero rows (the masked loss gives non-zero rows on train nodes only), the dense products
// run on the compacted rows and the aggregation skips the zero rows.
#include <cub/cub.cuh>
#include <thrust/iterator/counting_iterator.h>

#include "internal.cuh"

using namespace mixgcn;

namespace {

__global__ void pos_scatter_kernel(int64_t count, const int32_t* __restrict__ idx, int32_t* __restrict__ pos) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) pos[idx[i]] = (int32_t)i;
}

// The selection filled idx[0, *selected).  If the caller's count differs, report it; slots
// [*selected, expected) were not written by the selection and still hold old workspace contents, so
// they are pointed at row 0 (a valid row) before the gather / scatter / position kernels read them.
__global__ void check_count_kernel(const int64_t* selected, int64_t expected, int32_t* idx, int32_t* status) {
    const int64_t sel = *selected;
    if (threadIdx.x == 0 && blockIdx.x == 0 && sel != expected) atomicMax(status, DEV_BAD_ROW_COUNT);
    for (int64_t i = sel + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < expected; i += (int64_t)gridDim.x * blockDim.x)
        idx[i] = 0;
}

// dst[i, :] = src[idx[i], :], float4 wide (ld multiples of 4, 16-byte aligned), d4 = ceil(d/4) groups per row
__global__ void gather_rows_kernel(int64_t count, int d4, const int32_t* __restrict__ idx, const float* __restrict__ src,
                                   int64_t ld_src, float* __restrict__ dst, int64_t ld_dst, int64_t n_rows, int32_t* status) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count * d4) return;
    const int64_t i = t / d4; const int c = (int)(t % d4);
    const int64_t r = idx[i];
    if (!index_ok(r, n_rows, status, SITE_ROW_LIST)) return;
    reinterpret_cast<float4*>(dst + i * ld_dst)[c] = __ldg(reinterpret_cast<const float4*>(src + r * ld_src) + c);
}

// number of non-zero bytes (integer sum: order-free)
__global__ void count_rows_kernel(int64_t n, const uint8_t* __restrict__ mask, unsigned long long* count) {
    unsigned int c = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        c += mask[i] ? 1u : 0u;
    for (int o = 16; o > 0; o >>= 1) c += __shfl_down_sync(0xFFFFFFFFu, c, o);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(count, (unsigned long long)c);
}

// dst[idx[i], :] = src[i, :]
__global__ void scatter_rows_kernel(int64_t count, int d4, const int32_t* __restrict__ idx, const float* __restrict__ src,
                                    int64_t ld_src, float* __restrict__ dst, int64_t ld_dst, int64_t n_rows, int32_t* status) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count * d4) return;
    const int64_t i = t / d4; const int c = (int)(t % d4);
    const int64_t r = idx[i];
    if (!index_ok(r, n_rows, status, SITE_ROW_LIST)) return;
    reinterpret_cast<float4*>(dst + r * ld_dst)[c] = __ldg(reinterpret_cast<const float4*>(src + i * ld_src) + c);
}

}  // namespace

namespace mixgcn {

mixgcn_status ensure_workspace_rows(mixgcn_ctx* ctx, int64_t bytes) {
    if (bytes <= ctx->workspace_rows_bytes) return MIXGCN_OK;
    int64_t want = bytes + (bytes >> 3);
    want = (want + 255) & ~(int64_t)255;
    void* p = nullptr;
    MIXGCN_CUDA(cudaDeviceSynchronize());
    if (ctx->workspace_rows) cudaFree(ctx->workspace_rows);
    ctx->workspace_rows = nullptr; ctx->workspace_rows_bytes = 0;
    if (cudaMalloc(&p, (size_t)want) != cudaSuccess) {
        cudaGetLastError();
        MIXGCN_FAIL(MIXGCN_ENOMEM, "row-sparse workspace of %lld bytes could not be allocated", (long long)want);
    }
    ctx->workspace_rows = p; ctx->workspace_rows_bytes = want;
    return MIXGCN_OK;
}

// Carves the row-sparse workspace and fills the row list and the position map of `mask`.
// idx has capacity n >= count (memory-safe whatever the mask holds); if the number of set rows differs
// from `count` the device status word receives DEV_BAD_ROW_COUNT and the unfilled slots name row 0.
mixgcn_status build_row_set(mixgcn_ctx* ctx, int64_t n, const uint8_t* mask, int64_t count, int64_t ld_a, int64_t ld_b,
                            RowSet* rs, cudaStream_t s) {
    if (count < 0 || count > n) MIXGCN_FAIL(MIXGCN_EINVAL, "row set: the row count must lie in [0, n] (count %lld, n %lld)", (long long)count, (long long)n);
    size_t tb = 0;
    thrust::counting_iterator<int32_t> ids(0);
    MIXGCN_CUDA(cub::DeviceSelect::Flagged(nullptr, tb, ids, mask, (int32_t*)nullptr, (int64_t*)nullptr, n, s));
    auto up = [](int64_t x) { return (x + 255) & ~(int64_t)255; };
    const int64_t o_pos = 0, o_idx = o_pos + up(n * 4), o_sel = o_idx + up(n * 4), o_tmp = o_sel + 256,
                  o_a = o_tmp + up((int64_t)tb), o_b = o_a + up(count * ld_a * 4), total = o_b + up(count * ld_b * 4);
    MIXGCN_TRY(ensure_workspace_rows(ctx, total));
    char* base = reinterpret_cast<char*>(ctx->workspace_rows);
    rs->pos = reinterpret_cast<int32_t*>(base + o_pos);
    rs->idx = reinterpret_cast<int32_t*>(base + o_idx);
    int64_t* selected = reinterpret_cast<int64_t*>(base + o_sel);
    rs->a = reinterpret_cast<float*>(base + o_a);
    rs->b = reinterpret_cast<float*>(base + o_b);
    rs->count = count;
    LaunchScope scope(ctx, PH_ELEM, s, 4);
    MIXGCN_CUDA(cub::DeviceSelect::Flagged(base + o_tmp, tb, ids, mask, rs->idx, selected, n, s));
    check_count_kernel<<<64, 256, 0, s>>>(selected, count, rs->idx, ctx->d_status);
    MIXGCN_CUDA(cudaMemsetAsync(rs->pos, 0xFF, (size_t)n * 4, s));       // -1 everywhere
    if (count > 0) pos_scatter_kernel<<<(unsigned)((count + 255) / 256), 256, 0, s>>>(count, rs->idx, rs->pos);
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

mixgcn_status launch_gather_rows(mixgcn_ctx* ctx, int64_t n_rows, int64_t count, int32_t d, const int32_t* idx, const float* src,
                                 int64_t ld_src, float* dst, int64_t ld_dst, cudaStream_t s) {
    if (count <= 0) return MIXGCN_OK;
    const int d4 = (d + 3) / 4;
    LaunchScope scope(ctx, PH_ELEM, s);
    gather_rows_kernel<<<(unsigned)((count * d4 + 255) / 256), 256, 0, s>>>(count, d4, idx, src, ld_src, dst, ld_dst, n_rows, ctx->d_status);
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

mixgcn_status launch_scatter_rows(mixgcn_ctx* ctx, int64_t n_rows, int64_t count, int32_t d, const int32_t* idx, const float* src,
                                  int64_t ld_src, float* dst, int64_t ld_dst, cudaStream_t s) {
    if (count <= 0) return MIXGCN_OK;
    const int d4 = (d + 3) / 4;
    LaunchScope scope(ctx, PH_ELEM, s);
    scatter_rows_kernel<<<(unsigned)((count * d4 + 255) / 256), 256, 0, s>>>(count, d4, idx, src, ld_src, dst, ld_dst, n_rows, ctx->d_status);
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

}  // namespace mixgcn

extern "C" mixgcn_status mixgcn_count_rows(mixgcn_ctx* ctx, int64_t n, const uint8_t* row_mask, int64_t* count,
                                           void* stream) {
    if (!ctx || !row_mask || !count || n < 0) MIXGCN_FAIL(MIXGCN_EINVAL, "count_rows: bad argument");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    MIXGCN_TRY(ensure_workspace_rows(ctx, 256));
    unsigned long long* d = reinterpret_cast<unsigned long long*>(ctx->workspace_rows);
    MIXGCN_CUDA(cudaMemsetAsync(d, 0, sizeof(unsigned long long), s));
    if (n > 0) {
        LaunchScope scope(ctx, PH_ELEM, s);
        int64_t blocks = (n + 255) / 256;
        const int64_t cap = (int64_t)ctx->sm_count * 16;
        if (blocks > cap) blocks = cap;
        count_rows_kernel<<<(unsigned)blocks, 256, 0, s>>>(n, row_mask, d);
    }
    unsigned long long h = 0;
    MIXGCN_CUDA(cudaMemcpyAsync(&h, d, sizeof(h), cudaMemcpyDeviceToHost, s));
    MIXGCN_CUDA(cudaStreamSynchronize(s));
    *count = (int64_t)h;
    return MIXGCN_OK;
}
