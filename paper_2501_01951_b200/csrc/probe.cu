// Measurement helper, not a step of the method: the rate at which this GPU serves gathers of whole
// feature rows from a table, without any arithmetic or output to speak of.  With a table that fits the
// L2 it gives the denominator for aggregations whose input is L2-resident (their gathers are bound by
// the L2-to-SM path, not by HBM); with a table much larger than the L2, the rate of uncached row gathers.
#include "internal.cuh"

using namespace mixgcn;

namespace {

__device__ __forceinline__ uint64_t probe_mix(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

// Every warp reads `per_warp` pseudo-random rows of 128 floats (lane = float4 column, one 512-byte
// request per row, eight rows in flight) and adds them up; the sums leave the kernel only through a
// store that the data never triggers, so the loads cannot be removed.
__global__ void __launch_bounds__(256) probe_gather_kernel(const float* __restrict__ table, int64_t rows, int64_t per_warp,
                                                           uint64_t seed, float* __restrict__ sink) {
    const int lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t i = 0; i < per_warp; i += 32) {
        // lane l draws the row of gather i + l (uniform in [0, rows) by a multiply-high: no division in the loop)
        const uint64_t mine = __umul64hi(probe_mix(seed ^ (warp * 0x100000001B3ull + (uint64_t)(i + lane))), (uint64_t)rows);
        for (int t0 = 0; t0 < 32 && i + t0 < per_warp; t0 += 8) {
            float4 y[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const uint64_t r = __shfl_sync(0xFFFFFFFFu, mine, t0 + t);
                y[t] = __ldg(reinterpret_cast<const float4*>(table + r * 128) + lane);
            }
#pragma unroll
            for (int t = 0; t < 8; ++t) { acc.x += y[t].x; acc.y += y[t].y; acc.z += y[t].z; acc.w += y[t].w; }
        }
    }
    if (acc.x + acc.y + acc.z + acc.w == 1.2345678e38f) sink[0] = acc.x;
}

}  // namespace

extern "C" mixgcn_status mixgcn_probe_gather(mixgcn_ctx* ctx, const float* table, int64_t rows, int64_t gathers_per_warp,
                                             uint64_t seed, float* sink, int64_t* total_gathers, void* stream) {
    if (!ctx || !table || !sink) MIXGCN_FAIL(MIXGCN_EINVAL, "probe_gather: null argument");
    if (rows <= 0 || gathers_per_warp <= 0 || (gathers_per_warp & 7)) MIXGCN_FAIL(MIXGCN_EINVAL, "probe_gather: rows > 0 and gathers_per_warp a positive multiple of 8");
    if (!aligned16(table)) MIXGCN_FAIL(MIXGCN_EINVAL, "probe_gather: the table must be 16-byte aligned");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    const int blocks = ctx->sm_count * 8;
    if (total_gathers) *total_gathers = (int64_t)blocks * 8 * gathers_per_warp;
    LaunchScope scope(ctx, PH_ELEM, (cudaStream_t)stream);
    probe_gather_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(table, rows, gathers_per_warp, seed, sink);
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}
