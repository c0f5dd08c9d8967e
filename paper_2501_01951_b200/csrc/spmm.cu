// Neighbour aggregation Z = A_hat Y (Algorithm 2, aggregation line): deterministic, atomic-free,
// row-wise CSR SpMM.
//
//  - A group of LPR lanes owns one output row; each lane owns VPL float4 column groups, so a
//    gathered row of Y is read with coalesced 16-byte loads.
//  - (col,val) of the row are fetched LPR at a time (one coalesced load per group) and handed
//    round with warp shuffles; four gathered rows are in flight per lane before the FMAs.
//  - Rows are taken in descending entry-count order (the graph's schedule), so the hardware
//    block scheduler sees longest-first work; rows above HUB_THRESHOLD get a whole CTA whose
//    warps split the row into contiguous segments and combine in fixed warp order.
//  - Sums run over ascending column id inside a segment: the result is bit-reproducible.
//  - The epilogue (bias, ReLU, dropout mask, gate by another tensor's sign) is applied in
//    registers before the single write of Z.
#include "internal.cuh"

using namespace mixgcn;

namespace {

struct SpmmParams {
    const int64_t* rowptr;
    const int32_t* col;
    const float* val;
    const int32_t* perm;   // nullable: natural order
    int64_t idx_begin, idx_end;
    int32_t w;             // columns handled by this launch (slice width)
    int32_t j0;            // first column of the slice (multiple of 4)
    int32_t w_total;       // full width (for the dense drop-mask index)
    const float* Y; int64_t ldy;
    float* Z; int64_t ldz;
    // epilogue
    const float* bias; int relu;
    const uint8_t* drop; float keep_scale;
    const float* gate; int64_t ld_gate; float gate_scale;
};

__device__ __forceinline__ float epilogue1(const SpmmParams& p, float y, int64_t u, int j) {
    if (p.bias) y += p.bias[j];
    if (p.relu) y = fmaxf(y, 0.0f);
    if (p.drop) y = p.drop[u * p.w_total + j] ? y * p.keep_scale : 0.0f;
    if (p.gate) y = p.gate[u * p.ld_gate + j] > 0.0f ? y * p.gate_scale : 0.0f;
    return y;
}

__device__ __forceinline__ void store_row(const SpmmParams& p, int64_t u, int c4, float4 a) {
    const int j = p.j0 + c4 * 4;           // global column of a.x
    const int jend = p.j0 + p.w;           // one past the last valid column of the slice
    float r[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) r[t] = (j + t < jend) ? epilogue1(p, r[t], u, j + t) : 0.0f;
    *reinterpret_cast<float4*>(p.Z + u * p.ldz + j) = make_float4(r[0], r[1], r[2], r[3]);
}

__device__ __forceinline__ void fma4(float4& acc, float a, const float4& y) {
    acc.x = fmaf(a, y.x, acc.x); acc.y = fmaf(a, y.y, acc.y);
    acc.z = fmaf(a, y.z, acc.z); acc.w = fmaf(a, y.w, acc.w);
}

// Accumulate entries [b, e) of one row into acc[] for the lane's column groups.
template <int LPR, int VPL>
__device__ __forceinline__ void row_segment(const SpmmParams& p, int64_t b, int64_t e, int lig, unsigned mask,
                                            int w4, float4 (&acc)[VPL]) {
    const float* Yb = p.Y + p.j0;
    for (int64_t i0 = b; i0 < e; i0 += LPR) {
        int c = 0; float a = 0.0f;
        if (i0 + lig < e) { c = __ldg(p.col + i0 + lig); a = __ldg(p.val + i0 + lig); }
        const int cnt = (int)((e - i0) < LPR ? (e - i0) : LPR);
        int k = 0;
        for (; k + 4 <= cnt; k += 4) {
            int ck[4]; float ak[4]; float4 y[4][VPL];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                ck[t] = __shfl_sync(mask, c, k + t, LPR);
                ak[t] = __shfl_sync(mask, a, k + t, LPR);
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const float4* yr = reinterpret_cast<const float4*>(Yb + (int64_t)ck[t] * p.ldy);
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    const int c4 = lig + v * LPR;
                    y[t][v] = (c4 < w4) ? __ldg(yr + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int v = 0; v < VPL; ++v) fma4(acc[v], ak[t], y[t][v]);
        }
        for (; k < cnt; ++k) {
            const int c1 = __shfl_sync(mask, c, k, LPR);
            const float a1 = __shfl_sync(mask, a, k, LPR);
            const float4* yr = reinterpret_cast<const float4*>(Yb + (int64_t)c1 * p.ldy);
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                const int c4 = lig + v * LPR;
                if (c4 < w4) fma4(acc[v], a1, __ldg(yr + c4));
            }
        }
    }
}

template <int LPR, int VPL>
__global__ void __launch_bounds__(256) spmm_group_kernel(const SpmmParams p) {
    const int lig = threadIdx.x % LPR;
    const int64_t idx = p.idx_begin + ((int64_t)blockIdx.x * 256 + threadIdx.x) / LPR;
    if (idx >= p.idx_end) return;  // the whole group leaves together
    const unsigned mask = LPR == 32 ? 0xFFFFFFFFu : (((1u << LPR) - 1u) << ((threadIdx.x & 31) & ~(LPR - 1)));
    const int64_t u = p.perm ? (int64_t)__ldg(p.perm + idx) : idx;
    const int w4 = (p.w + 3) >> 2;
    float4 acc[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    row_segment<LPR, VPL>(p, __ldg(p.rowptr + u), __ldg(p.rowptr + u + 1), lig, mask, w4, acc);
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int c4 = lig + v * LPR;
        if (c4 < w4) store_row(p, u, c4, acc[v]);
    }
}

// One CTA (8 warps) per long row.
template <int VPL>
__global__ void __launch_bounds__(256) spmm_hub_kernel(const SpmmParams p) {
    extern __shared__ float4 part[];  // [8][w4]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t idx = p.idx_begin + blockIdx.x;
    const int64_t u = p.perm ? (int64_t)__ldg(p.perm + idx) : idx;
    const int w4 = (p.w + 3) >> 2;
    const int64_t b = __ldg(p.rowptr + u), e = __ldg(p.rowptr + u + 1);
    // contiguous segments, multiples of 32 entries so that every segment starts group-aligned
    int64_t per = ((e - b + 8 * 32 - 1) / (8 * 32)) * 32;
    int64_t sb = b + warp * per, se = sb + per;
    if (sb > e) sb = e;
    if (se > e) se = e;
    float4 acc[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    row_segment<32, VPL>(p, sb, se, lane, 0xFFFFFFFFu, w4, acc);
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int c4 = lane + v * 32;
        if (c4 < w4) part[warp * w4 + c4] = acc[v];
    }
    __syncthreads();
    for (int c4 = threadIdx.x; c4 < w4; c4 += 256) {
        float4 s = part[c4];
        for (int wq = 1; wq < 8; ++wq) {  // fixed order
            float4 t = part[wq * w4 + c4];
            s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
        }
        store_row(p, u, c4, s);
    }
}

template <int LPR, int VPL>
void launch_group(const SpmmParams& p, cudaStream_t s) {
    const int64_t rows = p.idx_end - p.idx_begin;
    if (rows <= 0) return;
    const int rows_per_block = 256 / LPR;
    const int64_t blocks = (rows + rows_per_block - 1) / rows_per_block;
    spmm_group_kernel<LPR, VPL><<<(unsigned)blocks, 256, 0, s>>>(p);
}

template <int VPL>
void launch_hub(const SpmmParams& p, cudaStream_t s) {
    const int64_t rows = p.idx_end - p.idx_begin;
    if (rows <= 0) return;
    const int w4 = (p.w + 3) >> 2;
    spmm_hub_kernel<VPL><<<(unsigned)rows, 256, 8 * w4 * sizeof(float4), s>>>(p);
}

void dispatch_group(const SpmmParams& p, cudaStream_t s) {
    const int w4 = (p.w + 3) >> 2;
    if (w4 <= 1) return launch_group<1, 1>(p, s);
    if (w4 <= 2) return launch_group<2, 1>(p, s);
    if (w4 <= 4) return launch_group<4, 1>(p, s);
    if (w4 <= 8) return launch_group<8, 1>(p, s);
    if (w4 <= 16) return launch_group<16, 1>(p, s);
    switch ((w4 + 31) / 32) {
        case 1: return launch_group<32, 1>(p, s);
        case 2: return launch_group<32, 2>(p, s);
        case 3: return launch_group<32, 3>(p, s);
        case 4: return launch_group<32, 4>(p, s);
        case 5: return launch_group<32, 5>(p, s);
        case 6: return launch_group<32, 6>(p, s);
        case 7: return launch_group<32, 7>(p, s);
        default: return launch_group<32, 8>(p, s);
    }
}

void dispatch_hub(const SpmmParams& p, cudaStream_t s) {
    const int w4 = (p.w + 3) >> 2;
    switch ((w4 + 31) / 32) {
        case 1: return launch_hub<1>(p, s);
        case 2: return launch_hub<2>(p, s);
        case 3: return launch_hub<3>(p, s);
        case 4: return launch_hub<4>(p, s);
        case 5: return launch_hub<5>(p, s);
        case 6: return launch_hub<6>(p, s);
        case 7: return launch_hub<7>(p, s);
        default: return launch_hub<8>(p, s);
    }
}

constexpr int MAX_SLICE = 1024;  // columns per launch: 8 float4 per lane

}  // namespace

namespace mixgcn {

// Rows [row_begin, row_end): when the range is the whole matrix the degree-sorted schedule is
// used (hub rows first); a partial range (pipeline chunk) runs in natural row order.
mixgcn_status launch_spmm(mixgcn_ctx* ctx, const mixgcn_graph* g, const CsrView& A, int64_t row_begin,
                          int64_t row_end, int32_t w, const float* Y, int64_t ldy, float* Z, int64_t ldz,
                          const mixgcn_epilogue* epi, cudaStream_t s) {
    if (row_end <= row_begin || w <= 0) return MIXGCN_OK;
    const bool whole = row_begin == 0 && row_end == g->n;
    SpmmParams p{};
    p.rowptr = A.rowptr; p.col = A.col; p.val = A.val;
    p.Y = Y; p.ldy = ldy; p.Z = Z; p.ldz = ldz; p.w_total = w;
    if (epi) {
        p.bias = epi->bias; p.relu = epi->relu; p.drop = epi->drop_mask; p.keep_scale = epi->keep_scale;
        p.gate = epi->gate; p.ld_gate = epi->ld_gate; p.gate_scale = epi->gate_scale;
    }
    for (int j0 = 0; j0 < w; j0 += MAX_SLICE) {
        p.j0 = j0;
        p.w = (w - j0) < MAX_SLICE ? (w - j0) : MAX_SLICE;
        if (whole) {
            p.perm = A.perm;
            if (A.n_hub > 0) {
                LaunchScope scope(ctx, PH_SPMM, s);
                p.idx_begin = 0; p.idx_end = A.n_hub;
                dispatch_hub(p, s);
            }
            if (A.n_hub < g->n) {
                LaunchScope scope(ctx, PH_SPMM, s);
                p.idx_begin = A.n_hub; p.idx_end = g->n;
                dispatch_group(p, s);
            }
        } else {
            LaunchScope scope(ctx, PH_SPMM, s);
            p.perm = nullptr; p.idx_begin = row_begin; p.idx_end = row_end;
            dispatch_group(p, s);
        }
    }
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

}  // namespace mixgcn

extern "C" mixgcn_status mixgcn_spmm(mixgcn_ctx* ctx, const mixgcn_graph* g, int transposed, int32_t w,
                                     const float* Y, int64_t ldy, float* Z, int64_t ldz,
                                     const mixgcn_epilogue* epi, void* stream) {
    if (!ctx || !g || !Y || !Z) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: null argument");
    if (w <= 0) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: w must be positive (got %d)", w);
    if (ldy < w || ldz < w || (ldy & 3) || (ldz & 3))
        MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: leading dimensions must be multiples of 4 and >= w (ldy=%lld ldz=%lld w=%d)",
                    (long long)ldy, (long long)ldz, w);
    if (!aligned16(Y) || !aligned16(Z)) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: Y and Z must be 16-byte aligned");
    if (Y == Z) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: Y and Z must not overlap");
    if (epi && epi->gate && epi->ld_gate < w) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: gate leading dimension < w");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    return launch_spmm(ctx, g, transposed ? g->bwd : g->fwd, 0, g->n, w, Y, ldy, Z, ldz, epi, (cudaStream_t)stream);
}
