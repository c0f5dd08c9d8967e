// Dense update products in plain fp32 on the CUDA cores (the strict-precision mode of the
// update line of Algorithm 2 and of its two backward products), plus the small streaming
// kernels around them (column sums for the bias gradient, the ReLU/dropout gate on a gradient).
//
// C = op(A) op(B): 128 x BN output tile per CTA, 16-deep k-steps staged through shared memory
// with the next step's global loads in flight during the FMAs; each thread owns an 8 x TN
// micro-tile.  Long reductions (K = number of nodes in the weight-gradient product) are split
// over CTAs into partial tiles that a second kernel adds in a fixed order in fp64, and inside a
// CTA the fp32 accumulator is flushed into a second-level sum every 1024 terms, so rounding
// error does not grow with the node count.
#include "internal.cuh"

using namespace mixgcn;

namespace {

constexpr int BM = 128, BK = 16, NT = 256, TM = 8;
constexpr int FLUSH_TILES = 64;  // 64 * 16 = 1024 terms per first-level accumulator

struct Epi {
    const float* bias; int relu;
    const uint8_t* drop; float keep_scale;
    const float* gate; int64_t ld_gate; float gate_scale;
    const uint32_t* gate_bits; int64_t ld_gate_bits;   // bit-packed gate (replaces `gate`)
    int64_t row0;
};

__device__ __forceinline__ float apply_epi(const Epi& e, float y, int64_t m, int64_t n, int64_t N) {
    if (e.bias) y += e.bias[n];
    if (e.relu) y = fmaxf(y, 0.0f);
    if (e.drop) y = e.drop[(e.row0 + m) * N + n] ? y * e.keep_scale : 0.0f;
    if (e.gate) y = e.gate[(e.row0 + m) * e.ld_gate + n] > 0.0f ? y * e.gate_scale : 0.0f;
    if (e.gate_bits) y = ((e.gate_bits[(e.row0 + m) * e.ld_gate_bits + (n >> 5)] >> (n & 31)) & 1u) ? y * e.gate_scale : 0.0f;
    return y;
}

// Up to four consecutive floats src[0..3], element t valid iff t < valid; invalid ones are zero.
__device__ __forceinline__ float4 load_tail(const float* src, int64_t valid) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid > 0) v.x = src[0];
    if (valid > 1) v.y = src[1];
    if (valid > 2) v.z = src[2];
    if (valid > 3) v.w = src[3];
    return v;
}

struct GemmParams {
    int64_t M, N, K;
    const float* A; int64_t lda;
    const float* B; int64_t ldb;
    float* C; int64_t ldc;       // output, or partial workspace [splits][M][N] when splits > 1
    int64_t k_per_split; int splits;
    int64_t m_tiles, n_tiles;
    int vec_a, vec_b, vec_c;     // 16-byte vector access is legal (pointer and ld aligned)
    Epi epi;
};

template <int BN, int TN, bool TA, bool TB>
__global__ void __launch_bounds__(NT) gemm_simt_kernel(const GemmParams p) {
    constexpr int LDA_S = BM + 4, LDB_S = BN + 4;
    __shared__ __align__(16) float As[BK][LDA_S];
    __shared__ __align__(16) float Bs[BK][LDB_S];
    constexpr int A_V = BM * BK / 4 / NT;   // float4 per thread for the A tile (2)
    constexpr int B_V = BK * BN / 4 / NT;   // float4 per thread for the B tile (2 or 1)

    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int64_t tile = blockIdx.x;
    const int64_t m0 = (tile / p.n_tiles) * BM, n0 = (tile % p.n_tiles) * BN;
    const int64_t kb = (int64_t)blockIdx.z * p.k_per_split;
    const int64_t ke = (kb + p.k_per_split < p.K) ? kb + p.k_per_split : p.K;

    float4 ra[A_V], rb[B_V];

    auto load_regs = [&](int64_t k0) {
#pragma unroll
        for (int i = 0; i < A_V; ++i) {
            const int f = tid + i * NT;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (!TA) {  // A is M x K, contiguous along k
                const int64_t m = m0 + f / 4, k = k0 + (f % 4) * 4;
                if (m < p.M) {
                    const float* src = p.A + m * p.lda + k;
                    if (p.vec_a && k + 3 < ke) v = __ldg(reinterpret_cast<const float4*>(src));
                    else v = load_tail(src, ke - k);
                }
            } else {    // A is K x M, contiguous along m
                const int64_t k = k0 + f / (BM / 4), m = m0 + (f % (BM / 4)) * 4;
                if (k < ke) {
                    const float* src = p.A + k * p.lda + m;
                    if (p.vec_a && m + 3 < p.M) v = __ldg(reinterpret_cast<const float4*>(src));
                    else v = load_tail(src, p.M - m);
                }
            }
            ra[i] = v;
        }
#pragma unroll
        for (int i = 0; i < B_V; ++i) {
            const int f = tid + i * NT;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (!TB) {  // B is K x N, contiguous along n
                const int64_t k = k0 + f / (BN / 4), n = n0 + (f % (BN / 4)) * 4;
                if (k < ke) {
                    const float* src = p.B + k * p.ldb + n;
                    if (p.vec_b && n + 3 < p.N) v = __ldg(reinterpret_cast<const float4*>(src));
                    else v = load_tail(src, p.N - n);
                }
            } else {    // B is N x K, contiguous along k
                const int64_t n = n0 + f / 4, k = k0 + (f % 4) * 4;
                if (n < p.N) {
                    const float* src = p.B + n * p.ldb + k;
                    if (p.vec_b && k + 3 < ke) v = __ldg(reinterpret_cast<const float4*>(src));
                    else v = load_tail(src, ke - k);
                }
            }
            rb[i] = v;
        }
    };
    auto store_smem = [&]() {
#pragma unroll
        for (int i = 0; i < A_V; ++i) {
            const int f = tid + i * NT;
            if (!TA) {
                const int m = f / 4, k = (f % 4) * 4;
                As[k][m] = ra[i].x; As[k + 1][m] = ra[i].y; As[k + 2][m] = ra[i].z; As[k + 3][m] = ra[i].w;
            } else {
                const int k = f / (BM / 4), m = (f % (BM / 4)) * 4;
                *reinterpret_cast<float4*>(&As[k][m]) = ra[i];
            }
        }
#pragma unroll
        for (int i = 0; i < B_V; ++i) {
            const int f = tid + i * NT;
            if (!TB) {
                const int k = f / (BN / 4), n = (f % (BN / 4)) * 4;
                *reinterpret_cast<float4*>(&Bs[k][n]) = rb[i];
            } else {
                const int n = f / 4, k = (f % 4) * 4;
                Bs[k][n] = rb[i].x; Bs[k + 1][n] = rb[i].y; Bs[k + 2][n] = rb[i].z; Bs[k + 3][n] = rb[i].w;
            }
        }
    };

    float acc[TM][TN], tot[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) { acc[i][j] = 0.f; tot[i][j] = 0.f; }

    int since_flush = 0;
    if (kb < ke) load_regs(kb);
    for (int64_t k0 = kb; k0 < ke; k0 += BK) {
        store_smem();
        __syncthreads();
        if (k0 + BK < ke) load_regs(k0 + BK);
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float a[TM], b[TN];
            const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * TM]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[k][ty * TM + 4]);
            a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w; a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
#pragma unroll
            for (int q = 0; q < TN / 4; ++q) {
                const float4 bq = *reinterpret_cast<const float4*>(&Bs[k][q * 64 + tx * 4]);
                b[q * 4] = bq.x; b[q * 4 + 1] = bq.y; b[q * 4 + 2] = bq.z; b[q * 4 + 3] = bq.w;
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
        if (++since_flush == FLUSH_TILES) {
            since_flush = 0;
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) { tot[i][j] += acc[i][j]; acc[i][j] = 0.f; }
        }
    }
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) tot[i][j] += acc[i][j];

    const bool partial = p.splits > 1;
    float* Cb = partial ? p.C + (int64_t)blockIdx.z * p.M * p.N : p.C;
    const int64_t ldc = partial ? p.N : p.ldc;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t m = m0 + ty * TM + i;
        if (m >= p.M) continue;
#pragma unroll
        for (int q = 0; q < TN / 4; ++q) {
            const int64_t n = n0 + q * 64 + tx * 4;
            float r[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                r[t] = tot[i][q * 4 + t];
                if (!partial && n + t < p.N) r[t] = apply_epi(p.epi, r[t], m, n + t, p.N);
            }
            float* dst = Cb + m * ldc + n;
            if (p.vec_c && n + 3 < p.N && !partial) *reinterpret_cast<float4*>(dst) = make_float4(r[0], r[1], r[2], r[3]);
            else {
#pragma unroll
                for (int t = 0; t < 4; ++t) if (n + t < p.N) dst[t] = r[t];
            }
        }
    }
}

// C[m][n] = epilogue( sum_z part[z][m][n] ), z ascending, fp64 accumulation.
__global__ void splitk_reduce_kernel(int64_t M, int64_t N, int splits, const float* __restrict__ part,
                                     float* __restrict__ C, int64_t ldc, const Epi epi) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M * N) return;
    double s = 0.0;
    for (int z = 0; z < splits; ++z) s += (double)part[(int64_t)z * M * N + i];
    const int64_t m = i / N, n = i % N;
    C[m * ldc + n] = apply_epi(epi, (float)s, m, n, N);
}

// Column sums of an n x d matrix: block b sums rows [b*R, (b+1)*R) into part[b][d].
// A thread owns one float4 column group and every (256/groups)-th row of the block's range, four
// rows in flight; the row lanes are then added in fixed order through shared memory.  Requires
// ld % 4 == 0 and a 16-byte aligned X (the activations' layout).
__global__ void __launch_bounds__(256) colsum_partial_kernel(int64_t n, int d, const float* __restrict__ X, int64_t ld,
                                                             int64_t rows_per_block, int groups_pad,
                                                             float* __restrict__ part) {
    __shared__ float4 sm[256];
    const int d4 = (d + 3) >> 2;
    const int rl_n = 256 / groups_pad;                 // row lanes
    const int cg = threadIdx.x % groups_pad, rl = threadIdx.x / groups_pad;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
    const int64_t r1 = (r0 + rows_per_block < n) ? r0 + rows_per_block : n;
    for (int g0 = 0; g0 < d4; g0 += groups_pad) {
        const int g = g0 + cg;
        float4 acc[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (g < d4) {
            const float4* base = reinterpret_cast<const float4*>(X) + g;
            const int64_t ld4 = ld >> 2;
            int64_t r = r0 + rl;
            for (; r + 3 * rl_n < r1; r += 4 * rl_n) {
                float4 v[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) v[t] = __ldg(base + (r + t * rl_n) * ld4);
#pragma unroll
                for (int t = 0; t < 4; ++t) { acc[t].x += v[t].x; acc[t].y += v[t].y; acc[t].z += v[t].z; acc[t].w += v[t].w; }
            }
            for (int t = 0; r < r1; r += rl_n, ++t) {
                const float4 v = __ldg(base + r * ld4);
                acc[t & 3].x += v.x; acc[t & 3].y += v.y; acc[t & 3].z += v.z; acc[t & 3].w += v.w;
            }
        }
        float4 s4;
        s4.x = (acc[0].x + acc[1].x) + (acc[2].x + acc[3].x);
        s4.y = (acc[0].y + acc[1].y) + (acc[2].y + acc[3].y);
        s4.z = (acc[0].z + acc[1].z) + (acc[2].z + acc[3].z);
        s4.w = (acc[0].w + acc[1].w) + (acc[2].w + acc[3].w);
        sm[threadIdx.x] = s4;
        __syncthreads();
        if (rl == 0 && g < d4) {
            float4 t = sm[cg];
            for (int q = 1; q < rl_n; ++q) {
                const float4 u = sm[q * groups_pad + cg];
                t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
            }
            float* dst = part + (int64_t)blockIdx.x * d + g * 4;
            const float tv[4] = {t.x, t.y, t.z, t.w};
            for (int c = 0; c < 4; ++c) if (g * 4 + c < d) dst[c] = tv[c];
        }
        __syncthreads();
    }
}

__global__ void colsum_final_kernel(int d, int blocks, const float* __restrict__ part, float* __restrict__ out) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d) return;
    double s = 0.0;
    for (int b = 0; b < blocks; ++b) s += (double)part[(int64_t)b * d + j];
    out[j] = (float)s;
}

// G <- G * 1[X_out > 0] (ReLU) * (drop ? keep_scale : 0): gradient w.r.t. the pre-activation.
__global__ void gate_kernel(int64_t n, int d, float* __restrict__ G, int64_t ldg, const float* __restrict__ Xo,
                            int64_t ldx, int relu, const uint8_t* __restrict__ drop, float keep_scale) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * d) return;
    const int64_t r = i / d; const int j = (int)(i % d);
    float g = G[r * ldg + j];
    if (relu && !(Xo[r * ldx + j] > 0.0f)) g = 0.0f;
    if (drop) g = drop[i] ? g * keep_scale : 0.0f;
    G[r * ldg + j] = g;
}

template <int BN, int TN>
void launch_variant(const GemmParams& p, int ta, int tb, dim3 grid, cudaStream_t s) {
    if (!ta && !tb) gemm_simt_kernel<BN, TN, false, false><<<grid, NT, 0, s>>>(p);
    else if (!ta && tb) gemm_simt_kernel<BN, TN, false, true><<<grid, NT, 0, s>>>(p);
    else if (ta && !tb) gemm_simt_kernel<BN, TN, true, false><<<grid, NT, 0, s>>>(p);
    else gemm_simt_kernel<BN, TN, true, true><<<grid, NT, 0, s>>>(p);
}

}  // namespace

namespace mixgcn {

mixgcn_status launch_gemm_simt(mixgcn_ctx* ctx, int ta, int tb, int64_t M, int64_t N, int64_t K,
                               const float* A, int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc,
                               const mixgcn_epilogue* epi, int64_t epi_row0, cudaStream_t s) {
    if (M <= 0 || N <= 0) return MIXGCN_OK;
    GemmParams p{};
    p.M = M; p.N = N; p.K = K; p.A = A; p.lda = lda; p.B = B; p.ldb = ldb; p.C = C; p.ldc = ldc;
    if (epi) {
        p.epi.bias = epi->bias; p.epi.relu = epi->relu; p.epi.drop = epi->drop_mask;
        p.epi.keep_scale = epi->keep_scale; p.epi.gate = epi->gate_bits ? nullptr : epi->gate; p.epi.ld_gate = epi->ld_gate;
        p.epi.gate_scale = epi->gate_scale;
        p.epi.gate_bits = epi->gate_bits; p.epi.ld_gate_bits = epi->ld_gate_bits;
    }
    p.epi.row0 = epi_row0;
    p.vec_a = aligned16(A) && (lda & 3) == 0;
    p.vec_b = aligned16(B) && (ldb & 3) == 0;
    p.vec_c = aligned16(C) && (ldc & 3) == 0;
    const int bn = N <= 64 ? 64 : 128;
    p.m_tiles = (M + BM - 1) / BM;
    p.n_tiles = (N + bn - 1) / bn;
    const int64_t tiles = p.m_tiles * p.n_tiles;
    int splits = 1;
    if (K > 8192 && tiles < 2 * ctx->sm_count) {
        int64_t want = (2 * ctx->sm_count + tiles - 1) / tiles;
        int64_t maxs = (K + 4095) / 4096;
        splits = (int)(want < maxs ? want : maxs);
        if (splits > 1024) splits = 1024;
        if (splits < 1) splits = 1;
    }
    int64_t kps = (K + splits - 1) / splits;
    kps = ((kps + BK - 1) / BK) * BK;
    if (kps <= 0) kps = BK;
    splits = (int)((K + kps - 1) / kps);
    if (splits < 1) splits = 1;
    p.k_per_split = kps; p.splits = splits;
    if (splits > 1) {
        MIXGCN_TRY(ensure_workspace(ctx, (int64_t)splits * M * N * (int64_t)sizeof(float)));
        p.C = reinterpret_cast<float*>(ctx->workspace);
    }
    if (tiles > 0x7FFFFFFFll) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "gemm: too many tiles");
    dim3 grid((unsigned)tiles, 1, (unsigned)splits);
    {
        LaunchScope scope(ctx, PH_GEMM, s);
        if (bn == 64) launch_variant<64, 4>(p, ta, tb, grid, s);
        else launch_variant<128, 8>(p, ta, tb, grid, s);
    }
    if (splits > 1) {
        LaunchScope scope(ctx, PH_GEMM, s);
        const int64_t total = M * N;
        splitk_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(M, N, splits, p.C, C, ldc, p.epi);
    }
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

mixgcn_status launch_splitk_reduce(mixgcn_ctx* ctx, int64_t M, int64_t N, int splits, const float* part, float* C,
                                   int64_t ldc, const mixgcn_epilogue* epi, cudaStream_t s) {
    Epi e{};
    if (epi) {
        e.bias = epi->bias; e.relu = epi->relu; e.drop = epi->drop_mask; e.keep_scale = epi->keep_scale;
        e.gate = epi->gate_bits ? nullptr : epi->gate; e.ld_gate = epi->ld_gate; e.gate_scale = epi->gate_scale;
        e.gate_bits = epi->gate_bits; e.ld_gate_bits = epi->ld_gate_bits;
    }
    LaunchScope scope(ctx, PH_GEMM, s);
    const int64_t total = M * N;
    splitk_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(M, N, splits, part, C, ldc, e);
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

mixgcn_status launch_colsum(mixgcn_ctx* ctx, int64_t n, int32_t d, const float* X, int64_t ld, float* out,
                            cudaStream_t s) {
    int64_t rows_per_block = 2048;
    int64_t blocks = (n + rows_per_block - 1) / rows_per_block;
    if (blocks > 2048) { rows_per_block = (n + 2047) / 2048; blocks = (n + rows_per_block - 1) / rows_per_block; }
    if (blocks < 1) blocks = 1;
    MIXGCN_TRY(ensure_workspace(ctx, blocks * d * (int64_t)sizeof(float)));
    float* part = reinterpret_cast<float*>(ctx->workspace);
    {
        LaunchScope scope(ctx, PH_ELEM, s);
        int groups_pad = 1;
        while (groups_pad < 256 && groups_pad < (d + 3) / 4) groups_pad <<= 1;
        colsum_partial_kernel<<<(unsigned)blocks, 256, 0, s>>>(n, d, X, ld, rows_per_block, groups_pad, part);
    }
    {
        LaunchScope scope(ctx, PH_ELEM, s);
        colsum_final_kernel<<<(d + 127) / 128, 128, 0, s>>>(d, (int)blocks, part, out);
    }
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

mixgcn_status launch_gate(mixgcn_ctx* ctx, int64_t n, int32_t d, float* G, int64_t ldg, const float* X_out,
                          int64_t ldx, int relu, const uint8_t* drop_mask, float keep_scale, cudaStream_t s) {
    const int64_t total = n * d;
    if (total <= 0) return MIXGCN_OK;
    LaunchScope scope(ctx, PH_ELEM, s);
    gate_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(n, d, G, ldg, X_out, ldx, relu, drop_mask, keep_scale);
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

}  // namespace mixgcn
