// Dense update products on the 5th-generation tensor cores (tcgen05) for sm_100a:
// the update line of Algorithm 2 (P = Z W) and its two backward products (dZ = dP W^T,
// dW = Z^T dP) with fp32 accumulation in tensor memory, in two operand kinds:
//   TF32 -- operands read straight from the fp32 activations (tcgen05.mma.kind::tf32);
//   BF16 -- operands are bf16 copies of the activations (tcgen05.mma.kind::f16), half the bytes per
//           operand element on the way from the L2 to shared memory and into the tensor core.
// The two kinds share every line of the kernels except the element size: a stage row is 128 bytes of
// K (32 fp32 or 64 bf16) and one instruction consumes 32 bytes of it (K = 8 or 16).
//
//  * Operands reach shared memory by TMA (cp.async.bulk.tensor, 128-byte swizzle, out-of-bounds
//    elements filled with zeros, so ragged M / N / K tails need no special code).
//  * One elected thread issues tcgen05.mma (M = 128, N <= 256); the 128 x N fp32 accumulator lives in
//    TMEM and is read back with tcgen05.ld for the fused epilogue (bias, ReLU, dropout mask, gate), the
//    single store of C and, on request, a bf16 copy of C for the next product.
//  * Stages are handed over with mbarriers; every wait is bounded: on expiry the CTA records
//    DEV_WAIT_EXPIRED in the status word, stops issuing work, frees its TMEM and returns.
//  * Two operand forms.  "KK": A is M x K row-major (K contiguous) and B is N x K row-major -- the
//    forward product and dZ, with the small weight matrix first packed (transposed if needed, zero
//    padded, converted to the kind's type) into the workspace.  "MM": A is K x M and B is K x N
//    row-major (M / N contiguous, K = node count) -- the weight gradient, split over CTAs along K into
//    partial tiles that the fixed-order fp64 reduction combines.
#include <cuda.h>

#include "internal.cuh"
#include "tc_ptx.cuh"

using namespace mixgcn;
using namespace mixgcn::tc;

namespace {

constexpr int TC_BM = 128;          // rows of D per CTA = UMMA M
constexpr int TC_THREADS = 192;

// What differs between the operand kinds.
template <int KIND>
struct KindCfg {
    static constexpr int EB = KIND == KIND_TF32 ? 4 : 2;        // bytes per operand element
    static constexpr int BK = 128 / EB;                         // elements of K per stage (one 128-byte swizzle row; BK k-rows in the MN-major form)
    static constexpr int MMA_K = 32 / EB;                       // K of one tcgen05.mma
    // MN-major form: a chunk is 128 bytes of M / N (BK elements wide) by BK k-rows
    static constexpr int CHUNK = 128 / EB;                      // elements of M / N per chunk
    static constexpr uint32_t MN_LAYOUT = KIND == KIND_TF32 ? 1u : 2u;
    static constexpr uint32_t MN_SBO = KIND == KIND_TF32 ? 512u : 1024u;   // one K atom (4 / 8 k-rows of 128 bytes)
    static constexpr uint32_t MN_CHUNK_BYTES = BK * 128;        // = leading byte offset
    static constexpr uint32_t MN_STEP = MMA_K * 128;            // k-rows of one instruction
};

struct TcEpi {
    const float* bias; int relu;
    const uint8_t* drop; float keep_scale;
    const float* gate; int64_t ld_gate; float gate_scale;
    const uint32_t* gate_bits; int64_t ld_gate_bits;   // bit-packed gate (replaces `gate`): bit j & 31 of word j >> 5 of row i
    uint32_t* sign_bits; int64_t ld_sign_bits;         // output: bit = (final y > 0), written by the K-major kernels' epilogues
    int64_t row0;
};

struct TcParams {
    int64_t M, N, K;
    int bn;                 // UMMA N: multiple of 16, 16..256
    int stages;
    int64_t m_tiles, n_tiles;
    int64_t k_per_split;    // MM form: multiple of the kind's BK
    int splits;
    float* C; int64_t ldc; int vec_c;
    uint16_t* C_lp; int64_t ldc_lp;   // nullable: bf16 copy of C (after the epilogue); ldc_lp a multiple of 8
    int raw;                // 1: store the accumulator unchanged (split-K partial)
    double* colsum_part;    // weight-gradient form, TF32: nullable [splits][N] column sums of B over this split's k-rows
    TcEpi epi;
    int32_t* status;
    uint32_t wait_limit;    // polls after which a wait gives up
    int debug_drop_load;    // test hook: the producer leaves out the loads of its first stage (the wait on it then expires)
    int epi_boxes;          // single-CTA K-major kernel: staging boxes per epilogue warp (1 or 2)
    // arg-max epilogue of the single-CTA K-major kernel (LOSS instances; one n-tile): C receives the train rows only
    const uint8_t* loss_mask; int32_t* loss_pred; int loss_zero_rows;
};

__device__ __forceinline__ float tc_apply_epi(const TcEpi& e, float y, int64_t m, int64_t n, int64_t N) {
    if (e.bias) y += e.bias[n];
    if (e.relu) y = fmaxf(y, 0.0f);
    if (e.drop) y = e.drop[(e.row0 + m) * N + n] ? y * e.keep_scale : 0.0f;
    if (e.gate) y = e.gate[(e.row0 + m) * e.ld_gate + n] > 0.0f ? y * e.gate_scale : 0.0f;
    if (e.gate_bits) y = ((e.gate_bits[(e.row0 + m) * e.ld_gate_bits + (n >> 5)] >> (n & 31)) & 1u) ? y * e.gate_scale : 0.0f;
    return y;
}

// bit q = (v[q] > 0) for the columns nb + q < N of one row's 32-column chunk
__device__ __forceinline__ uint32_t sign_word(const float (&v)[32], int64_t nb, int64_t N) {
    uint32_t w = 0;
#pragma unroll
    for (int q = 0; q < 32; ++q) w |= (v[q] > 0.0f ? 1u : 0u) << q;
    const int64_t left = N - nb;
    return left >= 32 ? w : (w & ((1u << (int)left) - 1u));
}

__device__ __forceinline__ bool aligned16_dev(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// 32 consecutive columns of one row as bf16 (round to nearest even); dst is 16-byte aligned when full.
__device__ __forceinline__ void store_lp_row(uint16_t* dst, const float (&v)[32], int valid) {
    if (valid >= 32) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
            reinterpret_cast<uint4*>(dst)[q] = make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                                                           pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
    } else {
#pragma unroll
        for (int q = 0; q < 32; ++q)
            if (q < valid) dst[q] = (uint16_t)(pack_bf16(v[q], 0.0f) & 0xFFFFu);
    }
}

// One output tile per CTA; MN_MAJOR = true is the split-K weight-gradient form (grid.z = split).
// Warp roles: warps 0-3 epilogue (TMEM lane quarter = warp id), warp 4 TMA producer, warp 5 TMEM
// allocation + MMA issue.
template <int KIND, bool MN_MAJOR>
__global__ void __launch_bounds__(TC_THREADS) gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a,
                                                             const __grid_constant__ CUtensorMap map_b,
                                                             const TcParams p) {
    using Cfg = KindCfg<KIND>;
    constexpr int BK = Cfg::BK;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[8], empty_bar[8], acc_bar;
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bn_pad = MN_MAJOR ? (p.bn + Cfg::CHUNK - 1) / Cfg::CHUNK * Cfg::CHUNK : (p.bn + 31) & ~31;
    const uint32_t a_bytes = TC_BM * 128, b_bytes = (uint32_t)bn_pad * 128;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    const int64_t tile = blockIdx.x;
    const int64_t m0 = (tile / p.n_tiles) * TC_BM, n0 = (tile % p.n_tiles) * p.bn;
    int64_t kb = 0, ke = p.K;
    if (MN_MAJOR) {
        kb = (int64_t)blockIdx.z * p.k_per_split;
        ke = kb + p.k_per_split < p.K ? kb + p.k_per_split : p.K;
    }
    const int nk = (int)((ke - kb + BK - 1) / BK);
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < p.bn) tmem_cols <<= 1;

    // Column sums of B (the bias gradient 1^T dP when B = dP) as a by-product: the four epilogue warps are
    // idle while the tiles stream through shared memory, so in the CTAs of the first row of tiles they add up
    // each stage's B tile (fp32 words, TF32 kind only) before the stage is released.
    const bool do_colsum = MN_MAJOR && KIND == KIND_TF32 && p.colsum_part != nullptr && tile / p.n_tiles == 0;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], do_colsum ? 5 : 1); }
        mbar_init(&acc_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_holder)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;

    if (warp == 4) {
        if (lane == 0) {
            // ---------------- TMA producer ----------------
            for (int ks = 0; ks < nk; ++ks) {
                const int s = ks % p.stages;
                const uint32_t ph = ((ks / p.stages) & 1) ^ 1;
                if (!mbar_wait(&empty_bar[s], ph, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); break; }
                uint8_t* sa = smem + (size_t)s * stage_bytes;
                uint8_t* sb = sa + a_bytes;
                mbar_expect_tx(&full_bar[s], stage_bytes);
                const int32_t k0 = (int32_t)(kb + (int64_t)ks * BK);
                if (!MN_MAJOR) {
                    tma_load_2d(sa, &map_a, k0, (int32_t)m0, &full_bar[s]);                  // 128 rows x 128 bytes of k
                    tma_load_2d(sb, &map_b, k0, (int32_t)n0, &full_bar[s]);                  // bn_pad rows x 128 bytes of k
                } else {
                    for (int c = 0; c < TC_BM / Cfg::CHUNK; ++c)                              // BK k-rows x 128 bytes of m each
                        tma_load_2d(sa + c * Cfg::MN_CHUNK_BYTES, &map_a, (int32_t)(m0 + Cfg::CHUNK * c), k0, &full_bar[s]);
                    for (int c = 0; c < bn_pad / Cfg::CHUNK; ++c)
                        tma_load_2d(sb + c * Cfg::MN_CHUNK_BYTES, &map_b, (int32_t)(n0 + Cfg::CHUNK * c), k0, &full_bar[s]);
                }
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            const uint32_t idesc = make_idesc<KIND>(TC_BM, p.bn, MN_MAJOR);
            bool ok = true;
            for (int ks = 0; ks < nk && ok; ++ks) {
                const int s = ks % p.stages;
                const uint32_t ph = (ks / p.stages) & 1;
                if (!mbar_wait(&full_bar[s], ph, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; break; }
                tc_fence_after();
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes), sb = sa + a_bytes;
#pragma unroll
                for (int kq = 0; kq < BK / Cfg::MMA_K; ++kq) {
                    uint64_t ad, bd;
                    if (!MN_MAJOR) {
                        ad = make_desc(sa + kq * 32, 16, 1024, 2);
                        bd = make_desc(sb + kq * 32, 16, 1024, 2);
                    } else {
                        ad = make_desc(sa + kq * Cfg::MN_STEP, Cfg::MN_CHUNK_BYTES, Cfg::MN_SBO, Cfg::MN_LAYOUT);
                        bd = make_desc(sb + kq * Cfg::MN_STEP, Cfg::MN_CHUNK_BYTES, Cfg::MN_SBO, Cfg::MN_LAYOUT);
                    }
                    tc_mma<KIND>(tmem_base, ad, bd, idesc, (ks | kq) != 0 ? 1u : 0u);
                }
                tc_commit(&empty_bar[s]);     // the stage is free once these MMAs have read it
            }
            if (ok) tc_commit(&acc_bar);      // the accumulator is complete
        }
    } else {
        // ---------------- epilogue: warps 0..3 own TMEM lanes 32*warp .. 32*warp+31 ----------------
        bool ok = true;
        if (do_colsum) {
            // warp w takes the 32-column chunks w and w + 4 of the B tile, lane l their column l.  A chunk is BK
            // k-rows of 128 bytes in the 128-byte swizzle with 32-byte atoms: the 32-byte group g of k-row r sits
            // at group position g ^ (r & 3).
            double sum[2] = {0.0, 0.0};
            const int chunks = bn_pad / Cfg::CHUNK;
            for (int ks = 0; ks < nk && ok; ++ks) {
                const int s = ks % p.stages;
                const uint32_t ph = (ks / p.stages) & 1;
                if (lane == 0) ok = mbar_wait(&full_bar[s], ph, &abort_flag, p.wait_limit);
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                if (!ok) { if (lane == 0) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); } break; }
                const uint8_t* sb = smem + (size_t)s * stage_bytes + a_bytes;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int cc = warp + 4 * h;
                    if (cc < chunks) {
                        const float* chunk = reinterpret_cast<const float*>(sb + (size_t)cc * Cfg::MN_CHUNK_BYTES);
                        float part = 0.0f;
#pragma unroll 8
                        for (int r = 0; r < BK; ++r) part += chunk[r * 32 + (lane ^ ((r & 3) << 3))];
                        sum[h] += (double)part;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[s]);      // this warp has read the stage
            }
            if (ok) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int cc = warp + 4 * h;
                    const int64_t n = n0 + cc * 32 + lane;
                    if (cc < chunks && cc * 32 + lane < p.bn && n < p.N) p.colsum_part[(int64_t)blockIdx.z * p.N + n] = sum[h];
                }
            }
        }
        if (ok && nk > 0) {
            if (lane == 0) ok = mbar_wait(&acc_bar, 0, &abort_flag, p.wait_limit);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok && lane == 0) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); }
        }
        __syncwarp();
        tc_fence_after();
        if (ok) {
            const int64_t m = m0 + warp * 32 + lane;
            float* Cb = p.C + (MN_MAJOR && p.raw ? (int64_t)blockIdx.z * p.M * p.N : 0);
            for (int c0 = 0; c0 < p.bn; c0 += 32) {
                uint32_t r[32];
                if (nk > 0) {
                    tc_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, r);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                if (m < p.M) {
                    const int64_t nb = n0 + c0;
                    float* dst = Cb + m * p.ldc + nb;
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        v[j] = __uint_as_float(r[j]);
                        if (!p.raw && nb + j < p.N) v[j] = tc_apply_epi(p.epi, v[j], m, nb + j, p.N);
                    }
                    if (p.vec_c && nb + 31 < p.N && c0 + 31 < p.bn) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (nb + j < p.N && c0 + j < p.bn) dst[j] = v[j];
                    }
                }
            }
        }
    }
    if (threadIdx.x == 0 && abort_flag) {
        // a wait expired: give copies that may still be in flight time to land before the CTA retires
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

constexpr int KK_EPI_WARPS = 8;                       // two per TMEM lane quarter, each takes every other 32-column chunk
constexpr int KK_THREADS = (KK_EPI_WARPS + 2) * 32;    // + TMA producer warp + MMA warp
constexpr int KK_BIAS_MAX = 1024;

// Persistent K-major kernel for the tall products (M = node count): each CTA walks over output tiles
// (n fastest, so consecutive tiles of a CTA share their A rows in L2).  The TMA producer runs ahead
// through a ring of stages across tile boundaries, the accumulator is double-buffered in TMEM so the
// epilogue of tile j overlaps the loads and MMAs of tile j+1, and when the packed weight matrix is
// small enough it is loaded into shared memory once per CTA and stays there.  The epilogue (eight
// warps) applies bias / ReLU from registers and shared memory, writes 32-row x 128-byte boxes in the
// 128-byte swizzle and hands them to TMA stores, which also clip ragged M / N edges; the optional bf16
// copy of C goes out with 16-byte stores straight from the registers.
// LOSS instances (one n-tile, N <= 256: a row of C is a row of logits for a masked loss): the epilogue finds
// every row's arg-max (-> pred) and writes the logits of the TRAIN rows only (the others are zeroed or left
// alone) -- all the loss that follows needs.  The two epilogue warps of a lane quarter then take alternate
// TILES (one accumulator buffer each) instead of alternate column chunks, so that one thread sees its whole row.
template <int KIND, bool LOSS = false>
__global__ void __launch_bounds__(KK_THREADS, 1) gemm_tc_kk_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                const __grid_constant__ CUtensorMap map_b,
                                                                const __grid_constant__ CUtensorMap map_c,
                                                                const TcParams p, const int b_resident, const int tma_store) {
    using Cfg = KindCfg<KIND>;
    constexpr int BK = Cfg::BK;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[8], empty_bar[8], acc_full[2], acc_empty[2], b_bar;
    __shared__ __align__(16) float s_bias[KK_BIAS_MAX + 32];
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bn32 = (p.bn + 31) & ~31;
    const uint32_t a_bytes = TC_BM * 128, b_bytes = (uint32_t)bn32 * 128;
    const int nk = (int)((p.K + BK - 1) / BK);
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // layout: [resident B: nk * b_bytes] [ring of stages: A (+ B when not resident)] [one output box per epilogue warp]
    uint8_t* smem_b_res = smem;
    uint8_t* smem_ring = smem + (b_resident ? (size_t)nk * b_bytes : 0);
    const uint32_t stage_bytes = a_bytes + (b_resident ? 0u : b_bytes);
    uint8_t* smem_out = smem_ring + (size_t)p.stages * stage_bytes;

    const int64_t tiles = p.m_tiles * p.n_tiles;
    uint32_t acc_stride = 32;
    while ((int)acc_stride < p.bn) acc_stride <<= 1;
    const uint32_t tmem_cols = acc_stride * 2;
    const bool bias_in_smem = p.epi.bias != nullptr && p.N <= KK_BIAS_MAX;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], LOSS ? KK_EPI_WARPS / 2 : KK_EPI_WARPS); }
        mbar_init(&b_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (bias_in_smem)
        for (int i = threadIdx.x; i < KK_BIAS_MAX + 32; i += KK_THREADS) s_bias[i] = i < p.N ? p.epi.bias[i] : 0.0f;
    if (warp == KK_EPI_WARPS + 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_holder)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;

    if (warp == KK_EPI_WARPS) {
        if (lane == 0) {
            // ---------------- TMA producer ----------------
            bool ok = true;
            if (b_resident) {
                mbar_expect_tx(&b_bar, (uint32_t)nk * b_bytes);
                for (int ks = 0; ks < nk; ++ks) tma_load_2d(smem_b_res + (size_t)ks * b_bytes, &map_b, ks * BK, 0, &b_bar);
            }
            uint32_t it = 0;
            for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                const int32_t m0 = (int32_t)((tile / p.n_tiles) * TC_BM), n0 = (int32_t)((tile % p.n_tiles) * p.bn);
                for (int ks = 0; ks < nk; ++ks, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = ((it / p.stages) & 1) ^ 1;
                    if (!mbar_wait(&empty_bar[s], ph, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; break; }
                    uint8_t* sa = smem_ring + (size_t)s * stage_bytes;
                    mbar_expect_tx(&full_bar[s], stage_bytes);
                    if (p.debug_drop_load && it == 0) continue;      // test hook: this stage never fills
                    tma_load_2d(sa, &map_a, ks * BK, m0, &full_bar[s]);
                    if (!b_resident) tma_load_2d(sa + a_bytes, &map_b, ks * BK, n0, &full_bar[s]);
                }
            }
        }
    } else if (warp == KK_EPI_WARPS + 1) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            const uint32_t idesc = make_idesc<KIND>(TC_BM, p.bn, false);
            bool ok = true;
            if (b_resident) {
                if (!mbar_wait(&b_bar, 0, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; }
            }
            uint32_t it = 0, j = 0;
            for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++j) {
                const uint32_t buf = j & 1;
                if (!mbar_wait(&acc_empty[buf], ((j >> 1) & 1) ^ 1, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * acc_stride;
                for (int ks = 0; ks < nk; ++ks, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (it / p.stages) & 1;
                    if (!mbar_wait(&full_bar[s], ph, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem_ring + (size_t)s * stage_bytes);
                    const uint32_t sb = b_resident ? smem_u32(smem_b_res + (size_t)ks * b_bytes) : sa + a_bytes;
#pragma unroll
                    for (int kq = 0; kq < BK / Cfg::MMA_K; ++kq)
                        tc_mma<KIND>(d_tmem, make_desc(sa + kq * 32, 16, 1024, 2), make_desc(sb + kq * 32, 16, 1024, 2), idesc,
                                     (ks | kq) != 0 ? 1u : 0u);
                    tc_commit(&empty_bar[s]);
                }
                if (ok) tc_commit(&acc_full[buf]);
            }
        }
    } else if constexpr (LOSS) {
        // ---------------- arg-max epilogue: warp w reads TMEM lanes 32*(w&3).. of the tiles j = (w>>2), (w>>2)+2, ... ----------------
        // A thread sees its whole row of logits (sums + bias), 32 columns at a time: per chunk a tree of maxima
        // and the lowest position that attains it (independent operations, no long dependent chain), then one
        // strict comparison against the running maximum (an earlier chunk keeps a tie).  The row itself is
        // written only if it is a train row (zeros elsewhere when every row is wanted).
        const int quarter = warp & 3, half = warp >> 2;
        const bool add_bias = p.epi.bias != nullptr && bias_in_smem;
        const bool use_tma = tma_store != 0;              // every row is written: through the staged boxes
        const int N = (int)p.N;
        uint8_t* const box = smem_out + (size_t)warp * p.epi_boxes * 4096;
        uint32_t j = (uint32_t)half;
        bool ok = true;
        for (int64_t tile = blockIdx.x + (int64_t)half * gridDim.x; tile < tiles && ok; tile += 2 * (int64_t)gridDim.x, j += 2) {
            const uint32_t buf = j & 1;
            const int64_t m0 = tile * TC_BM;                 // one n-tile
            const int64_t m = m0 + quarter * 32 + lane;
            const bool row_ok = m < p.M;
            const bool train = row_ok && __ldg(p.loss_mask + m) != 0;     // requested before the accumulator is waited for
            if (lane == 0) ok = mbar_wait(&acc_full[buf], (j >> 1) & 1, &abort_flag, p.wait_limit);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) { if (lane == 0) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); } break; }
            tc_fence_after();
            const uint32_t t_row = tmem_base + buf * acc_stride + ((uint32_t)(quarter * 32) << 16);
            float mx = -INFINITY; int arg = 0;             // nothing but -inf / NaN: 0
            for (int c0 = 0; c0 < p.bn; c0 += 32) {
                uint32_t r[32];
                tc_ld32(t_row + (uint32_t)c0, r);
                tc_wait_ld();
                float x[32];
                if (add_bias) {
                    const float4* sb4 = reinterpret_cast<const float4*>(s_bias + c0);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float4 b4 = sb4[q];
                        x[4 * q] = __uint_as_float(r[4 * q]) + b4.x; x[4 * q + 1] = __uint_as_float(r[4 * q + 1]) + b4.y;
                        x[4 * q + 2] = __uint_as_float(r[4 * q + 2]) + b4.z; x[4 * q + 3] = __uint_as_float(r[4 * q + 3]) + b4.w;
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < 32; ++q) x[q] = __uint_as_float(r[q]);
                }
                // the row's values leave first (train rows; zeros for the others when every row is written)
                if (use_tma) {
                    if (lane == 0) bulk_wait_read<0>();       // the store that last used this box has read it
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<float4*>(box + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                            train ? make_float4(x[4 * q], x[4 * q + 1], x[4 * q + 2], x[4 * q + 3]) : make_float4(0.f, 0.f, 0.f, 0.f);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&map_c, box, c0, (int32_t)(m0 + quarter * 32));
                        bulk_commit();
                    }
                } else if (train || (p.loss_zero_rows && row_ok)) {
                    float* dst = p.C + m * p.ldc + c0;
                    if (p.vec_c && c0 + 31 < N) {
#pragma unroll
                        for (int q = 0; q < 32; q += 4)
                            *reinterpret_cast<float4*>(dst + q) = train ? make_float4(x[q], x[q + 1], x[q + 2], x[q + 3]) : make_float4(0.f, 0.f, 0.f, 0.f);
                    } else {
#pragma unroll
                        for (int q = 0; q < 32; ++q)
                            if (c0 + q < N) dst[q] = train ? x[q] : 0.0f;
                    }
                }
                if (c0 + 32 > N) {                            // ragged last chunk: columns beyond N are not data
#pragma unroll
                    for (int q = 0; q < 32; ++q)
                        if (c0 + q >= N) x[q] = -INFINITY;
                }
                float t[16];
#pragma unroll
                for (int q = 0; q < 16; ++q) t[q] = fmaxf(x[q], x[q + 16]);
#pragma unroll
                for (int w = 8; w > 0; w >>= 1)
#pragma unroll
                    for (int q = 0; q < w; ++q) t[q] = fmaxf(t[q], t[q + w]);
                const float cm = t[0];
                if (__any_sync(0xFFFFFFFFu, cm > mx)) {       // some row of the warp has a new maximum in this chunk
                    int a4[4] = {32, 32, 32, 32};
#pragma unroll
                    for (int q = 31; q >= 0; --q)
                        if (x[q] == cm) a4[q & 3] = q;
                    const int ca = min(min(a4[0], a4[1]), min(a4[2], a4[3]));
                    if (cm > mx) { mx = cm; arg = c0 + ca; }
                }
            }
            if (row_ok && p.loss_pred) p.loss_pred[m] = arg;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
        if (tma_store && lane == 0) bulk_wait_all();
    } else {
        // ---------------- epilogue: warp w reads TMEM lanes 32*(w&3).., 32-column chunks (w>>2), (w>>2)+2, ... ----------------
        const int quarter = warp & 3, half = warp >> 2;
        // The dropout mask and the gate are per-element tensors of C's shape.  With TMA stores they are
        // applied on the staged box, where a row's 128 bytes belong to eight adjacent lanes (coalesced
        // reads of the gate); otherwise element by element from the registers, like a bias wider than the
        // shared-memory copy.
        const bool has_gate = p.epi.gate != nullptr || p.epi.gate_bits != nullptr;
        const bool post = (p.epi.drop != nullptr || has_gate) && tma_store;
        const bool generic = !post && (p.epi.drop != nullptr || has_gate || (p.epi.bias != nullptr && !bias_in_smem));
        const bool wide_bias = post && p.epi.bias != nullptr && !bias_in_smem;
        const bool add_bias = p.epi.bias != nullptr && bias_in_smem, relu = p.epi.relu != 0;
        const bool gate_vec = p.epi.gate != nullptr && aligned16_dev(p.epi.gate) && (p.epi.ld_gate & 3) == 0;
        // one staging box per warp, or two (short K: the epilogue is the critical path, and the second box is
        // filled while the TMA store of the first is still reading it)
        const int nboxes = p.epi_boxes;
        uint8_t* const box_base = smem_out + (size_t)warp * nboxes * 4096;
        uint32_t box_turn = 0;
        uint32_t j = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++j) {
            const uint32_t buf = j & 1;
            const int64_t m0 = (tile / p.n_tiles) * TC_BM;
            const int n0 = (int)((tile % p.n_tiles) * p.bn);
            if (lane == 0) ok = mbar_wait(&acc_full[buf], (j >> 1) & 1, &abort_flag, p.wait_limit);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) { if (lane == 0) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); } break; }
            tc_fence_after();
            const int64_t m = m0 + quarter * 32 + lane;
            const bool row_ok = m < p.M;
            for (int c0 = half * 32; c0 < p.bn; c0 += 64) {
                const int nb = n0 + c0;
                // the gate's 32 x 32 block in the staged-box orientation (lane = row it * 4 + lane / 8,
                // 16-byte chunk lane % 8), requested before the accumulator is read so that the loads overlap it
                float4 g4[8];
                if (post && p.epi.gate_bits) {
                    // bit-packed gate: this lane's row, the chunk's word (kept in the first slot of the fp32 gate's registers:
                    // the two forms exclude each other)
                    g4[0].x = __uint_as_float(row_ok ? __ldg(p.epi.gate_bits + (p.epi.row0 + m) * p.epi.ld_gate_bits + (nb >> 5)) : 0u);
                } else if (post && gate_vec) {
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int64_t mr = m0 + quarter * 32 + it * 4 + (lane >> 3);
                        const int nc = nb + (lane & 7) * 4;
                        g4[it] = (mr < p.M && nc < p.N) ? __ldg(reinterpret_cast<const float4*>(p.epi.gate + (p.epi.row0 + mr) * p.epi.ld_gate + nc))
                                                         : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                uint32_t r[32];
                tc_ld32(tmem_base + buf * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
                tc_wait_ld();
                float v[32];
#pragma unroll
                for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(r[q]);
                if (!generic) {
                    if (add_bias) {
                        const float4* sb4 = reinterpret_cast<const float4*>(s_bias + nb);
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const float4 b4 = sb4[q];
                            v[4 * q] += b4.x; v[4 * q + 1] += b4.y; v[4 * q + 2] += b4.z; v[4 * q + 3] += b4.w;
                        }
                    } else if (wide_bias) {
#pragma unroll
                        for (int q = 0; q < 32; ++q)
                            if (nb + q < p.N) v[q] += p.epi.bias[nb + q];
                    }
                    if (relu) {
#pragma unroll
                        for (int q = 0; q < 32; ++q) v[q] = fmaxf(v[q], 0.0f);
                    }
                } else if (row_ok) {
#pragma unroll
                    for (int q = 0; q < 32; ++q)
                        if (nb + q < p.N) v[q] = tc_apply_epi(p.epi, v[q], m, nb + q, p.N);
                }
                if (p.epi.sign_bits && row_ok && !post) p.epi.sign_bits[(p.epi.row0 + m) * p.epi.ld_sign_bits + (nb >> 5)] = sign_word(v, nb, p.N);
                if (p.C_lp && row_ok && !post) {
                    const int64_t left = p.N - nb, here = p.bn - c0;
                    const int valid = (int)(left < here ? left : here);
                    store_lp_row(p.C_lp + m * p.ldc_lp + nb, v, valid);
                }
                if (tma_store) {
                    // rows of 128 bytes in the 128-byte swizzle the tensor map expects: 16-byte chunk q of row r
                    // lives at chunk position q ^ (r & 7).  The box is clipped to the matrix by the TMA unit.
                    uint8_t* const box = box_base + (nboxes == 2 ? (box_turn & 1u) * 4096 : 0);
                    ++box_turn;
                    if (lane == 0) {                             // the store that last used this box has read it
                        if (nboxes == 2) bulk_wait_read<1>(); else bulk_wait_read<0>();
                    }
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<float4*>(box + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                            make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                    if (post) {
                        __syncwarp();
#pragma unroll
                        for (int it = 0; it < 8; ++it) {
                            const int rr = it * 4 + (lane >> 3), ch = lane & 7;
                            const uint32_t gw_rr = __shfl_sync(0xFFFFFFFFu, __float_as_uint(g4[0].x), rr);   // every lane takes part (before any lane skips)
                            const int64_t mr = m0 + quarter * 32 + rr;
                            const int nc = nb + ch * 4;
                            if (mr >= p.M || nc >= p.N || c0 + ch * 4 >= p.bn) continue;
                            float4* cell = reinterpret_cast<float4*>(box + rr * 128 + ((ch ^ (rr & 7)) << 4));
                            const float4 y4 = *cell;
                            float y[4] = {y4.x, y4.y, y4.z, y4.w};
                            const int nv = p.N - nc < 4 ? (int)(p.N - nc) : 4;
                            if (p.epi.drop) {
                                const uint8_t* dm = p.epi.drop + (p.epi.row0 + mr) * p.N + nc;
#pragma unroll
                                for (int t = 0; t < 4; ++t) if (t < nv) y[t] = dm[t] ? y[t] * p.epi.keep_scale : 0.0f;
                            }
                            if (p.epi.gate_bits) {
                                const uint32_t nib = (gw_rr >> (ch * 4)) & 0xFu;
#pragma unroll
                                for (int t = 0; t < 4; ++t) y[t] = ((nib >> t) & 1u) ? y[t] * p.epi.gate_scale : 0.0f;
                            } else if (p.epi.gate) {
                                const float* gp = p.epi.gate + (p.epi.row0 + mr) * p.epi.ld_gate + nc;
                                float gq[4] = {0.f, 0.f, 0.f, 0.f};
                                if (gate_vec) {       // the whole group lies inside the row's allocation (ld_gate % 4 == 0)
                                    gq[0] = g4[it].x; gq[1] = g4[it].y; gq[2] = g4[it].z; gq[3] = g4[it].w;
                                } else {
#pragma unroll
                                    for (int t = 0; t < 4; ++t) if (t < nv) gq[t] = __ldg(gp + t);
                                }
#pragma unroll
                                for (int t = 0; t < 4; ++t) y[t] = gq[t] > 0.0f ? y[t] * p.epi.gate_scale : 0.0f;
                            }
                            *cell = make_float4(y[0], y[1], y[2], y[3]);
                            if (p.C_lp) {
                                uint16_t* dl = p.C_lp + mr * p.ldc_lp + nc;
                                if (nv == 4) *reinterpret_cast<uint2*>(dl) = make_uint2(pack_bf16(y[0], y[1]), pack_bf16(y[2], y[3]));
                                else {
#pragma unroll
                                    for (int t = 0; t < 4; ++t) if (t < nv) dl[t] = (uint16_t)(pack_bf16(y[t], 0.0f) & 0xFFFFu);
                                }
                            }
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&map_c, box, nb, (int32_t)(m0 + quarter * 32));
                        bulk_commit();
                    }
                } else if (row_ok) {
                    float* dst = p.C + m * p.ldc + nb;
                    if (p.vec_c && nb + 31 < p.N && c0 + 31 < p.bn) {
#pragma unroll
                        for (int q = 0; q < 32; q += 4)
                            *reinterpret_cast<float4*>(dst + q) = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
                    } else {
#pragma unroll
                        for (int q = 0; q < 32; ++q)
                            if (nb + q < p.N && c0 + q < p.bn) dst[q] = v[q];
                    }
                }
            }
            // this warp is done reading the buffer: hand it back to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
        if (tma_store && lane == 0) bulk_wait_all();   // this warp's stores have completed before the CTA retires
    }
    if (threadIdx.x == 0 && abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == KK_EPI_WARPS + 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// The same persistent K-major product on PAIRS of CTAs (a thread-block cluster of two, tcgen05
// .cta_group::2): a pair owns a 256 x 256 output tile.  Each CTA loads its own 128 rows of A and its own
// half (128 rows) of the packed B tile per stage -- 32 KB per CTA instead of the 48 KB a lone CTA needs
// for a 128 x 256 tile, which is what the L2-to-shared-memory path and the operand reads from shared
// memory were short of -- and the pair's leader (even cluster rank) issues one M = 256 instruction that
// both SMs' tensor cores execute, each accumulating its 128 rows in its own tensor memory.
//  * full[s] lives in the leader: its producer arms it with the bytes of BOTH CTAs' loads, and the
//    peer's TMA loads report their bytes to it as well.
//  * empty[s] and acc_full[b] exist in both CTAs and are signalled together by a commit that arrives on
//    the barrier at the same offset in each CTA.
//  * acc_empty[b] lives in the leader and counts the epilogue warps of both CTAs (the peer's arrive
//    remotely).
// The CTAs of a pair meet at a cluster barrier after the barriers are initialised and before tensor memory
// is freed, so neither can exit while the other's loads, MMAs or arrivals still refer to it.
constexpr int PAIR_BM = 256, PAIR_BN = 256;

template <int KIND>
__global__ void __launch_bounds__(KK_THREADS, 1) gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                     const __grid_constant__ CUtensorMap map_b,
                                                                     const __grid_constant__ CUtensorMap map_c,
                                                                     const TcParams p, const int tma_store) {
    using Cfg = KindCfg<KIND>;
    constexpr int BK = Cfg::BK;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[8], empty_bar[8], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();              // 0 = leader of the pair
    const bool leader = rank == 0;
    constexpr uint32_t a_bytes = TC_BM * 128, b_bytes = (PAIR_BN / 2) * 128;
    constexpr uint32_t stage_bytes = a_bytes + b_bytes;   // per CTA
    const int nk = (int)((p.K + BK - 1) / BK);
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_ring = smem;
    uint8_t* smem_out = smem_ring + (size_t)p.stages * stage_bytes;

    const int64_t tiles = p.m_tiles * p.n_tiles;          // 256 x 256 tiles
    constexpr uint32_t acc_stride = PAIR_BN, tmem_cols = 2 * PAIR_BN;
    // the bias is read from global memory (every lane the same 128 bytes: a broadcast the L1 serves), which
    // leaves the shared memory a copy of it would take to a sixth stage of the ring
    const bool bias_vec = p.epi.bias != nullptr && aligned16_dev(p.epi.bias);

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 2 * KK_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == KK_EPI_WARPS + 1) {
        // the same warp of each CTA of the pair allocates, to the same shared-memory word
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_holder)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                   // both CTAs' barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;
    const uint32_t n_clusters = num_clusters_x(), cluster = cluster_id_x();

    if (warp == KK_EPI_WARPS) {
        if (lane == 0) {
            // ---------------- TMA producer (both CTAs) ----------------
            bool ok = true;
            uint32_t it = 0;
            for (int64_t tile = cluster; tile < tiles && ok; tile += n_clusters) {
                const int32_t m0 = (int32_t)((tile / p.n_tiles) * PAIR_BM + rank * TC_BM);
                const int32_t n0 = (int32_t)((tile % p.n_tiles) * PAIR_BN + rank * (PAIR_BN / 2));
                for (int ks = 0; ks < nk; ++ks, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = ((it / p.stages) & 1) ^ 1;
                    if (!mbar_wait(&empty_bar[s], ph, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; break; }
                    uint8_t* sa = smem_ring + (size_t)s * stage_bytes;
                    const uint32_t lead_full = mapa_shared(smem_u32(&full_bar[s]), 0);
                    if (leader) mbar_expect_tx(&full_bar[s], 2 * stage_bytes);
                    tma_load_2d_pair(sa, &map_a, ks * BK, m0, lead_full);
                    tma_load_2d_pair(sa + a_bytes, &map_b, ks * BK, n0, lead_full);
                }
            }
        }
    } else if (warp == KK_EPI_WARPS + 1) {
        if (lane == 0 && leader) {
            // ---------------- MMA issuer (leader only) ----------------
            const uint32_t idesc = make_idesc<KIND>(PAIR_BM, PAIR_BN, false);
            bool ok = true;
            uint32_t it = 0, j = 0;
            for (int64_t tile = cluster; tile < tiles && ok; tile += n_clusters, ++j) {
                const uint32_t buf = j & 1;
                if (!mbar_wait(&acc_empty[buf], ((j >> 1) & 1) ^ 1, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * acc_stride;
                for (int ks = 0; ks < nk; ++ks, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (it / p.stages) & 1;
                    if (!mbar_wait(&full_bar[s], ph, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem_ring + (size_t)s * stage_bytes), sb = sa + a_bytes;
#pragma unroll
                    for (int kq = 0; kq < BK / Cfg::MMA_K; ++kq)
                        tc_mma_pair<KIND>(d_tmem, make_desc(sa + kq * 32, 16, 1024, 2), make_desc(sb + kq * 32, 16, 1024, 2), idesc,
                                          (ks | kq) != 0 ? 1u : 0u);
                    tc_commit_pair(&empty_bar[s], 3);
                }
                if (ok) tc_commit_pair(&acc_full[buf], 3);
            }
        }
    } else {
        // ---------------- epilogue (both CTAs): this CTA's 128 rows of the tile ----------------
        const int quarter = warp & 3, half = warp >> 2;
        const bool has_gate = p.epi.gate != nullptr || p.epi.gate_bits != nullptr;
        const bool post = (p.epi.drop != nullptr || has_gate) && tma_store;
        const bool generic = !post && (p.epi.drop != nullptr || has_gate);
        const bool add_bias = p.epi.bias != nullptr, relu = p.epi.relu != 0;
        const bool gate_vec = p.epi.gate != nullptr && aligned16_dev(p.epi.gate) && (p.epi.ld_gate & 3) == 0;
        uint8_t* box = smem_out + (size_t)warp * 4096;
        uint32_t j = 0;
        bool ok = true;
        for (int64_t tile = cluster; tile < tiles && ok; tile += n_clusters, ++j) {
            const uint32_t buf = j & 1;
            const int64_t m0 = (tile / p.n_tiles) * PAIR_BM + rank * TC_BM;
            const int n0 = (int)((tile % p.n_tiles) * PAIR_BN);
            if (lane == 0) ok = mbar_wait(&acc_full[buf], (j >> 1) & 1, &abort_flag, p.wait_limit);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) { if (lane == 0) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); } break; }
            tc_fence_after();
            const int64_t m = m0 + quarter * 32 + lane;
            const bool row_ok = m < p.M;
            for (int c0 = half * 32; c0 < PAIR_BN; c0 += 64) {
                const int nb = n0 + c0;
                if (nb >= p.N) break;                     // columns beyond N: nothing to store (warp-uniform)
                float4 g4[8];
                if (post && p.epi.gate_bits) {
                    // bit-packed gate: this lane's row, the chunk's word (kept in the first slot of the fp32 gate's registers:
                    // the two forms exclude each other)
                    g4[0].x = __uint_as_float(row_ok ? __ldg(p.epi.gate_bits + (p.epi.row0 + m) * p.epi.ld_gate_bits + (nb >> 5)) : 0u);
                } else if (post && gate_vec) {
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int64_t mr = m0 + quarter * 32 + it * 4 + (lane >> 3);
                        const int nc = nb + (lane & 7) * 4;
                        g4[it] = (mr < p.M && nc < p.N) ? __ldg(reinterpret_cast<const float4*>(p.epi.gate + (p.epi.row0 + mr) * p.epi.ld_gate + nc))
                                                         : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                uint32_t r[32];
                tc_ld32(tmem_base + buf * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
                tc_wait_ld();
                float v[32];
#pragma unroll
                for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(r[q]);
                if (!generic) {
                    if (add_bias) {
                        if (bias_vec && nb + 31 < p.N) {
                            const float4* gb4 = reinterpret_cast<const float4*>(p.epi.bias + nb);
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const float4 b4 = __ldg(gb4 + q);
                                v[4 * q] += b4.x; v[4 * q + 1] += b4.y; v[4 * q + 2] += b4.z; v[4 * q + 3] += b4.w;
                            }
                        } else {
#pragma unroll
                            for (int q = 0; q < 32; ++q)
                                if (nb + q < p.N) v[q] += __ldg(p.epi.bias + nb + q);
                        }
                    }
                    if (relu) {
#pragma unroll
                        for (int q = 0; q < 32; ++q) v[q] = fmaxf(v[q], 0.0f);
                    }
                } else if (row_ok) {
#pragma unroll
                    for (int q = 0; q < 32; ++q)
                        if (nb + q < p.N) v[q] = tc_apply_epi(p.epi, v[q], m, nb + q, p.N);
                }
                if (p.epi.sign_bits && row_ok && !post) p.epi.sign_bits[(p.epi.row0 + m) * p.epi.ld_sign_bits + (nb >> 5)] = sign_word(v, nb, p.N);
                if (p.C_lp && row_ok && !post) {
                    const int64_t left = p.N - nb;
                    store_lp_row(p.C_lp + m * p.ldc_lp + nb, v, (int)(left < 32 ? left : 32));
                }
                if (tma_store) {
                    if (lane == 0) bulk_wait_read<0>();
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<float4*>(box + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                            make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                    if (post) {
                        __syncwarp();
#pragma unroll
                        for (int it = 0; it < 8; ++it) {
                            const int rr = it * 4 + (lane >> 3), ch = lane & 7;
                            const uint32_t gw_rr = __shfl_sync(0xFFFFFFFFu, __float_as_uint(g4[0].x), rr);   // every lane takes part (before any lane skips)
                            const int64_t mr = m0 + quarter * 32 + rr;
                            const int nc = nb + ch * 4;
                            if (mr >= p.M || nc >= p.N) continue;
                            float4* cell = reinterpret_cast<float4*>(box + rr * 128 + ((ch ^ (rr & 7)) << 4));
                            const float4 y4 = *cell;
                            float y[4] = {y4.x, y4.y, y4.z, y4.w};
                            const int nv = p.N - nc < 4 ? (int)(p.N - nc) : 4;
                            if (p.epi.drop) {
                                const uint8_t* dm = p.epi.drop + (p.epi.row0 + mr) * p.N + nc;
#pragma unroll
                                for (int t = 0; t < 4; ++t) if (t < nv) y[t] = dm[t] ? y[t] * p.epi.keep_scale : 0.0f;
                            }
                            if (p.epi.gate_bits) {
                                const uint32_t nib = (gw_rr >> (ch * 4)) & 0xFu;
#pragma unroll
                                for (int t = 0; t < 4; ++t) y[t] = ((nib >> t) & 1u) ? y[t] * p.epi.gate_scale : 0.0f;
                            } else if (p.epi.gate) {
                                const float* gp = p.epi.gate + (p.epi.row0 + mr) * p.epi.ld_gate + nc;
                                float gq[4] = {0.f, 0.f, 0.f, 0.f};
                                if (gate_vec) {
                                    gq[0] = g4[it].x; gq[1] = g4[it].y; gq[2] = g4[it].z; gq[3] = g4[it].w;
                                } else {
#pragma unroll
                                    for (int t = 0; t < 4; ++t) if (t < nv) gq[t] = __ldg(gp + t);
                                }
#pragma unroll
                                for (int t = 0; t < 4; ++t) y[t] = gq[t] > 0.0f ? y[t] * p.epi.gate_scale : 0.0f;
                            }
                            *cell = make_float4(y[0], y[1], y[2], y[3]);
                            if (p.C_lp) {
                                uint16_t* dl = p.C_lp + mr * p.ldc_lp + nc;
                                if (nv == 4) *reinterpret_cast<uint2*>(dl) = make_uint2(pack_bf16(y[0], y[1]), pack_bf16(y[2], y[3]));
                                else {
#pragma unroll
                                    for (int t = 0; t < 4; ++t) if (t < nv) dl[t] = (uint16_t)(pack_bf16(y[t], 0.0f) & 0xFFFFu);
                                }
                            }
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&map_c, box, nb, (int32_t)(m0 + quarter * 32));
                        bulk_commit();
                    }
                } else if (row_ok) {
                    float* dst = p.C + m * p.ldc + nb;
                    if (p.vec_c && nb + 31 < p.N) {
#pragma unroll
                        for (int q = 0; q < 32; q += 4)
                            *reinterpret_cast<float4*>(dst + q) = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
                    } else {
#pragma unroll
                        for (int q = 0; q < 32; ++q)
                            if (nb + q < p.N) dst[q] = v[q];
                    }
                }
            }
            // this warp is done reading the buffer: tell the leader's MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&acc_empty[buf]), 0));
        }
        if (tma_store && lane == 0) bulk_wait_all();
    }
    if (threadIdx.x == 0 && abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                   // the peer is done with this CTA's shared and tensor memory
    if (warp == KK_EPI_WARPS + 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// The weight-gradient form (both operands MN-major, K = node count split over the grid's z dimension) on
// CTA pairs: a pair owns a 256 x 256 tile of one K split; each CTA loads its 128 columns of A and of B per
// stage and writes its 128 rows of the (partial) tile.  Barriers as in gemm_tc_pair_kernel.
template <int KIND>
__global__ void __launch_bounds__(TC_THREADS, 1) gemm_tc_mm_pair_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                        const __grid_constant__ CUtensorMap map_b,
                                                                        const TcParams p) {
    using Cfg = KindCfg<KIND>;
    constexpr int BK = Cfg::BK;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[8], empty_bar[8], acc_bar;
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    constexpr uint32_t a_bytes = TC_BM * 128, b_bytes = (PAIR_BN / 2) * 128;
    constexpr uint32_t stage_bytes = a_bytes + b_bytes;
    constexpr int CHUNKS = TC_BM / Cfg::CHUNK;            // 128-byte-wide chunks per 128 columns of A or B
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    const int64_t tile = cluster_id_x();
    const int64_t m0 = (tile / p.n_tiles) * PAIR_BM + rank * TC_BM;
    const int64_t n0 = (tile % p.n_tiles) * PAIR_BN;
    const int64_t kb = (int64_t)blockIdx.z * p.k_per_split;
    const int64_t ke = kb + p.k_per_split < p.K ? kb + p.k_per_split : p.K;
    const int nk = (int)((ke - kb + BK - 1) / BK);
    constexpr uint32_t tmem_cols = PAIR_BN;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&acc_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_holder)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;

    if (warp == 4) {
        if (lane == 0) {
            // ---------------- TMA producer (both CTAs) ----------------
            for (int ks = 0; ks < nk; ++ks) {
                const int s = ks % p.stages;
                const uint32_t ph = ((ks / p.stages) & 1) ^ 1;
                if (!mbar_wait(&empty_bar[s], ph, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); break; }
                uint8_t* sa = smem + (size_t)s * stage_bytes;
                uint8_t* sb = sa + a_bytes;
                const uint32_t lead_full = mapa_shared(smem_u32(&full_bar[s]), 0);
                if (leader) mbar_expect_tx(&full_bar[s], 2 * stage_bytes);
                const int32_t k0 = (int32_t)(kb + (int64_t)ks * BK);
                for (int c = 0; c < CHUNKS; ++c)
                    tma_load_2d_pair(sa + c * Cfg::MN_CHUNK_BYTES, &map_a, (int32_t)(m0 + Cfg::CHUNK * c), k0, lead_full);
                for (int c = 0; c < CHUNKS; ++c)
                    tma_load_2d_pair(sb + c * Cfg::MN_CHUNK_BYTES, &map_b, (int32_t)(n0 + rank * (PAIR_BN / 2) + Cfg::CHUNK * c), k0, lead_full);
            }
        }
    } else if (warp == 5) {
        if (lane == 0 && leader) {
            // ---------------- MMA issuer (leader only) ----------------
            const uint32_t idesc = make_idesc<KIND>(PAIR_BM, PAIR_BN, true);
            bool ok = true;
            for (int ks = 0; ks < nk && ok; ++ks) {
                const int s = ks % p.stages;
                const uint32_t ph = (ks / p.stages) & 1;
                if (!mbar_wait(&full_bar[s], ph, &abort_flag, p.wait_limit)) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); ok = false; break; }
                tc_fence_after();
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes), sb = sa + a_bytes;
#pragma unroll
                for (int kq = 0; kq < BK / Cfg::MMA_K; ++kq)
                    tc_mma_pair<KIND>(tmem_base, make_desc(sa + kq * Cfg::MN_STEP, Cfg::MN_CHUNK_BYTES, Cfg::MN_SBO, Cfg::MN_LAYOUT),
                                      make_desc(sb + kq * Cfg::MN_STEP, Cfg::MN_CHUNK_BYTES, Cfg::MN_SBO, Cfg::MN_LAYOUT), idesc,
                                      (ks | kq) != 0 ? 1u : 0u);
                tc_commit_pair(&empty_bar[s], 3);
            }
            if (ok) tc_commit_pair(&acc_bar, 3);
        }
    } else {
        // ---------------- epilogue: this CTA's 128 rows ----------------
        bool ok = true;
        if (nk > 0) {
            if (lane == 0) ok = mbar_wait(&acc_bar, 0, &abort_flag, p.wait_limit);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok && lane == 0) { abort_flag = 1; atomicMax(p.status, DEV_WAIT_EXPIRED); }
        }
        __syncwarp();
        tc_fence_after();
        if (ok) {
            const int64_t m = m0 + warp * 32 + lane;
            float* Cb = p.C + (p.raw ? (int64_t)blockIdx.z * p.M * p.N : 0);
            for (int c0 = 0; c0 < PAIR_BN; c0 += 32) {
                const int64_t nb = n0 + c0;
                if (nb >= p.N) break;
                uint32_t r[32];
                if (nk > 0) {
                    tc_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, r);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                if (m < p.M) {
                    float* dst = Cb + m * p.ldc + nb;
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        v[j] = __uint_as_float(r[j]);
                        if (!p.raw && nb + j < p.N) v[j] = tc_apply_epi(p.epi, v[j], m, nb + j, p.N);
                    }
                    if (p.vec_c && nb + 31 < p.N) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (nb + j < p.N) dst[j] = v[j];
                    }
                }
            }
        }
    }
    if (threadIdx.x == 0 && abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// dst[n][k] = trans ? src[k][n] : src[n][k] for n < N, k < K, zero elsewhere; dst is rows x kpad of
// fp32 (TF32 kind) or bf16 (round to nearest even).
template <int KIND>
__global__ void pack_b_kernel(const float* __restrict__ src, int64_t ld, int trans, int N, int K, int rows, int kpad,
                              void* __restrict__ dst) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)rows * kpad) return;
    const int n = (int)(i / kpad), k = (int)(i % kpad);
    float v = 0.0f;
    if (n < N && k < K) v = trans ? src[(int64_t)k * ld + n] : src[(int64_t)n * ld + k];
    if (KIND == KIND_TF32) reinterpret_cast<float*>(dst)[i] = v;
    else reinterpret_cast<uint16_t*>(dst)[i] = (uint16_t)(pack_bf16(v, 0.0f) & 0xFFFFu);
}

// out[n] = sum over splits (ascending) of part[z][n]
__global__ void colsum_splits_kernel(int64_t N, int splits, const double* __restrict__ part, float* __restrict__ out) {
    const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    double sacc = 0.0;
    for (int z = 0; z < splits; ++z) sacc += part[(int64_t)z * N + n];
    out[n] = (float)sacc;
}

// dst[r][c] = bf16(src[r][c]) for c < d (round to nearest even); four columns per thread.
__global__ void to_bf16_kernel(int64_t rows, int d4, const float* __restrict__ src, int64_t ld_src, int d,
                               uint16_t* __restrict__ dst, int64_t ld_dst) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows * d4) return;
    const int64_t r = t / d4; const int c = (int)(t % d4) * 4;
    const float4 v = __ldg(reinterpret_cast<const float4*>(src + r * ld_src + c));
    uint16_t* o = dst + r * ld_dst + c;
    if (c + 3 < d) {
        *reinterpret_cast<uint2*>(o) = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
    } else {
        const float f[4] = {v.x, v.y, v.z, v.w};
        for (int q = 0; q < 4; ++q) if (c + q < d) o[q] = (uint16_t)(pack_bf16(f[q], 0.0f) & 0xFFFFu);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// 2-D tensor of fp32 (eb = 4) or bf16 (eb = 2): `inner` contiguous elements per row, `outer` rows of `ld`
// elements; 128-byte swizzle unless stated.
bool encode_2d(CUtensorMap* map, const void* base, int eb, int64_t inner, int64_t outer, int64_t ld, int box_inner,
               int box_outer, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    EncodeTiledFn fn = get_encode();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)ld * (cuuint64_t)eb};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, eb == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
              dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int pick_bn(int64_t N) {
    int64_t bn = (N + 15) / 16 * 16;
    if (bn > 256) {
        // split N evenly into tiles that are multiples of 32 and <= 256
        int64_t tiles = (N + 255) / 256;
        bn = ((N + tiles - 1) / tiles + 31) / 32 * 32;
    }
    return (int)bn;
}

// Number of K splits for `tiles` output tiles on a machine that runs `slots` CTAs (or CTA pairs) at a
// time: the split count, up to max_splits, whose tiles * splits units fill whole waves of `slots` best
// (a last wave that is one sixth full costs a third of the time of a two-wave launch).
int pick_splits(int64_t tiles, int64_t slots, int64_t max_splits) {
    int64_t hi = 4 * slots / tiles + 1;
    if (hi > max_splits) hi = max_splits;
    if (hi < 1) hi = 1;
    int best = (int)hi;
    double best_eff = 0.0;
    for (int64_t sp = 1; sp <= hi; ++sp) {
        const int64_t units = tiles * sp, waves = (units + slots - 1) / slots;
        if (units < slots && sp < hi) continue;                 // does not fill the machine once
        const double eff = (double)units / (double)(waves * slots);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = (int)sp; }
    }
    return best;
}

template <int KIND>
mixgcn_status launch_kind(mixgcn_ctx* ctx, int ta, int tb, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                          const void* B, int64_t ldb, float* C, int64_t ldc, const mixgcn_epilogue* epi, int64_t epi_row0,
                          cudaStream_t s, uint16_t* C_lp, int64_t ldc_lp, float* colsum_b, bool* colsum_done, const LossFuse* loss,
                          bool* bits_done) {
    using Cfg = KindCfg<KIND>;
    constexpr int EB = Cfg::EB, BK = Cfg::BK;
    // the loss epilogue exists in the single-CTA K-major kernel for one n-tile and a bias-only epilogue
    if (loss && (ta || N > 256 || C_lp || ctx->debug_drop_load || (epi && (epi->relu || epi->drop_mask || epi->gate || epi->gate_bits || epi->sign_bits)))) return MIXGCN_EUNSUPPORTED;
    if (ta && epi && (epi->gate_bits || epi->sign_bits)) return MIXGCN_EUNSUPPORTED;      // bit-packed masks: K-major products only
    constexpr int64_t LD_ALIGN = 16 / EB;           // TMA strides are multiples of 16 bytes
    if (M <= 0 || N <= 0 || K <= 0) return MIXGCN_EUNSUPPORTED;
    if (ta && tb) return MIXGCN_EUNSUPPORTED;
    if (!aligned16(A) || (lda % LD_ALIGN)) return MIXGCN_EUNSUPPORTED;
    if (ta && (!aligned16(B) || (ldb % LD_ALIGN))) return MIXGCN_EUNSUPPORTED;
    if (M >= (1ll << 31) || N >= (1ll << 31) || K >= (1ll << 31)) return MIXGCN_EUNSUPPORTED;
    if (C_lp && (ta || !aligned16(C_lp) || (ldc_lp & 7) || ldc_lp < N)) return MIXGCN_EUNSUPPORTED;
    if (!get_encode()) return MIXGCN_EUNSUPPORTED;

    TcParams p{};
    p.M = M; p.N = N; p.K = K;
    p.bn = pick_bn(N);
    p.m_tiles = (M + TC_BM - 1) / TC_BM;
    p.n_tiles = (N + p.bn - 1) / p.bn;
    p.C = C; p.ldc = ldc; p.vec_c = aligned16(C) && (ldc & 3) == 0;
    p.C_lp = C_lp; p.ldc_lp = ldc_lp;
    p.status = ctx->d_status;
    p.wait_limit = ctx->debug_wait_limit > 0 ? (uint32_t)ctx->debug_wait_limit : WAIT_LIMIT_DEFAULT;
    if (epi) {
        p.epi.bias = epi->bias; p.epi.relu = epi->relu; p.epi.drop = epi->drop_mask; p.epi.keep_scale = epi->keep_scale;
        p.epi.gate = epi->gate_bits ? nullptr : epi->gate; p.epi.ld_gate = epi->ld_gate; p.epi.gate_scale = epi->gate_scale;
        p.epi.gate_bits = epi->gate_bits; p.epi.ld_gate_bits = epi->ld_gate_bits;
        p.epi.sign_bits = epi->sign_bits; p.epi.ld_sign_bits = epi->ld_sign_bits;
    }
    p.epi.row0 = epi_row0;
    const int64_t tiles = p.m_tiles * p.n_tiles;
    if (tiles > 0x7FFFFFFFll) return MIXGCN_EUNSUPPORTED;
    const int bn32 = (p.bn + 31) & ~31;
    CUtensorMap map_a, map_b;

    if (!ta) {
        // KK form: pack B as rows x kpad (K contiguous), rows = n_tiles * bn32
        const int kpad = (int)((K + BK - 1) / BK * BK);
        // Wide, deep products (the compute-bound ones) run on CTA pairs with 256 x 256 tiles.
        const bool want_pairs = N >= 512 && K >= 512 && M >= 4096 && !ctx->debug_drop_load && !ctx->no_cta_pairs;
        int rows = (int)(p.n_tiles * p.bn > bn32 ? p.n_tiles * p.bn : bn32);
        if (want_pairs) {
            const int rows_pairs = (int)((N + PAIR_BN - 1) / PAIR_BN * PAIR_BN);
            if (rows_pairs > rows) rows = rows_pairs;
        }
        MIXGCN_TRY(ensure_workspace(ctx, (int64_t)rows * kpad * EB));
        void* packed = ctx->workspace;
        if (!encode_2d(&map_a, A, EB, K, M, lda, BK, TC_BM)) return MIXGCN_EUNSUPPORTED;
        if (!encode_2d(&map_b, packed, EB, kpad, rows, kpad, BK, bn32)) return MIXGCN_EUNSUPPORTED;
        {
            LaunchScope scope(ctx, PH_GEMM, s);
            const int64_t total = (int64_t)rows * kpad;
            pack_b_kernel<KIND><<<(unsigned)((total + 255) / 256), 256, 0, s>>>(reinterpret_cast<const float*>(B), ldb, tb ? 0 : 1,
                                                                                 (int)N, (int)K, rows, kpad, packed);
        }
        p.splits = 1; p.k_per_split = K; p.raw = 0;
        p.debug_drop_load = ctx->debug_drop_load;
        if (want_pairs) {
            TcParams q = p;
            q.bn = PAIR_BN;
            q.m_tiles = (M + PAIR_BM - 1) / PAIR_BM;
            q.n_tiles = (N + PAIR_BN - 1) / PAIR_BN;
            const int rows2 = (int)(q.n_tiles * PAIR_BN);
            const size_t stage2 = TC_BM * 128 + (PAIR_BN / 2) * 128;
            q.stages = 6;
            const size_t smem2 = (size_t)q.stages * stage2 + 8 * 4096 + 1024;
            const int tma_store2 = q.vec_c ? 1 : 0;
            CUtensorMap map_b2, map_c2 = map_a;
            bool ok2 = rows2 <= rows && encode_2d(&map_b2, packed, EB, kpad, rows2, kpad, BK, PAIR_BN / 2);
            if (ok2 && tma_store2) ok2 = encode_2d(&map_c2, C, 4, N, M, ldc, 32, 32);
            if (ok2) {
                MIXGCN_CUDA(cudaFuncSetAttribute(gemm_tc_pair_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2));
                cudaLaunchConfig_t cfg = {};
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeClusterDimension;
                attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
                cfg.blockDim = dim3(KK_THREADS, 1, 1);
                cfg.dynamicSmemBytes = smem2;
                cfg.stream = s;
                cfg.attrs = attr; cfg.numAttrs = 1;
                cfg.gridDim = dim3((unsigned)(ctx->sm_count & ~1), 1, 1);
                int max_clusters = 0;
                if (cudaOccupancyMaxActiveClusters(&max_clusters, gemm_tc_pair_kernel<KIND>, &cfg) != cudaSuccess) { cudaGetLastError(); max_clusters = 0; }
                const int64_t tiles2 = q.m_tiles * q.n_tiles;
                int64_t clusters = max_clusters < tiles2 ? max_clusters : tiles2;
                if (clusters >= 1) {
                    cfg.gridDim = dim3((unsigned)(2 * clusters), 1, 1);
                    LaunchScope scope(ctx, PH_GEMM, s);
                    MIXGCN_CUDA(cudaLaunchKernelEx(&cfg, gemm_tc_pair_kernel<KIND>, map_a, map_b2, map_c2, q, tma_store2));
                    ctx->gemm_pair_launches++;
                    // the epilogue wrote the sign bitmap unless the per-element terms ran on the staged boxes
                    if (bits_done) *bits_done = q.epi.sign_bits && !(tma_store2 && (q.epi.drop || q.epi.gate || q.epi.gate_bits));
                    return MIXGCN_OK;
                }
            }
        }
        // keep the packed weights resident in shared memory when they are small and there is one n-tile
        const int nk = kpad / BK;
        const size_t b_all = (size_t)nk * bn32 * 128;
        const int b_resident = (p.n_tiles == 1 && b_all <= 96 * 1024) ? 1 : 0;
        const size_t stage = TC_BM * 128 + (b_resident ? 0 : (size_t)bn32 * 128);
        // short K (one or two stages per tile): the tensor core is idle most of the time and the epilogue is
        // the critical path -- it gets a second staging box per warp out of the ring's budget
        p.epi_boxes = nk <= 2 ? 2 : 1;
        const size_t box_bytes = (size_t)KK_EPI_WARPS * p.epi_boxes * 4096;
        const size_t budget = (b_resident ? 200 * 1024 - b_all : 192 * 1024) - box_bytes;
        int stages = (int)(budget / stage);
        if (stages > 8) stages = 8;
        if (stages < 2) stages = 2;
        p.stages = stages;
        const size_t smem_kk = (b_resident ? b_all : 0) + (size_t)stages * stage + box_bytes + 1024;
        const int tma_store = (p.vec_c && (!loss || loss->zero_rows)) ? 1 : 0;     // a loss that leaves the other rows alone writes train rows only
        CUtensorMap map_c = map_a;
        if (tma_store && !encode_2d(&map_c, C, 4, N, M, ldc, 32, 32)) return MIXGCN_EUNSUPPORTED;
        int64_t grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
        if (loss) {
            if (p.n_tiles != 1) return MIXGCN_EUNSUPPORTED;
            p.loss_mask = loss->train_mask; p.loss_pred = loss->pred; p.loss_zero_rows = loss->zero_rows;
            MIXGCN_CUDA(cudaFuncSetAttribute(gemm_tc_kk_kernel<KIND, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_kk));
            LaunchScope scope(ctx, PH_GEMM, s);
            gemm_tc_kk_kernel<KIND, true><<<dim3((unsigned)grid, 1, 1), KK_THREADS, smem_kk, s>>>(map_a, map_b, map_c, p, b_resident, tma_store);
            MIXGCN_CUDA(cudaGetLastError());
            return MIXGCN_OK;
        }
        MIXGCN_CUDA(cudaFuncSetAttribute(gemm_tc_kk_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_kk));
        LaunchScope scope(ctx, PH_GEMM, s);
        gemm_tc_kk_kernel<KIND><<<dim3((unsigned)grid, 1, 1), KK_THREADS, smem_kk, s>>>(map_a, map_b, map_c, p, b_resident, tma_store);
        MIXGCN_CUDA(cudaGetLastError());
        if (bits_done) *bits_done = p.epi.sign_bits && !(tma_store && (p.epi.drop || p.epi.gate || p.epi.gate_bits));
        return MIXGCN_OK;
    }

    // MM form (weight gradient): wide results (both widths >= 512) on CTA pairs with 256 x 256 tiles
    if (M >= 512 && N >= 512 && K >= 4096 && !ctx->no_cta_pairs) {
        TcParams q = p;
        q.bn = PAIR_BN;
        q.m_tiles = (M + PAIR_BM - 1) / PAIR_BM;
        q.n_tiles = (N + PAIR_BN - 1) / PAIR_BN;
        const int64_t tiles2 = q.m_tiles * q.n_tiles;
        const int pairs = ctx->sm_count / 2;
        int64_t sp = pick_splits(tiles2, pairs, (K + 4095) / 4096);
        int64_t kps2 = (K + sp - 1) / sp;
        kps2 = (kps2 + BK - 1) / BK * BK;
        sp = (K + kps2 - 1) / kps2;
        q.k_per_split = kps2; q.splits = (int)sp;
        q.stages = 6;
        const CUtensorMapSwizzle sw2 = KIND == KIND_TF32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B;
        bool ok2 = tiles2 <= 0x3FFFFFFF && encode_2d(&map_a, A, EB, M, K, lda, Cfg::CHUNK, BK, sw2) &&
                   encode_2d(&map_b, B, EB, N, K, ldb, Cfg::CHUNK, BK, sw2);
        if (ok2) {
            if (sp > 1) {
                MIXGCN_TRY(ensure_workspace(ctx, sp * M * N * (int64_t)sizeof(float)));
                q.C = reinterpret_cast<float*>(ctx->workspace); q.ldc = N; q.vec_c = (N & 3) == 0; q.raw = 1;
            } else {
                q.raw = 0;
            }
            const size_t smem2 = (size_t)q.stages * (TC_BM * 128 + (PAIR_BN / 2) * 128) + 1024;
            MIXGCN_CUDA(cudaFuncSetAttribute(gemm_tc_mm_pair_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2));
            cudaLaunchConfig_t cfg = {};
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.gridDim = dim3((unsigned)(2 * tiles2), 1, (unsigned)sp);
            cfg.blockDim = dim3(TC_THREADS, 1, 1);
            cfg.dynamicSmemBytes = smem2;
            cfg.stream = s;
            cfg.attrs = attr; cfg.numAttrs = 1;
            {
                LaunchScope scope(ctx, PH_GEMM, s);
                MIXGCN_CUDA(cudaLaunchKernelEx(&cfg, gemm_tc_mm_pair_kernel<KIND>, map_a, map_b, q));
            }
            ctx->gemm_pair_launches++;
            if (sp > 1) MIXGCN_TRY(launch_splitk_reduce(ctx, M, N, (int)sp, q.C, C, ldc, epi, s));
            return MIXGCN_OK;
        }
    }
    // split K over CTAs
    int splits = pick_splits(tiles, 2 * (int64_t)ctx->sm_count, (K + 2047) / 2048);      // two CTAs per SM
    if (splits > 2048) splits = 2048;
    int64_t kps = (K + splits - 1) / splits;
    kps = (kps + BK - 1) / BK * BK;
    splits = (int)((K + kps - 1) / kps);
    p.k_per_split = kps; p.splits = splits;
    const CUtensorMapSwizzle sw = KIND == KIND_TF32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B;
    if (!encode_2d(&map_a, A, EB, M, K, lda, Cfg::CHUNK, BK, sw)) return MIXGCN_EUNSUPPORTED;
    if (!encode_2d(&map_b, B, EB, N, K, ldb, Cfg::CHUNK, BK, sw)) return MIXGCN_EUNSUPPORTED;
    const int bn_pad = (p.bn + Cfg::CHUNK - 1) / Cfg::CHUNK * Cfg::CHUNK;
    const size_t stage_mm = (size_t)TC_BM * 128 + (size_t)bn_pad * 128;
    int stages_mm = (int)((96 * 1024) / stage_mm);      // aim at two CTAs per SM
    if (stages_mm < 2) stages_mm = 2;
    if (stages_mm > 6) stages_mm = 6;
    p.stages = stages_mm;
    const size_t smem = (size_t)stages_mm * stage_mm + 1024;
    // with fp32 words in shared memory (TF32 kind) the kernel also sums B's columns on request
    const bool fuse_colsum = KIND == KIND_TF32 && colsum_b != nullptr;
    const int64_t part_bytes = splits > 1 ? (((int64_t)splits * M * N * (int64_t)sizeof(float) + 255) & ~(int64_t)255) : 0;
    const int64_t cs_bytes = fuse_colsum ? (int64_t)splits * N * (int64_t)sizeof(double) : 0;
    if (part_bytes + cs_bytes > 0) MIXGCN_TRY(ensure_workspace(ctx, part_bytes + cs_bytes));
    if (splits > 1) {
        p.C = reinterpret_cast<float*>(ctx->workspace); p.ldc = N; p.vec_c = (N & 3) == 0; p.raw = 1;
    } else {
        p.raw = 0;
    }
    p.colsum_part = fuse_colsum ? reinterpret_cast<double*>(reinterpret_cast<char*>(ctx->workspace) + part_bytes) : nullptr;
    MIXGCN_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<KIND, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    {
        LaunchScope scope(ctx, PH_GEMM, s);
        gemm_tc_kernel<KIND, true><<<dim3((unsigned)tiles, 1, (unsigned)splits), TC_THREADS, smem, s>>>(map_a, map_b, p);
    }
    MIXGCN_CUDA(cudaGetLastError());
    if (splits > 1) MIXGCN_TRY(launch_splitk_reduce(ctx, M, N, splits, p.C, C, ldc, epi, s));
    if (fuse_colsum) {
        LaunchScope scope(ctx, PH_GEMM, s);
        colsum_splits_kernel<<<(unsigned)((N + 127) / 128), 128, 0, s>>>(N, splits, p.colsum_part, colsum_b);
        MIXGCN_CUDA(cudaGetLastError());
        if (colsum_done) *colsum_done = true;
    }
    return MIXGCN_OK;
}

}  // namespace

namespace mixgcn {

// Returns MIXGCN_EUNSUPPORTED (without touching anything) when this shape / alignment is not
// served by the tensor-core kernels; the caller then uses another kernel.
//   kind 0 (TF32): A, and B in the MM form, are fp32 (lda, ldb in fp32 elements, multiples of 4);
//   kind 1 (BF16): they are bf16 (lda, ldb in bf16 elements, multiples of 8).
// In the KK form B is always the fp32 weight matrix (packed and converted here).  C_lp (KK form only,
// nullable) receives a bf16 copy of C.  colsum_b (nullable; weight-gradient form): where the kernel taken
// can also produce the column sums of B (out[n] = sum_k B[k][n]) it does and sets *colsum_done; otherwise
// the caller computes them.
mixgcn_status launch_gemm_tc(mixgcn_ctx* ctx, int kind, int ta, int tb, int64_t M, int64_t N, int64_t K, const void* A,
                             int64_t lda, const void* B, int64_t ldb, float* C, int64_t ldc,
                             const mixgcn_epilogue* epi, int64_t epi_row0, cudaStream_t s, uint16_t* C_lp, int64_t ldc_lp,
                             float* colsum_b, bool* colsum_done, const LossFuse* loss, bool* bits_done) {
    if (colsum_done) *colsum_done = false;
    if (bits_done) *bits_done = false;
    if (kind == KIND_BF16)
        return launch_kind<KIND_BF16>(ctx, ta, tb, M, N, K, A, lda, B, ldb, C, ldc, epi, epi_row0, s, C_lp, ldc_lp, colsum_b, colsum_done, loss, bits_done);
    return launch_kind<KIND_TF32>(ctx, ta, tb, M, N, K, A, lda, B, ldb, C, ldc, epi, epi_row0, s, C_lp, ldc_lp, colsum_b, colsum_done, loss, bits_done);
}

// dst (rows x ld_dst bf16, ld_dst a multiple of 4) = bf16(src (rows x ld_src fp32, 16-byte aligned, ld_src % 4 == 0)), columns < d
mixgcn_status launch_to_bf16(mixgcn_ctx* ctx, int64_t rows, int32_t d, const float* src, int64_t ld_src, uint16_t* dst,
                             int64_t ld_dst, cudaStream_t s) {
    if (rows <= 0 || d <= 0) return MIXGCN_OK;
    const int d4 = (d + 3) / 4;
    LaunchScope scope(ctx, PH_ELEM, s);
    to_bf16_kernel<<<(unsigned)((rows * d4 + 255) / 256), 256, 0, s>>>(rows, d4, src, ld_src, d, dst, ld_dst);
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

}  // namespace mixgcn
