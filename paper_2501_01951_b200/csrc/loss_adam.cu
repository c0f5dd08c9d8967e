// Masked softmax cross-entropy with its gradient and arg-max (the loss line of Algorithm 2),
// and the Adam step (its weight-update line).  Both are streaming kernels; floating-point
// reductions run in a fixed order (per-warp shuffles, per-CTA partials, one final pass).
#include <stddef.h>

#include <atomic>

#include "internal.cuh"

using namespace mixgcn;

namespace {

constexpr int LOSS_WARPS = 8;

__global__ void count_mask_kernel(int64_t n, const uint8_t* __restrict__ mask, unsigned long long* count) {
    __shared__ unsigned int sm[8];
    unsigned int c = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        c += mask[i] ? 1u : 0u;
    for (int o = 16; o > 0; o >>= 1) c += __shfl_down_sync(0xFFFFFFFFu, c, o);
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int t = 0;
        for (int w = 0; w < 8; ++w) t += sm[w];
        if (t) atomicAdd(count, (unsigned long long)t);  // integer: order does not matter
    }
}

// One warp per row.  part[block] receives the block's sum of per-row losses.
__global__ void __launch_bounds__(LOSS_WARPS * 32) loss_rows_kernel(
    int64_t n, int C, const float* logits, int64_t ld, const int32_t* __restrict__ labels,
    const uint8_t* __restrict__ mask, const unsigned long long* __restrict__ count, float* dlogits,
    int32_t* __restrict__ pred, unsigned long long* n_correct, double* __restrict__ part, int32_t* status, bool zero_rows) {
    __shared__ double sm[LOSS_WARPS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long T = *count;
    const float invT = T ? (float)(1.0 / (double)T) : 0.0f;
    double local = 0.0;
    unsigned int correct = 0;
    const int64_t stride = (int64_t)gridDim.x * LOSS_WARPS;
    for (int64_t v = (int64_t)blockIdx.x * LOSS_WARPS + warp; v < n; v += stride) {
        const float* row = logits + v * ld;
        // arg-max with lowest-index ties
        float mx = -INFINITY; int arg = 0x7FFFFFFF;
        for (int c = lane; c < C; c += 32) {
            const float x = row[c];
            if (x > mx || (x == mx && c < arg)) { mx = x; arg = c; }
        }
        if (arg == 0x7FFFFFFF) arg = lane < C ? lane : 0;  // all -inf or NaN in this lane's columns
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float omx = __shfl_xor_sync(0xFFFFFFFFu, mx, o);
            const int oarg = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
            if (omx > mx || (omx == mx && oarg < arg)) { mx = omx; arg = oarg; }
        }
        if (pred && lane == 0) pred[v] = arg;
        const bool train = mask[v] != 0 && T != 0;
        int y = 0;
        bool ok = false;
        if (train) {
            y = labels[v];
            ok = y >= 0 && y < C;
            if (!ok && lane == 0) atomicMax(status, DEV_BAD_LABEL);
        }
        if (!train || !ok) {
            if (dlogits && (zero_rows || train)) for (int c = lane; c < C; c += 32) dlogits[v * ld + c] = 0.0f;
            continue;
        }
        float s = 0.0f;
        for (int c = lane; c < C; c += 32) s += expf(row[c] - mx);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        const float lse = mx + logf(s);
        const float py = row[y];
        if (lane == 0) { local += (double)(lse - py); if (arg == y) ++correct; }
        __syncwarp();  // dlogits may alias logits: every read of the row precedes the writes
        if (dlogits)
            for (int c = lane; c < C; c += 32) {
                const float g = (expf(row[c] - lse) - (c == y ? 1.0f : 0.0f)) * invT;
                dlogits[v * ld + c] = g;
            }
    }
    if (lane == 0) sm[warp] = local;
    if (n_correct && lane == 0 && correct) atomicAdd(n_correct, (unsigned long long)correct);
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < LOSS_WARPS; ++w) t += sm[w];
        part[blockIdx.x] = t;
    }
}

// Same computation for C <= 128 * VPL with the row held in registers: one float4-vectorised read of the
// logits, one float4 write of the gradient (requires ld % 4 == 0 and 16-byte aligned pointers).
template <int VPL>
__global__ void __launch_bounds__(LOSS_WARPS * 32) loss_rows_vec_kernel(
    int64_t n, int C, const float* logits, int64_t ld, const int32_t* __restrict__ labels,
    const uint8_t* __restrict__ mask, const unsigned long long* __restrict__ count, float* dlogits,
    int32_t* __restrict__ pred, unsigned long long* n_correct, double* __restrict__ part, int32_t* status, bool zero_rows) {
    __shared__ double sm[LOSS_WARPS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long T = *count;
    const float invT = T ? (float)(1.0 / (double)T) : 0.0f;
    const int C4 = (C + 3) >> 2;
    double local = 0.0;
    unsigned int correct = 0;
    const int64_t stride = (int64_t)gridDim.x * LOSS_WARPS;
    // the next row's loads are issued before the current row is reduced, so two rows per warp are in flight
    auto load_row = [&](int64_t v, float4 (&t)[VPL]) {
        const float4* row4 = reinterpret_cast<const float4*>(logits + v * ld);
#pragma unroll
        for (int q = 0; q < VPL; ++q) {
            const int g = lane + 32 * q;
            t[q] = (v < n && g < C4) ? row4[g] : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        }
    };
    float4 nxt[VPL];
    load_row((int64_t)blockIdx.x * LOSS_WARPS + warp, nxt);
    for (int64_t v = (int64_t)blockIdx.x * LOSS_WARPS + warp; v < n; v += stride) {
        float x[VPL][4];
#pragma unroll
        for (int q = 0; q < VPL; ++q) {
            const int g = lane + 32 * q;
            x[q][0] = nxt[q].x; x[q][1] = nxt[q].y; x[q][2] = nxt[q].z; x[q][3] = nxt[q].w;
#pragma unroll
            for (int e = 0; e < 4; ++e) if (g * 4 + e >= C) x[q][e] = -INFINITY;   // pad columns are not data
        }
        load_row(v + stride, nxt);
        float mx = -INFINITY; int arg = 0x7FFFFFFF;
#pragma unroll
        for (int q = 0; q < VPL; ++q)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = (lane + 32 * q) * 4 + e;
                if (c < C && (x[q][e] > mx || (x[q][e] == mx && c < arg))) { mx = x[q][e]; arg = c; }
            }
        if (arg == 0x7FFFFFFF) arg = lane * 4 < C ? lane * 4 : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float omx = __shfl_xor_sync(0xFFFFFFFFu, mx, o);
            const int oarg = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
            if (omx > mx || (omx == mx && oarg < arg)) { mx = omx; arg = oarg; }
        }
        if (pred && lane == 0) pred[v] = arg;
        const bool train = mask[v] != 0 && T != 0;
        int y = 0;
        bool ok = false;
        if (train) {
            y = labels[v];
            ok = y >= 0 && y < C;
            if (!ok && lane == 0) atomicMax(status, DEV_BAD_LABEL);
        }
        float4* out4 = dlogits ? reinterpret_cast<float4*>(dlogits + v * ld) : nullptr;
        if (!train || !ok) {
            if (out4 && (zero_rows || train)) {
#pragma unroll
                for (int q = 0; q < VPL; ++q) {
                    const int g = lane + 32 * q;
                    if (g < C4) out4[g] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            continue;
        }
        float s = 0.0f;
#pragma unroll
        for (int q = 0; q < VPL; ++q)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if ((lane + 32 * q) * 4 + e < C) s += expf(x[q][e] - mx);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        const float lse = mx + logf(s);
        // the label's logit lives in lane (y/4) % 32, slot (y/4) / 32, element y % 4
        float py = 0.0f;
#pragma unroll
        for (int q = 0; q < VPL; ++q)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if ((lane + 32 * q) * 4 + e == y) py = x[q][e];
        py = __shfl_sync(0xFFFFFFFFu, py, (y >> 2) & 31);
        if (lane == 0) { local += (double)(lse - py); if (arg == y) ++correct; }
        if (out4) {
#pragma unroll
            for (int q = 0; q < VPL; ++q) {
                const int g = lane + 32 * q;
                if (g < C4) {
                    float r[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = g * 4 + e;
                        r[e] = c < C ? (expf(x[q][e] - lse) - (c == y ? 1.0f : 0.0f)) * invT : 0.0f;
                    }
                    out4[g] = make_float4(r[0], r[1], r[2], r[3]);
                }
            }
        }
    }
    if (lane == 0) sm[warp] = local;
    if (n_correct && lane == 0 && correct) atomicAdd(n_correct, (unsigned long long)correct);
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < LOSS_WARPS; ++w) t += sm[w];
        part[blockIdx.x] = t;
    }
}

// Train rows only: a warp scans 32 mask bytes, then handles the train rows among them one by one.
// Rows outside the mask are neither read nor written (pred receives -1 there).
__global__ void __launch_bounds__(LOSS_WARPS * 32) loss_rows_subset_kernel(
    int64_t n, int C, const float* logits, int64_t ld, const int32_t* __restrict__ labels,
    const uint8_t* __restrict__ mask, const unsigned long long* __restrict__ count, float* dlogits,
    int32_t* __restrict__ pred, unsigned long long* n_correct, double* __restrict__ part, int32_t* status) {
    __shared__ double sm[LOSS_WARPS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long T = *count;
    const float invT = T ? (float)(1.0 / (double)T) : 0.0f;
    double local = 0.0;
    unsigned int correct = 0;
    const int64_t stride = (int64_t)gridDim.x * LOSS_WARPS * 32;
    for (int64_t v0 = ((int64_t)blockIdx.x * LOSS_WARPS + warp) * 32; v0 < n; v0 += stride) {
        const int64_t vl = v0 + lane;
        const bool mine = vl < n && mask[vl] != 0 && T != 0;
        if (pred && vl < n && !mine) pred[vl] = -1;
        unsigned live = __ballot_sync(0xFFFFFFFFu, mine);
        while (live) {
            const int64_t v = v0 + __ffs(live) - 1;
            live &= live - 1;
            const float* row = logits + v * ld;
            float mx = -INFINITY; int arg = 0x7FFFFFFF;
            for (int c = lane; c < C; c += 32) {
                const float x = row[c];
                if (x > mx || (x == mx && c < arg)) { mx = x; arg = c; }
            }
            if (arg == 0x7FFFFFFF) arg = lane < C ? lane : 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float omx = __shfl_xor_sync(0xFFFFFFFFu, mx, o);
                const int oarg = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
                if (omx > mx || (omx == mx && oarg < arg)) { mx = omx; arg = oarg; }
            }
            if (pred && lane == 0) pred[v] = arg;
            const int y = labels[v];
            if (y < 0 || y >= C) {
                if (lane == 0) atomicMax(status, DEV_BAD_LABEL);
                __syncwarp();
                if (dlogits) for (int c = lane; c < C; c += 32) dlogits[v * ld + c] = 0.0f;
                continue;
            }
            float s = 0.0f;
            for (int c = lane; c < C; c += 32) s += expf(row[c] - mx);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
            const float lse = mx + logf(s);
            const float py = row[y];
            if (lane == 0) { local += (double)(lse - py); if (arg == y) ++correct; }
            __syncwarp();  // dlogits may alias logits: every read of the row precedes the writes
            if (dlogits)
                for (int c = lane; c < C; c += 32) dlogits[v * ld + c] = (expf(row[c] - lse) - (c == y ? 1.0f : 0.0f)) * invT;
            __syncwarp();
        }
    }
    if (lane == 0) sm[warp] = local;
    if (n_correct && lane == 0 && correct) atomicAdd(n_correct, (unsigned long long)correct);
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < LOSS_WARPS; ++w) t += sm[w];
        part[blockIdx.x] = t;
    }
}

// ---- rows staged through shared memory, four lanes per row ------------------------------------
// For C up to a few hundred the warp-per-row kernels spend more issue slots on shuffles than on data.
// Here a CTA takes tiles of ROWS consecutive rows: a tile is one contiguous piece of memory
// (ROWS x ld floats), fetched by a single bulk-async copy into shared memory while the previous tile
// is being worked on (two buffers).  Four adjacent lanes own a row, a quarter of its columns each,
// walked from a lane-dependent starting point so that a warp's 32 lanes spread over the banks; the
// arg-max keeps the lowest index among equal maxima explicitly, so the order does not matter.  The few
// train rows are then finished by whole warps (exponentials and gradient stores over 32 lanes).
constexpr uint32_t LOSS_WAIT_LIMIT = 1u << 22;
constexpr int LOSS_TILE_KB = 72;     // shared memory a CTA of the tile kernel takes at most (two tile buffers)
constexpr int LOSS_LANES_PER_ROW = 4;

__device__ __forceinline__ uint32_t loss_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool loss_mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < LOSS_WAIT_LIMIT; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(loss_smem_u32(bar)), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

template <int ROWS>
__global__ void __launch_bounds__(ROWS * LOSS_LANES_PER_ROW) loss_rows_tile_kernel(
    int64_t n, int C, const float* logits, int64_t ld, const int32_t* __restrict__ labels,
    const uint8_t* __restrict__ mask, const unsigned long long* __restrict__ count, float* dlogits,
    int32_t* __restrict__ pred, unsigned long long* n_correct, double* __restrict__ part, int32_t* status,
    bool zero_rows, int64_t n_tiles) {
    constexpr int THREADS = ROWS * LOSS_LANES_PER_ROW;
    extern __shared__ __align__(128) unsigned char loss_smem[];
    float* const tile0 = reinterpret_cast<float*>(loss_smem);
    float* const tile1 = tile0 + (int64_t)ROWS * ld;
    __shared__ __align__(8) uint64_t bar[2];
    __shared__ double red[THREADS / 32];
    __shared__ uint8_t keep_row[2][ROWS];      // rows of the tile whose gradient row was written as a train row
    __shared__ int expired;
    const int tid = threadIdx.x, lane = tid & 31;
    const int r_own = tid / LOSS_LANES_PER_ROW, q = tid % LOSS_LANES_PER_ROW;
    const unsigned long long T = *count;
    const float invT = T ? (float)(1.0 / (double)T) : 0.0f;
    const int ld4 = (int)(ld >> 2);
    const int seg = (C + LOSS_LANES_PER_ROW - 1) / LOSS_LANES_PER_ROW;
    const int c_lo = q * seg < C ? q * seg : C, c_hi = (q + 1) * seg < C ? (q + 1) * seg : C;
    if (tid == 0) {
        expired = 0;
        for (int b = 0; b < 2; ++b)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(loss_smem_u32(&bar[b])), "r"(1u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    auto issue = [&](int64_t t, int b) {
        const int64_t row0 = t * ROWS;
        const int64_t rows = (n - row0) < ROWS ? (n - row0) : ROWS;
        const uint32_t bytes = (uint32_t)(rows * ld * (int64_t)sizeof(float));    // a multiple of 16: ld % 4 == 0
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(loss_smem_u32(&bar[b])), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(loss_smem_u32(b ? tile1 : tile0)), "l"(reinterpret_cast<uint64_t>(logits + row0 * ld)), "r"(bytes),
                       "r"(loss_smem_u32(&bar[b])) : "memory");
    };
    double local = 0.0;
    unsigned int correct = 0;
    uint32_t phase0 = 0u, phase1 = 0u;       // parity to wait for on each buffer's barrier
    int buf = 0;
    int64_t t = blockIdx.x;
    if (tid == 0 && t < n_tiles) issue(t, 0);                       // the first tile; later ones are requested one iteration ahead
    for (; t < n_tiles; t += gridDim.x, buf ^= 1) {
        const int64_t row0 = t * ROWS, v = row0 + r_own;
        // mask byte and label of this thread's row, requested before the wait so that their latency is hidden
        uint8_t my_mask = 0; int my_y = 0;
        if (v < n && q == 0) { my_mask = mask[v]; my_y = labels[v]; }
        if (!loss_mbar_wait(&bar[buf], buf ? phase1 : phase0)) expired = 1;       // bounded: give up instead of hanging
        if (buf) phase1 ^= 1u; else phase0 ^= 1u;
        __syncthreads();               // this tile has landed; every thread is done with the previous tile
        if (expired) {
            if (tid == 0) atomicMax(status, DEV_WAIT_EXPIRED);         // no other copy is in flight at this point
            break;
        }
        // refill the other buffer (the previous tile's) while this one is worked on
        if (tid == 0 && t + gridDim.x < n_tiles) issue(t + gridDim.x, buf ^ 1);
        const int rows = (int)((n - row0) < ROWS ? (n - row0) : ROWS);
        const float* tile = buf ? tile1 : tile0;
        const float* row = tile + (int64_t)r_own * ld;
        float mx = -INFINITY; int arg = 0x7FFFFFFF;
        if (v < n && c_hi > c_lo) {
            // two independent (max, index) chains over [start, c_hi) then [c_lo, start): plain counted
            // loops so that the shared-memory loads are issued ahead of the compares
            const int start = c_lo + lane % (c_hi - c_lo);
            float mx2 = -INFINITY; int arg2 = 0x7FFFFFFF;
            auto scan = [&](int c0, int c1) {
                int c = c0;
#pragma unroll 4
                for (; c + 1 < c1; c += 2) {
                    const float x = row[c], x2 = row[c + 1];
                    if (x > mx || (x == mx && c < arg)) { mx = x; arg = c; }
                    if (x2 > mx2 || (x2 == mx2 && c + 1 < arg2)) { mx2 = x2; arg2 = c + 1; }
                }
                if (c < c1) { const float x = row[c]; if (x > mx || (x == mx && c < arg)) { mx = x; arg = c; } }
            };
            scan(start, c_hi);
            scan(c_lo, start);
            if (mx2 > mx || (mx2 == mx && arg2 < arg)) { mx = mx2; arg = arg2; }
        }
        // the four lanes of a row agree on its maximum and the lowest index that attains it
#pragma unroll
        for (int o = 1; o < LOSS_LANES_PER_ROW; o <<= 1) {
            const float omx = __shfl_xor_sync(0xFFFFFFFFu, mx, o);
            const int oarg = __shfl_xor_sync(0xFFFFFFFFu, arg, o);
            if (omx > mx || (omx == mx && oarg < arg)) { mx = omx; arg = oarg; }
        }
        if (arg == 0x7FFFFFFF) arg = 0;                                // every entry NaN
        const bool wrote = v < n && q == 0 && my_mask != 0 && T != 0;
        if (v < n && q == 0 && pred) pred[v] = arg;
        if (dlogits && zero_rows) {
            if (q == 0) keep_row[buf][r_own] = wrote ? 1 : 0;
            __syncthreads();           // keep_row is complete
            // zero gradient rows of the other nodes, written by the whole CTA in memory order
            float4* out4 = reinterpret_cast<float4*>(dlogits + row0 * ld);
            const int total4 = rows * ld4;
            for (int i = tid; i < total4; i += THREADS) {
                const int r = i / ld4;
                if (!keep_row[buf][r]) out4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        // train rows (few): the whole warp works on each of them in turn -- lanes stride over the columns
        unsigned live = __ballot_sync(0xFFFFFFFFu, wrote);
        while (live) {
            const int src = __ffs(live) - 1;
            live &= live - 1;
            const float r_mx = __shfl_sync(0xFFFFFFFFu, mx, src);
            const int r_arg = __shfl_sync(0xFFFFFFFFu, arg, src);
            const int y = __shfl_sync(0xFFFFFFFFu, my_y, src);
            const int r = ((tid & ~31) + src) / LOSS_LANES_PER_ROW;
            const float* rr = tile + (int64_t)r * ld;
            float* out = dlogits ? dlogits + (row0 + r) * ld : nullptr;
            if (y < 0 || y >= C) {
                if (lane == 0) atomicMax(status, DEV_BAD_LABEL);
                if (out) for (int j = lane; j < C; j += 32) out[j] = 0.0f;
                continue;
            }
            float sum = 0.0f;
            for (int j = lane; j < C; j += 32) sum += expf(rr[j] - r_mx);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
            const float lse = r_mx + logf(sum);
            if (lane == 0) { local += (double)(lse - rr[y]); if (r_arg == y) ++correct; }
            if (out) for (int j = lane; j < C; j += 32) out[j] = (expf(rr[j] - lse) - (j == y ? 1.0f : 0.0f)) * invT;
        }
    }
    // fixed-order block sum of the per-warp losses
    for (int o = 16; o > 0; o >>= 1) local += __shfl_down_sync(0xFFFFFFFFu, local, o);
    for (int o = 16; o > 0; o >>= 1) correct += __shfl_down_sync(0xFFFFFFFFu, correct, o);
    if (lane == 0) red[tid >> 5] = local;
    if (n_correct && lane == 0 && correct) atomicAdd(n_correct, (unsigned long long)correct);
    __syncthreads();
    if (tid == 0) {
        double s = 0.0;
        for (int w = 0; w < THREADS / 32; ++w) s += red[w];
        part[blockIdx.x] = s;
    }
}

template <int ROWS>
cudaError_t launch_loss_tile(int grid, size_t smem, cudaStream_t s, int64_t n, int C, const float* logits, int64_t ld,
                             const int32_t* labels, const uint8_t* mask, const unsigned long long* count, float* dlogits,
                             int32_t* pred, unsigned long long* n_correct, double* part, int32_t* status, bool zero_rows,
                             int64_t n_tiles) {
    cudaError_t e = cudaFuncSetAttribute(loss_rows_tile_kernel<ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    loss_rows_tile_kernel<ROWS><<<grid, ROWS * LOSS_LANES_PER_ROW, smem, s>>>(n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part,
                                                         status, zero_rows, n_tiles);
    return cudaGetLastError();
}

// Launches the row pass and returns how many block partials it writes to `part` (<= warp_blocks, the
// capacity the caller sized `part` for), or -1 on a launch error.  With sm_count > 0 and a row that
// fits, the shared-memory tile kernel (one lane per row) is used; otherwise one warp per row, with
// the row in registers when C <= 256 and the layout allows float4 access.
int launch_loss_rows(unsigned warp_blocks, cudaStream_t s, int64_t n, int C, const float* logits, int64_t ld,
                     const int32_t* labels, const uint8_t* mask, const unsigned long long* count, float* dlogits,
                     int32_t* pred, unsigned long long* n_correct, double* part, int32_t* status, bool zero_rows = true,
                     int sm_count = 0) {
    const bool vec = (ld & 3) == 0 && aligned16(logits) && (!dlogits || aligned16(dlogits));
    // Several CTAs per SM (each with two tile buffers) keep some computing while others wait for their
    // copies: a CTA takes at most LOSS_TILE_KB of shared memory; rows per tile follow from that.
    constexpr int64_t TILE_SMEM = LOSS_TILE_KB * 1024;
    // The tile kernel treats a tile as one dense piece of rows x ld floats (it copies and zeroes whole
    // rows), so it is taken only when the row holds nothing but its C columns and their pad to a multiple
    // of 4; a wider ld (a column slice of a larger buffer) goes to the per-row kernels, which touch columns
    // below round4(C) only.
    if (vec && sm_count > 0 && C >= 8 && ld == ((int64_t)C + 3) / 4 * 4 && 2 * 32 * ld * 4 <= TILE_SMEM) {
        const int rows = 2 * 128 * ld * 4 <= TILE_SMEM ? 128 : (2 * 64 * ld * 4 <= TILE_SMEM ? 64 : 32);
        const int64_t n_tiles = (n + rows - 1) / rows;
        int64_t per_sm = (220 * 1024) / (2 * rows * ld * 4 + 1024);
        if (per_sm > 2048 / (rows * LOSS_LANES_PER_ROW)) per_sm = 2048 / (rows * LOSS_LANES_PER_ROW);
        if (per_sm < 1) per_sm = 1;
        int64_t grid = n_tiles < per_sm * sm_count ? n_tiles : per_sm * sm_count;
        if (grid > (int64_t)warp_blocks) grid = warp_blocks;
        const size_t smem = (size_t)(2 * rows * ld * 4);
        cudaError_t e = rows == 128 ? launch_loss_tile<128>((int)grid, smem, s, n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows, n_tiles)
                      : rows == 64  ? launch_loss_tile<64>((int)grid, smem, s, n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows, n_tiles)
                                    : launch_loss_tile<32>((int)grid, smem, s, n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows, n_tiles);
        return e == cudaSuccess ? (int)grid : -1;
    }
    if (vec && C <= 128)
        loss_rows_vec_kernel<1><<<warp_blocks, LOSS_WARPS * 32, 0, s>>>(n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows);
    else if (vec && C <= 256)
        loss_rows_vec_kernel<2><<<warp_blocks, LOSS_WARPS * 32, 0, s>>>(n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows);
    else
        loss_rows_kernel<<<warp_blocks, LOSS_WARPS * 32, 0, s>>>(n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows);
    return cudaGetLastError() == cudaSuccess ? (int)warp_blocks : -1;
}

__global__ void loss_final_kernel(int blocks, const double* __restrict__ part,
                                  const unsigned long long* __restrict__ count, float* loss, int32_t* status) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const unsigned long long T = *count;
    if (T == 0) { *loss = 0.0f; atomicMax(status, DEV_EMPTY_MASK); return; }
    double t = 0.0;
    for (int b = 0; b < blocks; ++b) t += part[b];
    *loss = (float)(t / (double)T);
}

// Final pass of the loss taken inside the aggregation: the per-row terms of the train rows are added in row
// order (block b owns rows [b * chunk, (b + 1) * chunk), its threads stride through them, fixed-order tree
// within the block, blocks added in order by loss_final_kernel), and the correct predictions are counted.
constexpr int FUSE_REDUCE_THREADS = 256;
__global__ void __launch_bounds__(FUSE_REDUCE_THREADS) loss_rows_reduce_kernel(
    int64_t n, int C, int64_t chunk, const uint8_t* __restrict__ mask, const int32_t* __restrict__ labels,
    const float* __restrict__ row_loss, const int32_t* __restrict__ pred, double* __restrict__ part,
    unsigned long long* n_correct) {
    __shared__ double sm[FUSE_REDUCE_THREADS];
    __shared__ unsigned int sc[FUSE_REDUCE_THREADS / 32];
    const int64_t r0 = (int64_t)blockIdx.x * chunk, r1 = r0 + chunk < n ? r0 + chunk : n;
    double local = 0.0;
    unsigned int correct = 0;
    for (int64_t v = r0 + threadIdx.x; v < r1; v += FUSE_REDUCE_THREADS) {
        if (!mask[v]) continue;
        const int y = labels[v];
        if (y < 0 || y >= C) continue;            // reported by the aggregation's epilogue; contributes nothing
        local += (double)row_loss[v];
        if (pred && pred[v] == y) ++correct;
    }
    sm[threadIdx.x] = local;
    for (int o = 16; o > 0; o >>= 1) correct += __shfl_down_sync(0xFFFFFFFFu, correct, o);
    if ((threadIdx.x & 31) == 0) sc[threadIdx.x >> 5] = correct;
    __syncthreads();
    for (int half = FUSE_REDUCE_THREADS / 2; half > 0; half >>= 1) {
        if (threadIdx.x < half) sm[threadIdx.x] += sm[threadIdx.x + half];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        part[blockIdx.x] = sm[0];
        unsigned int t = 0;
        for (int w = 0; w < FUSE_REDUCE_THREADS / 32; ++w) t += sc[w];
        if (n_correct && t) atomicAdd(n_correct, (unsigned long long)t);   // integer: order does not matter
    }
}

constexpr int ADAM_MAX_TENSORS = 16;
struct AdamBatch {
    float* p[ADAM_MAX_TENSORS];
    const float* g[ADAM_MAX_TENSORS];
    float* m[ADAM_MAX_TENSORS];
    float* v[ADAM_MAX_TENSORS];
    int64_t numel[ADAM_MAX_TENSORS];
    int count;
    float lr, beta1, beta2, eps, inv_c1, inv_c2;
};

__global__ void adam_kernel(const AdamBatch b) {
    const int t = blockIdx.y;
    if (t >= b.count) return;
    const int64_t nel = b.numel[t];
    float* __restrict__ p = b.p[t]; const float* __restrict__ g = b.g[t];
    float* __restrict__ m = b.m[t]; float* __restrict__ v = b.v[t];
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nel; i += (int64_t)gridDim.x * blockDim.x) {
        const float gi = g[i];
        const float mi = b.beta1 * m[i] + (1.0f - b.beta1) * gi;
        const float vi = b.beta2 * v[i] + (1.0f - b.beta2) * gi * gi;
        m[i] = mi; v[i] = vi;
        const float mhat = mi * b.inv_c1, vhat = vi * b.inv_c2;
        p[i] = p[i] - b.lr * mhat / (sqrtf(vhat) + b.eps);
    }
}

}  // namespace

namespace mixgcn {

// Scratch of the fused loss (a block of its own): [count u64][pad][partials double[blocks]][row_loss float[n]].
// Counts the train nodes (the gradient's 1/#T is needed inside the kernel that takes the loss) and clears n_correct.
mixgcn_status loss_fuse_begin(mixgcn_ctx* ctx, int64_t n, const int32_t* labels, const uint8_t* train_mask, int32_t* pred,
                              int64_t* n_correct, cudaStream_t s, LossFuse* out) {
    const int64_t cap = (int64_t)ctx->sm_count * 16;
    int64_t blocks = (n + 4095) / 4096;
    if (blocks > cap) blocks = cap;
    const int64_t off_rows = (16 + blocks * (int64_t)sizeof(double) + 255) & ~(int64_t)255;
    const int64_t need = off_rows + n * (int64_t)sizeof(float);
    if (need > ctx->workspace_loss_bytes) {
        MIXGCN_CUDA(cudaDeviceSynchronize());      // the old block may still be in use by enqueued kernels
        cudaFree(ctx->workspace_loss);
        ctx->workspace_loss = nullptr; ctx->workspace_loss_bytes = 0;
        void* q = nullptr;
        if (cudaMalloc(&q, (size_t)need) != cudaSuccess) {
            cudaGetLastError();
            MIXGCN_FAIL(MIXGCN_ENOMEM, "loss scratch of %lld bytes could not be allocated", (long long)need);
        }
        ctx->workspace_loss = q; ctx->workspace_loss_bytes = need;
    }
    char* base = reinterpret_cast<char*>(ctx->workspace_loss);
    unsigned long long* count = reinterpret_cast<unsigned long long*>(base);
    MIXGCN_CUDA(cudaMemsetAsync(count, 0, sizeof(unsigned long long), s));
    if (n_correct) MIXGCN_CUDA(cudaMemsetAsync(n_correct, 0, sizeof(int64_t), s));
    {
        LaunchScope scope(ctx, PH_LOSS, s);
        int64_t cb = (n + 255) / 256; if (cb > cap) cb = cap;
        count_mask_kernel<<<(unsigned)cb, 256, 0, s>>>(n, train_mask, count);
    }
    MIXGCN_CUDA(cudaGetLastError());
    out->labels = labels; out->train_mask = train_mask; out->count = count; out->pred = pred;
    out->part = reinterpret_cast<double*>(base + 16); out->n_part = (int)blocks;
    out->row_loss = reinterpret_cast<float*>(base + off_rows);
    out->zero_rows = ctx->loss_train_rows_only == 2 ? 0 : 1;
    return MIXGCN_OK;
}

mixgcn_status loss_fuse_end(mixgcn_ctx* ctx, int64_t n, int32_t C, const LossFuse& lf, float* loss, int64_t* n_correct, cudaStream_t s) {
    const int64_t chunk = (n + lf.n_part - 1) / lf.n_part;
    {
        LaunchScope scope(ctx, PH_LOSS, s);
        loss_rows_reduce_kernel<<<(unsigned)lf.n_part, FUSE_REDUCE_THREADS, 0, s>>>(n, C, chunk, lf.train_mask, lf.labels, lf.row_loss, lf.pred, lf.part,
                                                                                  reinterpret_cast<unsigned long long*>(n_correct));
    }
    {
        LaunchScope scope(ctx, PH_LOSS, s);
        loss_final_kernel<<<1, 32, 0, s>>>(lf.n_part, lf.part, lf.count, loss, ctx->d_status);
    }
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

}  // namespace mixgcn

extern "C" mixgcn_status mixgcn_loss_softmax_xent(mixgcn_ctx* ctx, int64_t n, int32_t C, const float* logits,
                                                  int64_t ld, const int32_t* labels, const uint8_t* train_mask,
                                                  float* loss, float* dlogits, int32_t* pred, int64_t* n_correct,
                                                  void* stream) {
    if (!ctx || !logits || !labels || !train_mask || !loss) MIXGCN_FAIL(MIXGCN_EINVAL, "loss: null argument");
    if (n <= 0 || C <= 0 || C > 4096) MIXGCN_FAIL(MIXGCN_EINVAL, "loss: need n > 0 and 1 <= C <= 4096 (n=%lld C=%d)", (long long)n, C);
    if (ld < C) MIXGCN_FAIL(MIXGCN_EINVAL, "loss: ld (%lld) < C (%d)", (long long)ld, C);
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    int64_t blocks = (n + LOSS_WARPS - 1) / LOSS_WARPS;
    const int64_t cap = (int64_t)ctx->sm_count * 16;
    if (blocks > cap) blocks = cap;
    // workspace: [count u64][pad][partials double[blocks]]
    MIXGCN_TRY(mixgcn::ensure_workspace(ctx, 16 + blocks * (int64_t)sizeof(double)));
    unsigned long long* count = reinterpret_cast<unsigned long long*>(ctx->workspace);
    double* part = reinterpret_cast<double*>(reinterpret_cast<char*>(ctx->workspace) + 16);
    MIXGCN_CUDA(cudaMemsetAsync(count, 0, sizeof(unsigned long long), s));
    if (n_correct) MIXGCN_CUDA(cudaMemsetAsync(n_correct, 0, sizeof(int64_t), s));
    {
        LaunchScope scope(ctx, PH_LOSS, s);
        int64_t cb = (n + 255) / 256; if (cb > cap) cb = cap;
        count_mask_kernel<<<(unsigned)cb, 256, 0, s>>>(n, train_mask, count);
    }
    int n_part = (int)blocks;
    {
        LaunchScope scope(ctx, PH_LOSS, s);
        if (ctx->loss_train_rows_only == 1)
            loss_rows_subset_kernel<<<(unsigned)blocks, LOSS_WARPS * 32, 0, s>>>(n, C, logits, ld, labels, train_mask, count, dlogits, pred,
                                                                              reinterpret_cast<unsigned long long*>(n_correct), part, ctx->d_status);
        else
            n_part = launch_loss_rows((unsigned)blocks, s, n, C, logits, ld, labels, train_mask, count, dlogits, pred,
                                      reinterpret_cast<unsigned long long*>(n_correct), part, ctx->d_status,
                                      ctx->loss_train_rows_only != 2, ctx->sm_count);
    }
    if (n_part < 0) MIXGCN_FAIL(MIXGCN_ECUDA, "loss: kernel launch failed: %s", cudaGetErrorString(cudaGetLastError()));
    {
        LaunchScope scope(ctx, PH_LOSS, s);
        loss_final_kernel<<<1, 32, 0, s>>>(n_part, part, count, loss, ctx->d_status);
    }
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

extern "C" mixgcn_status mixgcn_adam_step(mixgcn_ctx* ctx, int32_t n_tensors, float* const* param,
                                          const float* const* grad, float* const* m, float* const* v,
                                          const int64_t* numel, int64_t t, float lr, float beta1, float beta2,
                                          float eps, void* stream) {
    if (!ctx || n_tensors < 0 || (n_tensors > 0 && (!param || !grad || !m || !v || !numel)))
        MIXGCN_FAIL(MIXGCN_EINVAL, "adam: null argument");
    if (t < 1) MIXGCN_FAIL(MIXGCN_EINVAL, "adam: step count t must be >= 1 (got %lld)", (long long)t);
    for (int i = 0; i < n_tensors; ++i) {
        if (numel[i] < 0 || (numel[i] > 0 && (!param[i] || !grad[i] || !m[i] || !v[i])))
            MIXGCN_FAIL(MIXGCN_EINVAL, "adam: tensor %d has a null pointer or negative size", i);
    }
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    cudaStream_t s = (cudaStream_t)stream;
    const double c1 = 1.0 - pow((double)beta1, (double)t), c2 = 1.0 - pow((double)beta2, (double)t);
    for (int base = 0; base < n_tensors; base += ADAM_MAX_TENSORS) {
        AdamBatch b{};
        int64_t mx = 0;
        b.count = n_tensors - base < ADAM_MAX_TENSORS ? n_tensors - base : ADAM_MAX_TENSORS;
        for (int i = 0; i < b.count; ++i) {
            b.p[i] = param[base + i]; b.g[i] = grad[base + i]; b.m[i] = m[base + i]; b.v[i] = v[base + i];
            b.numel[i] = numel[base + i];
            if (b.numel[i] > mx) mx = b.numel[i];
        }
        if (mx == 0) continue;
        b.lr = lr; b.beta1 = beta1; b.beta2 = beta2; b.eps = eps;
        b.inv_c1 = (float)(1.0 / c1); b.inv_c2 = (float)(1.0 / c2);
        int64_t bx = (mx + 255) / 256; if (bx > 1024) bx = 1024;
        LaunchScope scope(ctx, PH_ADAM, s);
        adam_kernel<<<dim3((unsigned)bx, (unsigned)b.count), 256, 0, s>>>(b);
    }
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of the loss.
//
// Some callers cannot take device memory from the CUDA allocator: a process that has handed the
// whole GPU to its own memory pool (so cudaMalloc fails), or a latency-critical loop that cannot
// afford the device-wide synchronisation cudaMalloc and cudaFree imply.  They cannot create a
// mixgcn_ctx either (its status word and workspace come from cudaMalloc).  For them the loss
// kernels above run here with their scratch in a fixed array that is part of the library image.
// ------------------------------------------------------------------------------------------------
namespace {

constexpr int NOALLOC_MAX_PARTIALS = 32768;   // one fp64 partial per block
constexpr int NOALLOC_ROWS_PER_BLOCK = 1024;  // => at most 33,554,432 rows
constexpr int NOALLOC_MAX_DEVICES = 64;

struct NoAllocScratch {
    unsigned long long count;      // train nodes, cleared at the start of every call
    int32_t status;                // 0 ok, 1 empty train mask, 2 label out of range, 3 bounded wait expired; cleared likewise
    int32_t pad;
    double part[NOALLOC_MAX_PARTIALS];
};

// Held by every GPU that loads the library, until the process exits (about 256 KB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

// In host code the array's name is only a handle for the runtime, not a device address; the real
// address is looked up once per device (with that device current) and cached here.  Host threads that
// make their first call on a device at the same time both store the same address: the entries are
// atomic so that this is well defined.
std::atomic<NoAllocScratch*> g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};

}  // namespace

extern "C" mixgcn_status mixgcn_loss_softmax_xent_noalloc(int64_t n, int32_t C, const float* logits, int64_t ld,
                                                          const int32_t* labels, const uint8_t* train_mask,
                                                          float* loss, float* dlogits, int32_t* pred,
                                                          int64_t* n_correct, int32_t* status, void* stream) {
    if (!logits || !labels || !train_mask || !loss) MIXGCN_FAIL(MIXGCN_EINVAL, "loss_noalloc: null argument");
    if (n <= 0 || C <= 0 || C > 4096)
        MIXGCN_FAIL(MIXGCN_EINVAL, "loss_noalloc: need n > 0 and 1 <= C <= 4096 (n=%lld C=%d)", (long long)n, C);
    if (ld < C) MIXGCN_FAIL(MIXGCN_EINVAL, "loss_noalloc: ld (%lld) < C (%d)", (long long)ld, C);
    const int64_t max_rows = (int64_t)NOALLOC_MAX_PARTIALS * NOALLOC_ROWS_PER_BLOCK;
    if (n > max_rows)
        MIXGCN_FAIL(MIXGCN_EUNSUPPORTED,
                    "loss_noalloc: n = %lld exceeds the %lld rows the built-in scratch covers; use mixgcn_loss_softmax_xent",
                    (long long)n, (long long)max_rows);
    int device = -1;
    MIXGCN_CUDA(cudaGetDevice(&device));
    if (device < 0 || device >= NOALLOC_MAX_DEVICES) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "loss_noalloc: device index %d not supported", device);
    if (!g_noalloc_ptr[device].load(std::memory_order_acquire)) {
        // first call on this device: resolve the device address of the scratch array
        void* p = nullptr;
        MIXGCN_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        if (!p) MIXGCN_FAIL(MIXGCN_ECUDA, "loss_noalloc: the scratch symbol has no device address");
        g_noalloc_ptr[device].store(reinterpret_cast<NoAllocScratch*>(p), std::memory_order_release);
    }
    NoAllocScratch* sc = g_noalloc_ptr[device].load(std::memory_order_acquire);
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t blocks = (n + NOALLOC_ROWS_PER_BLOCK - 1) / NOALLOC_ROWS_PER_BLOCK;
    // the array keeps the previous call's contents: clear the counter and the status word
    MIXGCN_CUDA(cudaMemsetAsync(sc, 0, offsetof(NoAllocScratch, part), s));
    if (n_correct) MIXGCN_CUDA(cudaMemsetAsync(n_correct, 0, sizeof(int64_t), s));
    int64_t cb = (n + 255) / 256;
    if (cb > 4096) cb = 4096;
    count_mask_kernel<<<(unsigned)cb, 256, 0, s>>>(n, train_mask, &sc->count);
    int sm_count = 0;
    MIXGCN_CUDA(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device));
    const int n_part = launch_loss_rows((unsigned)blocks, s, n, C, logits, ld, labels, train_mask, &sc->count, dlogits, pred,
                                        reinterpret_cast<unsigned long long*>(n_correct), sc->part, &sc->status, true, sm_count);
    if (n_part < 0) MIXGCN_FAIL(MIXGCN_ECUDA, "loss_noalloc: kernel launch failed: %s", cudaGetErrorString(cudaGetLastError()));
    loss_final_kernel<<<1, 32, 0, s>>>(n_part, sc->part, &sc->count, loss, &sc->status);
    if (status) MIXGCN_CUDA(cudaMemcpyAsync(status, &sc->status, sizeof(int32_t), cudaMemcpyDeviceToDevice, s));
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}
