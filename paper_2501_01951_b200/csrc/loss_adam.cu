// Masked softmax cross-entropy with its gradient and arg-max (the loss line of Algorithm 2),
// and the Adam step (its weight-update line).  Both are streaming kernels; floating-point
// reductions run in a fixed order (per-warp shuffles, per-CTA partials, one final pass).
#include <stddef.h>

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

// Picks the register-resident kernel when the row fits (C <= 256) and the layout allows float4 access.
void launch_loss_rows(unsigned blocks, cudaStream_t s, int64_t n, int C, const float* logits, int64_t ld,
                      const int32_t* labels, const uint8_t* mask, const unsigned long long* count, float* dlogits,
                      int32_t* pred, unsigned long long* n_correct, double* part, int32_t* status, bool zero_rows = true) {
    const bool vec = (ld & 3) == 0 && aligned16(logits) && (!dlogits || aligned16(dlogits));
    if (vec && C <= 128)
        loss_rows_vec_kernel<1><<<blocks, LOSS_WARPS * 32, 0, s>>>(n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows);
    else if (vec && C <= 256)
        loss_rows_vec_kernel<2><<<blocks, LOSS_WARPS * 32, 0, s>>>(n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows);
    else
        loss_rows_kernel<<<blocks, LOSS_WARPS * 32, 0, s>>>(n, C, logits, ld, labels, mask, count, dlogits, pred, n_correct, part, status, zero_rows);
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
    {
        LaunchScope scope(ctx, PH_LOSS, s);
        if (ctx->loss_train_rows_only == 1)
            loss_rows_subset_kernel<<<(unsigned)blocks, LOSS_WARPS * 32, 0, s>>>(n, C, logits, ld, labels, train_mask, count, dlogits, pred,
                                                                              reinterpret_cast<unsigned long long*>(n_correct), part, ctx->d_status);
        else
            launch_loss_rows((unsigned)blocks, s, n, C, logits, ld, labels, train_mask, count, dlogits, pred,
                             reinterpret_cast<unsigned long long*>(n_correct), part, ctx->d_status, ctx->loss_train_rows_only != 2);
    }
    {
        LaunchScope scope(ctx, PH_LOSS, s);
        loss_final_kernel<<<1, 32, 0, s>>>((int)blocks, part, count, loss, ctx->d_status);
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
    int32_t status;                // 0 ok, 1 empty train mask, 2 label out of range; cleared likewise
    int32_t pad;
    double part[NOALLOC_MAX_PARTIALS];
};

// Held by every GPU that loads the library, until the process exits (about 256 KB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

// In host code the array's name is only a handle for the runtime, not a device address; the real
// address is looked up once per device (with that device current) and cached here.
NoAllocScratch* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};

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
    if (!g_noalloc_ptr[device]) {
        // first call on this device: resolve the device address of the scratch array
        void* p = nullptr;
        MIXGCN_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        if (!p) MIXGCN_FAIL(MIXGCN_ECUDA, "loss_noalloc: the scratch symbol has no device address");
        g_noalloc_ptr[device] = reinterpret_cast<NoAllocScratch*>(p);
    }
    NoAllocScratch* sc = g_noalloc_ptr[device];
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t blocks = (n + NOALLOC_ROWS_PER_BLOCK - 1) / NOALLOC_ROWS_PER_BLOCK;
    // the array keeps the previous call's contents: clear the counter and the status word
    MIXGCN_CUDA(cudaMemsetAsync(sc, 0, offsetof(NoAllocScratch, part), s));
    if (n_correct) MIXGCN_CUDA(cudaMemsetAsync(n_correct, 0, sizeof(int64_t), s));
    int64_t cb = (n + 255) / 256;
    if (cb > 4096) cb = 4096;
    count_mask_kernel<<<(unsigned)cb, 256, 0, s>>>(n, train_mask, &sc->count);
    launch_loss_rows((unsigned)blocks, s, n, C, logits, ld, labels, train_mask, &sc->count, dlogits, pred,
                     reinterpret_cast<unsigned long long*>(n_correct), sc->part, &sc->status);
    loss_final_kernel<<<1, 32, 0, s>>>((int)blocks, sc->part, &sc->count, loss, &sc->status);
    if (status) MIXGCN_CUDA(cudaMemcpyAsync(status, &sc->status, sizeof(int32_t), cudaMemcpyDeviceToDevice, s));
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}
