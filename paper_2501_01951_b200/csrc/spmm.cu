// Neighbour aggregation Z = A_hat Y (Algorithm 2, aggregation line): deterministic, atomic-free,
// row-wise CSR SpMM.
//
//  - A group of LPR lanes owns one output row (or one segment of a long row); each lane owns VPL
//    float4 column groups, so a gathered row of Y is read with coalesced 16-byte loads.
//  - The work list is the graph's schedule: one 16-byte record (first entry, length, row) per
//    unit, longest first, so a unit starts after ONE dependent load instead of a chain through
//    the permutation and the row pointers.
//  - (col,val) of the unit are fetched LPR at a time (one coalesced load per group) and handed
//    round with warp shuffles; U gathered rows (U * VPL = 8 float4 per lane) are in flight before
//    the FMAs, with a predicated tail instead of a one-by-one remainder.
//  - Degree buckets: rows of up to 12 / 5 / 2 entries share a warp 2- / 4- / 8-fold (fewer lanes per
//    row, more float4 per lane), so short rows still keep eight loads per lane in flight.
//  - Rows longer than SPMM_SEG entries are cut (at column-block boundaries and every SPMM_SEG
//    entries) into segments that run as independent units, in order of their first column, and
//    write partial rows to scratch: hub rows that gather the same rows of Y do so close in time
//    and share them through the L2.  A second kernel adds the segments of each row in entry order
//    and applies the epilogue.  Every sum has a fixed order: the result is bit-reproducible.
//  - The epilogue (bias, ReLU, dropout mask, gate by another tensor's sign) is applied in
//    registers before the single write of Z.
#include "internal.cuh"

using namespace mixgcn;

// Launch shapes the measurements settled on (workload with 30M nodes, width 128, and the wide / dense ones).
constexpr int SPMM_MINB = 4;          // CTAs per SM asked of the compiler for the narrow (VPL <= 2) group kernels
constexpr int SPMM_FOLD_WMAX = 128;   // widest aggregation the two folds below apply to
constexpr int SPMM_FOLD_SEG = 2;      // long-row segments at widths <= 128: 16 lanes x 2 float4 per unit (1 would be 32 lanes x 1)
constexpr int SPMM_FOLD_MED = 2;      // the same for rows of 13..512 entries
constexpr int SPMM_SHORT_RB = 4;      // rows a warp of the short-row kernel takes at once
constexpr int SPMM_SHORT_MINB = 5;    // CTAs per SM asked of the compiler for it
constexpr int SPMM_SHORT_MAXE = 2;    // rows of at most this many entries go to the short-row kernel
constexpr int SPMM_U = 8;             // float4 loads a lane keeps in flight

namespace {

struct SpmmParams {
    const SpmmRec* rec;    // schedule records, or null: unit idx is row idx of the CSR
    const int64_t* rowptr;
    const int32_t* col;
    const float* val;
    int64_t idx_begin, idx_end;
    int32_t w;             // columns handled by this launch (slice width)
    int32_t j0;            // first column of the slice (multiple of 4)
    int32_t w_total;       // full width (for the dense drop-mask index)
    const float* Y; int64_t ldy;
    float* Z; int64_t ldz;
    uint16_t* Z_lp; int64_t ldz_lp;   // nullable: bf16 copy of Z (after the epilogue) for a bf16 dense product that follows
    float* partial;        // non-null: unit idx writes its raw sums to partial[idx * ldp + ...]
    int64_t ldp;
    // row-sparse input (spmm_sparse_kernel): rows v of the input with in_mask[v] == 0 are exactly zero
    // and are skipped; a kept row v is read from Y row in_pos[v] (in_pos == null: row v itself)
    const uint8_t* in_mask;
    const int32_t* in_pos;
    uint8_t* out_mask;     // nullable: receives 1 for output rows that received a contribution, else 0
    // row filter (spmm_filtered_kernel): only output rows u with row_filter[u] != 0 are computed and written
    const uint8_t* row_filter;
    const int32_t* seg_perm;   // segment records carry the long row's index i; its row is seg_perm[i] (null: the record's row)
    // sampled aggregation Z = (A_hat Y) (.) M, Eq. 4: bit j of row u of the bitmap says whether output (u, j) is kept
    // The same bitmap serves a bit-packed gate (the bitmap mask buffer of Section 3.2.1 holding a ReLU mask): kept
    // outputs are then scaled by bits_scale and nothing is skipped (bits_skip = 0).
    const uint32_t* out_bits;  // [n x ld_bits] words, null: every output is kept
    int64_t ld_bits;
    float bits_scale;          // factor of the kept outputs (1 for the sampled aggregation, the gate's scale for a gate)
    int bits_skip;             // 1: lanes whose four columns of a row are all masked skip that row's gathers
    // epilogue
    const float* bias; int relu;
    const uint8_t* drop; float keep_scale;
    const float* gate; int64_t ld_gate; float gate_scale;
    const float* residual; int64_t ld_residual; float residual_scale;
    // loss epilogue (kernels instantiated with LOSS): labels, train mask, number of train nodes, per-row loss, arg-max
    const int32_t* loss_labels; const uint8_t* loss_mask; const unsigned long long* loss_count;
    float* loss_row; int32_t* loss_pred; int loss_zero_rows;
    // limits for the index tests of the bounds-checked debug build (unused otherwise)
    int32_t* status;
    int64_t n_cols;        // column ids lie in [0, n_cols) (they index in_mask / in_pos, or Y itself)
    int64_t y_rows;        // rows of Y
    int64_t n_out;         // output rows
    int64_t n_long;        // long rows of the schedule (a segment record's `row` is an ordinal among them)
    int64_t nnz;           // stored entries
    int64_t n_partial;     // partial-row slots
};

// entry range and row of a unit: tested in the debug build before anything is addressed with them
__device__ __forceinline__ bool unit_ok(const SpmmParams& p, int64_t b, int64_t e, int64_t u) {
    return index_ok(b, p.nnz + 1, p.status, SITE_SPMM_RANGE) && index_ok(e, p.nnz + 1, p.status, SITE_SPMM_RANGE) &&
           index_ok(u, p.partial ? p.n_long : p.n_out, p.status, SITE_SPMM_ROW);   // a segment's record names its long row by ordinal
}

__device__ __forceinline__ float epilogue1(const SpmmParams& p, float y, int64_t u, int j) {
    if (p.residual) y = fmaf(p.residual_scale, p.residual[u * p.ld_residual + j], y);
    if (p.bias) y += p.bias[j];
    if (p.relu) y = fmaxf(y, 0.0f);
    if (p.drop) y = p.drop[u * p.w_total + j] ? y * p.keep_scale : 0.0f;
    if (p.gate) y = p.gate[u * p.ld_gate + j] > 0.0f ? y * p.gate_scale : 0.0f;
    return y;
}

// four fp32 -> four bf16 (round to nearest even), 8 bytes
__device__ __forceinline__ void store_lp4(uint16_t* dst, float x, float y, float z, float w) {
    uint32_t lo, hi;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(y), "f"(x));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(w), "f"(z));
    *reinterpret_cast<uint2*>(dst) = make_uint2(lo, hi);
}

__device__ __forceinline__ void store_row(const SpmmParams& p, int64_t u, int c4, float4 a) {
    const int j = p.j0 + c4 * 4;           // global column of a.x
    const int jend = p.j0 + p.w;           // one past the last valid column of the slice
    float r[4] = {a.x, a.y, a.z, a.w};
    if (!p.bias && !p.residual && a.x == 0.0f && a.y == 0.0f && a.z == 0.0f && a.w == 0.0f) {
        // ReLU, dropout and the gate all map 0 to 0: no mask or gate byte needs to be read (the empty
        // rows of a row-sparse aggregation take this path)
        if (p.Z) *reinterpret_cast<float4*>(p.Z + u * p.ldz + j) = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.Z_lp) *reinterpret_cast<uint2*>(p.Z_lp + u * p.ldz_lp + j) = make_uint2(0u, 0u);
        return;
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) r[t] = (j + t < jend) ? epilogue1(p, r[t], u, j + t) : 0.0f;
    if (p.out_bits) {
        const uint32_t nib = (__ldg(p.out_bits + u * p.ld_bits + (j >> 5)) >> (j & 31)) & 0xFu;   // j % 4 == 0: one word
#pragma unroll
        for (int t = 0; t < 4; ++t) r[t] = ((nib >> t) & 1u) ? r[t] * p.bits_scale : 0.0f;
    }
    if (p.Z) *reinterpret_cast<float4*>(p.Z + u * p.ldz + j) = make_float4(r[0], r[1], r[2], r[3]);   // null: bf16 copy only
    if (p.Z_lp) store_lp4(p.Z_lp + u * p.ldz_lp + j, r[0], r[1], r[2], r[3]);
}

// What stands between the sums and the stored row -- the general epilogue's code costs the gather loop registers
// under the cap, so the forms the epochs spend their time in have instances without it:
//   EPI_PLAIN  nothing (every forward aggregation of an aggregate-first layer, every partial row of a long-row segment)
//   EPI_BITS   a bit-packed gate only (the backward aggregation that produces a gated input gradient)
//   EPI_BIAS   bias, then ReLU if asked (the forward aggregation of an update-first layer)
//   EPI_GATE   an fp32 gate only, 16-byte aligned with a leading dimension that is a multiple of 4
//   EPI_LOSS   bias + soft-max cross-entropy (loss_epilogue)
//   EPI_ANY    everything store_row knows
enum { EPI_ANY = 0, EPI_LOSS = 1, EPI_PLAIN = 2, EPI_BITS = 3, EPI_BIAS = 4, EPI_GATE = 5 };
constexpr bool epi_is_lean(int epi) { return epi >= EPI_PLAIN; }

// store_row for the lean instances; pad columns of the last group are written as zeros, as store_row does.
template <int EPI>
__device__ __forceinline__ void store_lean(const SpmmParams& p, int64_t u, int c4, float4 y) {
    const int j = p.j0 + c4 * 4;
    const int left = p.j0 + p.w - j;             // valid columns of this group (>= 1)
    if constexpr (EPI == EPI_BIAS) {
        float4 b4;
        if (left >= 4) b4 = __ldg(reinterpret_cast<const float4*>(p.bias + j));
        else b4 = make_float4(__ldg(p.bias + j), left > 1 ? __ldg(p.bias + j + 1) : 0.0f, left > 2 ? __ldg(p.bias + j + 2) : 0.0f, 0.0f);
        y.x += b4.x; y.y += b4.y; y.z += b4.z; y.w += b4.w;
        if (p.relu) { y.x = fmaxf(y.x, 0.0f); y.y = fmaxf(y.y, 0.0f); y.z = fmaxf(y.z, 0.0f); y.w = fmaxf(y.w, 0.0f); }
    }
    if constexpr (EPI == EPI_GATE) {
        const float4 g4 = __ldg(reinterpret_cast<const float4*>(p.gate + u * p.ld_gate + j));   // inside the row: ld_gate % 4 == 0
        y.x = g4.x > 0.0f ? y.x * p.gate_scale : 0.0f; y.y = g4.y > 0.0f ? y.y * p.gate_scale : 0.0f;
        y.z = g4.z > 0.0f ? y.z * p.gate_scale : 0.0f; y.w = g4.w > 0.0f ? y.w * p.gate_scale : 0.0f;
    }
    if constexpr (EPI == EPI_BITS) {
        const uint32_t nib = (__ldg(p.out_bits + u * p.ld_bits + (j >> 5)) >> (j & 31)) & 0xFu;   // j % 4 == 0: one word
        y.x = (nib & 1u) ? y.x * p.bits_scale : 0.0f; y.y = (nib & 2u) ? y.y * p.bits_scale : 0.0f;
        y.z = (nib & 4u) ? y.z * p.bits_scale : 0.0f; y.w = (nib & 8u) ? y.w * p.bits_scale : 0.0f;
    }
    if (left < 4) { if (left < 2) y.y = 0.0f; if (left < 3) y.z = 0.0f; y.w = 0.0f; }
    if (p.Z) *reinterpret_cast<float4*>(p.Z + u * p.ldz + j) = y;
    if (p.Z_lp) store_lp4(p.Z_lp + u * p.ldz_lp + j, y.x, y.y, y.z, y.w);
}

// Which lean instance serves this launch (EPI_ANY: none does).
inline int pick_epi(const SpmmParams& p) {
    if (p.out_bits && p.bits_skip) return EPI_ANY;                 // the sampled aggregation skips gathers: general instance
    if (p.partial) return EPI_PLAIN;                               // a partial row never has an epilogue
    if (p.drop || p.residual) return EPI_ANY;
    const bool bias = p.bias != nullptr || p.relu, gate = p.gate != nullptr, bits = p.out_bits != nullptr;
    if (!bias && !gate && !bits) return EPI_PLAIN;
    if (bits && !bias && !gate) return EPI_BITS;
    if (bias && !gate && !bits && p.bias && (reinterpret_cast<uintptr_t>(p.bias) & 15u) == 0) return EPI_BIAS;
    if (gate && !bias && !bits && (reinterpret_cast<uintptr_t>(p.gate) & 15u) == 0 && (p.ld_gate & 3) == 0) return EPI_GATE;
    return EPI_ANY;
}

__device__ __forceinline__ void fma4(float4& acc, float a, const float4& y) {
    acc.x = fmaf(a, y.x, acc.x); acc.y = fmaf(a, y.y, acc.y);
    acc.z = fmaf(a, y.z, acc.z); acc.w = fmaf(a, y.w, acc.w);
}

// Soft-max cross-entropy of output row u taken from the registers that hold the aggregated row (the whole
// row belongs to one group of LPR lanes, lane `lig` holding float4 groups lig + v * LPR): logits = sums + bias;
// arg-max with lowest-index ties -> pred; on a train row the loss term lse - logit[label] -> loss_row[u] and the
// gradient (softmax - e_label) / #T -> Z row u.  The logits themselves are never written.
template <int LPR, int VPL>
__device__ __forceinline__ void loss_epilogue(const SpmmParams& p, int64_t u, int lig, unsigned mask, const float4 (&acc)[VPL]) {
    const int C = p.w;                 // one slice: j0 == 0
    const int w4 = (C + 3) >> 2;
    float x[VPL][4];
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int j = (lig + v * LPR) * 4;
        const float a[4] = {acc[v].x, acc[v].y, acc[v].z, acc[v].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) x[v][e] = j + e < C ? (p.bias ? a[e] + __ldg(p.bias + j + e) : a[e]) : -INFINITY;
    }
    float mx = -INFINITY; int arg = 0x7FFFFFFF;
#pragma unroll
    for (int v = 0; v < VPL; ++v)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int c = (lig + v * LPR) * 4 + e;
            if (c < C && (x[v][e] > mx || (x[v][e] == mx && c < arg))) { mx = x[v][e]; arg = c; }
        }
    if (arg == 0x7FFFFFFF) arg = lig * 4 < C ? lig * 4 : 0;       // nothing but -inf / NaN in this lane's columns
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) {
        const float omx = __shfl_xor_sync(mask, mx, o, LPR);
        const int oarg = __shfl_xor_sync(mask, arg, o, LPR);
        if (omx > mx || (omx == mx && oarg < arg)) { mx = omx; arg = oarg; }
    }
    if (p.loss_pred && lig == 0) p.loss_pred[u] = arg;
    const unsigned long long T = *p.loss_count;
    const bool train = __ldg(p.loss_mask + u) != 0 && T != 0;
    int y = 0; bool ok = false;
    if (train) {
        y = __ldg(p.loss_labels + u);
        ok = y >= 0 && y < C;
        if (!ok && lig == 0) atomicMax(p.status, DEV_BAD_LABEL);
    }
    if (!train || !ok) {
        if (p.loss_zero_rows || train) {
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                const int c4 = lig + v * LPR;
                if (c4 < w4) *reinterpret_cast<float4*>(p.Z + u * p.ldz + c4 * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        return;
    }
    float s = 0.0f;
#pragma unroll
    for (int v = 0; v < VPL; ++v)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if ((lig + v * LPR) * 4 + e < C) s += expf(x[v][e] - mx);
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(mask, s, o, LPR);
    const float lse = mx + logf(s);
    float py = 0.0f;        // the label's logit lives in lane (y/4) % LPR of the group
#pragma unroll
    for (int v = 0; v < VPL; ++v)
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if ((lig + v * LPR) * 4 + e == y) py = x[v][e];
    py = __shfl_sync(mask, py, (y >> 2) & (LPR - 1), LPR);
    if (lig == 0) p.loss_row[u] = lse - py;
    const float invT = (float)(1.0 / (double)T);
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int c4 = lig + v * LPR;
        if (c4 < w4) {
            float r[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = c4 * 4 + e;
                r[e] = c < C ? (expf(x[v][e] - lse) - (c == y ? 1.0f : 0.0f)) * invT : 0.0f;
            }
            *reinterpret_cast<float4*>(p.Z + u * p.ldz + c4 * 4) = make_float4(r[0], r[1], r[2], r[3]);
        }
    }
}

template <int LPR, int VPL>
struct Cfg {
    static constexpr int U0 = SPMM_U / VPL < 1 ? 1 : SPMM_U / VPL;
    static constexpr int U = U0 > LPR ? LPR : U0;   // gathered rows in flight per lane group
};

// Accumulate entries [b, e) into acc[] for the lane's column groups, ascending entry order.
// The (col, val) pair of the NEXT batch of LPR entries is requested before the current batch's gathers,
// so that the index load's latency is hidden behind them instead of preceding every batch.
template <int LPR, int VPL, bool FULL = false>     // FULL: the slice has exactly LPR * VPL column groups (no lane is idle)
__device__ __forceinline__ void row_segment(const SpmmParams& p, int64_t b, int64_t e, int lig, unsigned mask,
                                            int w4, float4 (&acc)[VPL], unsigned keep = 0xFFFFFFFFu) {
    constexpr int U = Cfg<LPR, VPL>::U;
    const float* Yb = p.Y + p.j0;
    int c = 0; float a = 0.0f;
    if (b + lig < e) { c = __ldg(p.col + b + lig); a = __ldg(p.val + b + lig); }
    for (int64_t i0 = b; i0 < e; i0 += LPR) {
        int c_next = 0; float a_next = 0.0f;
        if (i0 + LPR + lig < e) { c_next = __ldg(p.col + i0 + LPR + lig); a_next = __ldg(p.val + i0 + LPR + lig); }
        const int cnt = (int)((e - i0) < LPR ? (e - i0) : LPR);
        for (int k = 0; k < cnt; k += U) {
            int ck[U]; float ak[U]; float4 y[U][VPL];
#pragma unroll
            for (int t = 0; t < U; ++t) {
                ck[t] = __shfl_sync(mask, c, k + t, LPR);
                ak[t] = __shfl_sync(mask, a, k + t, LPR);
            }
#pragma unroll
            for (int t = 0; t < U; ++t) {
                const float4* yr = reinterpret_cast<const float4*>(Yb + (int64_t)ck[t] * p.ldy);
                const bool live = k + t < cnt && index_ok(ck[t], p.y_rows, p.status, SITE_SPMM_COL);
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    const int c4 = lig + v * LPR;
                    y[t][v] = (live && (FULL || c4 < w4) && ((keep >> v) & 1u)) ? __ldg(yr + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int t = 0; t < U; ++t)
                if (k + t < cnt) {
#pragma unroll
                    for (int v = 0; v < VPL; ++v) fma4(acc[v], ak[t], y[t][v]);
                }
        }
        c = c_next; a = a_next;
    }
}

// FULL (plain and bit-gate instances): the slice has exactly LPR * VPL column groups, so no load is predicated on its column.
template <int LPR, int VPL, int EPI = EPI_ANY, bool FULL = false>
__global__ void __launch_bounds__(256, VPL <= 2 ? SPMM_MINB : 1) spmm_group_kernel(const SpmmParams p) {
    constexpr bool LOSS = EPI == EPI_LOSS, PLAIN = epi_is_lean(EPI);
    const int lig = threadIdx.x % LPR;
    const int64_t idx = p.idx_begin + ((int64_t)blockIdx.x * 256 + threadIdx.x) / LPR;
    if (idx >= p.idx_end) return;  // the whole group leaves together
    const unsigned mask = LPR == 32 ? 0xFFFFFFFFu : (((1u << LPR) - 1u) << ((threadIdx.x & 31) & ~(LPR - 1)));
    int64_t b, e, u;
    if (p.rec) {
        const int4 r = __ldg(reinterpret_cast<const int4*>(p.rec + idx));
        b = ((int64_t)(uint32_t)r.y << 32) | (uint32_t)r.x;
        e = b + r.z;
        u = r.w;
    } else {
        u = idx;
        b = __ldg(p.rowptr + u);
        e = __ldg(p.rowptr + u + 1);
    }
    if (!unit_ok(p, b, e, u)) return;
    const int w4 = (p.w + 3) >> 2;
    float4 acc[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    unsigned keep = 0xFFFFFFFFu;
    if (!PLAIN && p.out_bits && p.bits_skip) {
        // Eq. 4: outputs the mask drops are never computed -- a lane whose four columns of this row are all
        // masked skips its gathers of every neighbour (the mask is known before the aggregation)
        const int64_t row = p.seg_perm ? __ldg(p.seg_perm + u) : u;
        keep = 0u;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int c4 = lig + v * LPR;
            if (c4 < w4) {
                const int j = p.j0 + c4 * 4;
                if ((__ldg(p.out_bits + row * p.ld_bits + (j >> 5)) >> (j & 31)) & 0xFu) keep |= 1u << v;
            }
        }
    }
    row_segment<LPR, VPL, FULL>(p, b, e, lig, mask, w4, acc, keep);
    if (p.partial) {
        float4* dst = reinterpret_cast<float4*>(p.partial + idx * p.ldp);
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int c4 = lig + v * LPR;
            if (c4 < w4) dst[c4] = acc[v];
        }
        return;
    }
    if constexpr (LOSS) {
        loss_epilogue<LPR, VPL>(p, u, lig, mask, acc);
    } else {
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int c4 = lig + v * LPR;
            if (c4 < w4) {
                if constexpr (PLAIN) store_lean<EPI>(p, u, c4, acc[v]);
                else store_row(p, u, c4, acc[v]);
            }
        }
    }
}

// Rows of at most MAXE entries, width <= 128: a warp takes RB schedule records at once.  Lanes read the
// records, column ids and values in one coalesced load each; every gathered row of Y is then a single
// 512-byte request of the whole warp (lane = float4 column), RB of them in flight; entries of a row are
// added in entry order, as everywhere else.
template <int RB, int MAXE, int EPI = EPI_ANY, int VPL = 1>      // VPL float4 per lane: widths up to 128 * VPL
__global__ void __launch_bounds__(256, VPL == 1 ? SPMM_SHORT_MINB : SPMM_MINB) spmm_short_kernel(const SpmmParams p) {
    static_assert(RB * MAXE <= 32, "one lane per (row, entry)");
    const int lane = threadIdx.x & 31;
    const int64_t idx0 = p.idx_begin + (((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5) * RB;
    if (idx0 >= p.idx_end) return;
    int4 rc = make_int4(0, 0, 0, 0);
    if (lane < RB && idx0 + lane < p.idx_end) rc = __ldg(reinterpret_cast<const int4*>(p.rec + idx0 + lane));
    if constexpr (DEBUG_BOUNDS) {
        const int64_t b0 = ((int64_t)(uint32_t)rc.y << 32) | (uint32_t)rc.x;
        if (!unit_ok(p, b0, b0 + rc.z, rc.w)) { rc.z = 0; rc.w = -1; }      // a bad record: no entries, no store
    }
    // lane (k, e) = (lane % RB, lane / RB) fetches entry e of row k
    const int k_of = lane % RB, e_of = lane / RB;
    const uint32_t lo = (uint32_t)__shfl_sync(0xFFFFFFFFu, rc.x, k_of), hi = (uint32_t)__shfl_sync(0xFFFFFFFFu, rc.y, k_of);
    const int len_of = __shfl_sync(0xFFFFFFFFu, rc.z, k_of);
    int c = 0; float a = 0.0f;
    if (e_of < MAXE && e_of < len_of) {
        const int64_t at = (((int64_t)hi << 32) | lo) + e_of;
        c = __ldg(p.col + at); a = __ldg(p.val + at);
    }
    const int w4 = (p.w + 3) >> 2;
    const float* Yb = p.Y + p.j0;
    float4 acc[RB][VPL];
#pragma unroll
    for (int k = 0; k < RB; ++k)
#pragma unroll
        for (int v = 0; v < VPL; ++v) acc[k][v] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int e = 0; e < MAXE; ++e) {
        float4 y[RB][VPL]; float ak[RB];
#pragma unroll
        for (int k = 0; k < RB; ++k) {
            const int ck = __shfl_sync(0xFFFFFFFFu, c, k + e * RB);
            ak[k] = __shfl_sync(0xFFFFFFFFu, a, k + e * RB);
            const int len_k = __shfl_sync(0xFFFFFFFFu, rc.z, k);
            const bool live = e < len_k && index_ok(ck, p.y_rows, p.status, SITE_SPMM_COL);
            const float4* yr = reinterpret_cast<const float4*>(Yb + (int64_t)ck * p.ldy);
#pragma unroll
            for (int v = 0; v < VPL; ++v)
                y[k][v] = (live && lane + 32 * v < w4) ? __ldg(yr + lane + 32 * v) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < RB; ++k) {
            const int len_k = __shfl_sync(0xFFFFFFFFu, rc.z, k);
            if (e < len_k) {
#pragma unroll
                for (int v = 0; v < VPL; ++v) fma4(acc[k][v], ak[k], y[k][v]);
            }
        }
    }
#pragma unroll
    for (int k = 0; k < RB; ++k) {
        const int64_t u = __shfl_sync(0xFFFFFFFFu, rc.w, k);
        if (idx0 + k < p.idx_end && (!DEBUG_BOUNDS || u >= 0)) {
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                const int c4 = lane + 32 * v;
                if (c4 < w4) {
                    if constexpr (epi_is_lean(EPI)) store_lean<EPI>(p, u, c4, acc[k][v]);      // as in spmm_group_kernel
                    else store_row(p, u, c4, acc[k][v]);
                }
            }
        }
    }
}

// Row-sparse input: most rows of Y are exactly zero (gradients of a masked loss and what they
// propagate to).  A unit scans its column ids, tests the row mask (one byte per entry, L2-resident)
// and gathers only the kept rows, four at a time, in entry order -- the same sum as the dense kernel
// with its zero terms left out.  Values are read for kept entries only.
template <int LPR, int VPL>
__global__ void __launch_bounds__(256) spmm_sparse_kernel(const SpmmParams p) {
    const int lig = threadIdx.x % LPR;
    const int64_t idx = p.idx_begin + ((int64_t)blockIdx.x * 256 + threadIdx.x) / LPR;
    if (idx >= p.idx_end) return;
    const int group_base = (threadIdx.x & 31) & ~(LPR - 1);
    const unsigned mask = LPR == 32 ? 0xFFFFFFFFu : (((1u << LPR) - 1u) << group_base);
    const int4 rc = __ldg(reinterpret_cast<const int4*>(p.rec + idx));
    const int64_t b = ((int64_t)(uint32_t)rc.y << 32) | (uint32_t)rc.x, e = b + rc.z;
    const int64_t u = rc.w;
    if (!unit_ok(p, b, e, u)) return;
    const int w4 = (p.w + 3) >> 2;
    const float* Yb = p.Y + p.j0;
    float4 acc[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    bool any = false;
    for (int64_t i0 = b; i0 < e; i0 += LPR) {
        int r = -1; float a = 0.0f;
        if (i0 + lig < e) {
            const int c = __ldg(p.col + i0 + lig);
            if (index_ok(c, p.n_cols, p.status, SITE_SPMM_COL) && __ldg(p.in_mask + c)) {
                r = p.in_pos ? __ldg(p.in_pos + c) : c;
                a = __ldg(p.val + i0 + lig);
            }
        }
        unsigned hits = __ballot_sync(mask, r >= 0) & mask;
        any |= hits != 0;
        constexpr int HB = VPL >= 4 ? 1 : 4 / VPL;     // kept rows gathered per batch
        while (hits) {
            int src[HB], nh = 0;
#pragma unroll
            for (int t = 0; t < HB; ++t) {
                src[t] = 0;
                if (hits) { src[t] = __ffs(hits) - 1 - group_base; hits &= hits - 1; ++nh; }
            }
            int rk[HB]; float ak[HB]; float4 y[HB][VPL];
#pragma unroll
            for (int t = 0; t < HB; ++t) {
                rk[t] = __shfl_sync(mask, r, src[t], LPR);
                ak[t] = __shfl_sync(mask, a, src[t], LPR);
            }
#pragma unroll
            for (int t = 0; t < HB; ++t) {
                const float4* yr = reinterpret_cast<const float4*>(Yb + (int64_t)(rk[t] < 0 ? 0 : rk[t]) * p.ldy);
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    const int c4 = lig + v * LPR;
                    y[t][v] = (t < nh && c4 < w4 && index_ok(rk[t], p.y_rows, p.status, SITE_SPMM_POS)) ? __ldg(yr + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int t = 0; t < HB; ++t)
                if (t < nh) {
#pragma unroll
                    for (int v = 0; v < VPL; ++v) fma4(acc[v], ak[t], y[t][v]);
                }
        }
    }
    if (p.partial) {
        float4* dst = reinterpret_cast<float4*>(p.partial + idx * p.ldp);
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int c4 = lig + v * LPR;
            if (c4 < w4) dst[c4] = acc[v];
        }
        return;
    }
    if (p.out_mask && lig == 0 && p.j0 == 0) p.out_mask[u] = any ? 1 : 0;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int c4 = lig + v * LPR;
        if (c4 < w4) store_row(p, u, c4, acc[v]);
    }
}

// Row-filtered output: only the rows u with row_filter[u] != 0 are wanted (the last layer of a
// training step needs its output on train nodes only).  A warp scans 32 schedule records, tests the
// filter byte of each record's row and computes the kept ones one after the other with all 32 lanes,
// entries in the same order as spmm_group_kernel (bitwise the same rows).
template <int VPL>
__global__ void __launch_bounds__(256) spmm_filtered_kernel(const SpmmParams p) {
    const int lane = threadIdx.x & 31;
    const int64_t idx0 = p.idx_begin + ((((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5) << 5);
    if (idx0 >= p.idx_end) return;
    int4 rc = make_int4(0, 0, 0, 0);
    bool live = false;
    if (idx0 + lane < p.idx_end) {
        rc = __ldg(reinterpret_cast<const int4*>(p.rec + idx0 + lane));
        const int64_t b0 = ((int64_t)(uint32_t)rc.y << 32) | (uint32_t)rc.x;
        if (unit_ok(p, b0, b0 + rc.z, rc.w)) {
            const int64_t row = p.seg_perm ? __ldg(p.seg_perm + rc.w) : rc.w;
            live = index_ok(row, p.n_out, p.status, SITE_SPMM_ROW) && __ldg(p.row_filter + row) != 0;
        }
    }
    unsigned bits = __ballot_sync(0xFFFFFFFFu, live);
    const int w4 = (p.w + 3) >> 2;
    while (bits) {
        const int src = __ffs(bits) - 1;
        bits &= bits - 1;
        const uint32_t lo = (uint32_t)__shfl_sync(0xFFFFFFFFu, rc.x, src), hi = (uint32_t)__shfl_sync(0xFFFFFFFFu, rc.y, src);
        const int len = __shfl_sync(0xFFFFFFFFu, rc.z, src);
        const int64_t u = __shfl_sync(0xFFFFFFFFu, rc.w, src);
        const int64_t b = ((int64_t)hi << 32) | lo, e = b + len;
        float4 acc[VPL];
#pragma unroll
        for (int v = 0; v < VPL; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        row_segment<32, VPL>(p, b, e, lane, 0xFFFFFFFFu, w4, acc);
        if (p.partial) {
            float4* dst = reinterpret_cast<float4*>(p.partial + (idx0 + src) * p.ldp);
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                const int c4 = lane + v * 32;
                if (c4 < w4) dst[c4] = acc[v];
            }
        } else {
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                const int c4 = lane + v * 32;
                if (c4 < w4) store_row(p, u, c4, acc[v]);
            }
        }
    }
}

// Long rows: add the segments' partial rows in entry order, apply the epilogue, write Z.
// One group of 32 lanes per long row.
template <bool LOSS = false>
__global__ void __launch_bounds__(256) spmm_combine_kernel(const SpmmParams p, int64_t n_long,
                                                           const int64_t* __restrict__ seg_off,
                                                           const int64_t* __restrict__ seg_pos,
                                                           const int32_t* __restrict__ perm) {
    const int lane = threadIdx.x & 31;
    const int64_t i = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    if (i >= n_long) return;
    const int64_t s0 = seg_off[i], s1 = seg_off[i + 1];
    const int64_t u = perm[i];
    if (!index_ok(s0, p.n_partial + 1, p.status, SITE_SPMM_SEG) || !index_ok(s1, p.n_partial + 1, p.status, SITE_SPMM_SEG) ||
        !index_ok(u, p.n_out, p.status, SITE_SPMM_ROW)) return;
    if (p.row_filter && !__ldg(p.row_filter + u)) return;
    const int w4 = (p.w + 3) >> 2;
    if (p.out_mask && lane == 0) p.out_mask[u] = 1;    // long rows are kept without looking (conservative)
    if constexpr (LOSS) {
        // the whole row (at most 64 float4) in registers, then the same epilogue as the other rows
        float4 row[2];
#pragma unroll
        for (int v = 0; v < 2; ++v) {
            const int c4 = lane + v * 32;
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c4 < w4)
                for (int64_t q = s0; q < s1; ++q) {
                    const int64_t slot = __ldg(seg_pos + q);
                    if (!index_ok(slot, p.n_partial, p.status, SITE_SPMM_SEG)) continue;
                    const float4 t = __ldg(reinterpret_cast<const float4*>(p.partial + slot * p.ldp) + c4);
                    s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
                }
            row[v] = s;
        }
        loss_epilogue<32, 2>(p, u, lane, 0xFFFFFFFFu, row);
    } else {
        for (int c4 = lane; c4 < w4; c4 += 32) {
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int64_t q = s0; q < s1; ++q) {
                const int64_t slot = __ldg(seg_pos + q);
                if (!index_ok(slot, p.n_partial, p.status, SITE_SPMM_SEG)) continue;
                const float4 t = __ldg(reinterpret_cast<const float4*>(p.partial + slot * p.ldp) + c4);
                s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
            }
            store_row(p, u, c4, s);
        }
    }
}

template <int LPR, int VPL, bool LOSS = false>
void launch_group(const SpmmParams& p, cudaStream_t s) {
    const int64_t units = p.idx_end - p.idx_begin;
    if (units <= 0) return;
    const int per_block = 256 / LPR;
    const int64_t blocks = (units + per_block - 1) / per_block;
    // nothing between the sums and the stored row (or a partial row, which never has an epilogue): the plain instance
    // (one float4 per lane: the lean instances gain nothing there and the assembler spills a register in them)
    constexpr bool lean = !LOSS && VPL >= 2;
    if constexpr (lean) {
        const bool full = LPR >= 8 && ((p.w + 3) >> 2) == LPR * VPL;     // (narrow groups: nothing to gain)
        switch (pick_epi(p)) {
            case EPI_PLAIN:
                if (full) spmm_group_kernel<LPR, VPL, EPI_PLAIN, (LPR >= 8)><<<(unsigned)blocks, 256, 0, s>>>(p);
                else spmm_group_kernel<LPR, VPL, EPI_PLAIN><<<(unsigned)blocks, 256, 0, s>>>(p);
                return;
            case EPI_BITS:
                if (full) spmm_group_kernel<LPR, VPL, EPI_BITS, (LPR >= 8)><<<(unsigned)blocks, 256, 0, s>>>(p);
                else spmm_group_kernel<LPR, VPL, EPI_BITS><<<(unsigned)blocks, 256, 0, s>>>(p);
                return;
            case EPI_BIAS: spmm_group_kernel<LPR, VPL, EPI_BIAS><<<(unsigned)blocks, 256, 0, s>>>(p); return;
            case EPI_GATE: spmm_group_kernel<LPR, VPL, EPI_GATE><<<(unsigned)blocks, 256, 0, s>>>(p); return;
            default: break;
        }
    }
    spmm_group_kernel<LPR, VPL, LOSS ? EPI_LOSS : EPI_ANY><<<(unsigned)blocks, 256, 0, s>>>(p);
}

// The same packing for an aggregation with the loss epilogue (width <= 256: at most two float4 per lane
// before folding).  Returns 0 if the shape has no instance.
int dispatch_loss(const SpmmParams& p, int fold, cudaStream_t s) {
    const int w4 = (p.w + 3) >> 2;
    int lpr = 1;
    while (lpr < 32 && lpr < w4) lpr <<= 1;
    int vpl = (w4 + lpr - 1) / lpr;
    while (fold > 1 && (lpr / fold < 1 || vpl * fold > 8)) fold >>= 1;
    lpr /= fold; vpl *= fold;
#define MIXGCN_SPMM_CASE(L, V) if (lpr == L && vpl == V) { launch_group<L, V, true>(p, s); return fold; }
    MIXGCN_SPMM_CASE(32, 1) MIXGCN_SPMM_CASE(32, 2)
    MIXGCN_SPMM_CASE(16, 1) MIXGCN_SPMM_CASE(16, 2) MIXGCN_SPMM_CASE(16, 4)
    MIXGCN_SPMM_CASE(8, 1) MIXGCN_SPMM_CASE(8, 2) MIXGCN_SPMM_CASE(8, 4) MIXGCN_SPMM_CASE(8, 8)
    MIXGCN_SPMM_CASE(4, 1) MIXGCN_SPMM_CASE(4, 2) MIXGCN_SPMM_CASE(4, 4) MIXGCN_SPMM_CASE(4, 8)
    MIXGCN_SPMM_CASE(2, 1) MIXGCN_SPMM_CASE(2, 2) MIXGCN_SPMM_CASE(2, 4) MIXGCN_SPMM_CASE(2, 8)
    MIXGCN_SPMM_CASE(1, 1) MIXGCN_SPMM_CASE(1, 2) MIXGCN_SPMM_CASE(1, 4) MIXGCN_SPMM_CASE(1, 8)
#undef MIXGCN_SPMM_CASE
    return 0;
}

// Base configuration for a slice of w4 float4 columns, then packed `fold`-fold (fold in {1,2,4,8}):
// fewer lanes per row, more float4 per lane.  Returns the fold actually used.
int dispatch(const SpmmParams& p, int fold, cudaStream_t s) {
    const int w4 = (p.w + 3) >> 2;
    int lpr = 1;
    while (lpr < 32 && lpr < w4) lpr <<= 1;
    int vpl = (w4 + lpr - 1) / lpr;
    while (fold > 1 && (lpr / fold < 1 || vpl * fold > 8)) fold >>= 1;
    lpr /= fold; vpl *= fold;
#define MIXGCN_SPMM_CASE(L, V) if (lpr == L && vpl == V) { launch_group<L, V>(p, s); return fold; }
    MIXGCN_SPMM_CASE(32, 1) MIXGCN_SPMM_CASE(32, 2) MIXGCN_SPMM_CASE(32, 3) MIXGCN_SPMM_CASE(32, 4)
    MIXGCN_SPMM_CASE(32, 5) MIXGCN_SPMM_CASE(32, 6) MIXGCN_SPMM_CASE(32, 7) MIXGCN_SPMM_CASE(32, 8)
    MIXGCN_SPMM_CASE(16, 1) MIXGCN_SPMM_CASE(16, 2) MIXGCN_SPMM_CASE(16, 4) MIXGCN_SPMM_CASE(16, 6) MIXGCN_SPMM_CASE(16, 8)
    MIXGCN_SPMM_CASE(8, 1) MIXGCN_SPMM_CASE(8, 2) MIXGCN_SPMM_CASE(8, 4) MIXGCN_SPMM_CASE(8, 8)
    MIXGCN_SPMM_CASE(4, 1) MIXGCN_SPMM_CASE(4, 2) MIXGCN_SPMM_CASE(4, 4) MIXGCN_SPMM_CASE(4, 8)
    MIXGCN_SPMM_CASE(2, 1) MIXGCN_SPMM_CASE(2, 2) MIXGCN_SPMM_CASE(2, 4) MIXGCN_SPMM_CASE(2, 8)
    MIXGCN_SPMM_CASE(1, 1) MIXGCN_SPMM_CASE(1, 2) MIXGCN_SPMM_CASE(1, 4) MIXGCN_SPMM_CASE(1, 8)
#undef MIXGCN_SPMM_CASE
    return 0;
}

template <int LPR, int VPL>
void launch_sparse(const SpmmParams& p, cudaStream_t s) {
    const int64_t units = p.idx_end - p.idx_begin;
    if (units <= 0) return;
    const int per_block = 256 / LPR;
    spmm_sparse_kernel<LPR, VPL><<<(unsigned)((units + per_block - 1) / per_block), 256, 0, s>>>(p);
}

void dispatch_sparse(const SpmmParams& p, int fold, cudaStream_t s) {
    const int w4 = (p.w + 3) >> 2;
    int lpr = 1;
    while (lpr < 32 && lpr < w4) lpr <<= 1;
    int vpl = (w4 + lpr - 1) / lpr;
    while (fold > 1 && (lpr / fold < 1 || vpl * fold > 8)) fold >>= 1;
    lpr /= fold; vpl *= fold;
#define MIXGCN_SPMM_CASE(L, V) if (lpr == L && vpl == V) { launch_sparse<L, V>(p, s); return; }
    MIXGCN_SPMM_CASE(32, 1) MIXGCN_SPMM_CASE(32, 2) MIXGCN_SPMM_CASE(32, 3) MIXGCN_SPMM_CASE(32, 4)
    MIXGCN_SPMM_CASE(32, 5) MIXGCN_SPMM_CASE(32, 6) MIXGCN_SPMM_CASE(32, 7) MIXGCN_SPMM_CASE(32, 8)
    MIXGCN_SPMM_CASE(16, 1) MIXGCN_SPMM_CASE(16, 2) MIXGCN_SPMM_CASE(16, 4) MIXGCN_SPMM_CASE(16, 6) MIXGCN_SPMM_CASE(16, 8)
    MIXGCN_SPMM_CASE(8, 1) MIXGCN_SPMM_CASE(8, 2) MIXGCN_SPMM_CASE(8, 4) MIXGCN_SPMM_CASE(8, 8)
    MIXGCN_SPMM_CASE(4, 1) MIXGCN_SPMM_CASE(4, 2) MIXGCN_SPMM_CASE(4, 4) MIXGCN_SPMM_CASE(4, 8)
    MIXGCN_SPMM_CASE(2, 1) MIXGCN_SPMM_CASE(2, 2) MIXGCN_SPMM_CASE(2, 4) MIXGCN_SPMM_CASE(2, 8)
    MIXGCN_SPMM_CASE(1, 1) MIXGCN_SPMM_CASE(1, 2) MIXGCN_SPMM_CASE(1, 4) MIXGCN_SPMM_CASE(1, 8)
#undef MIXGCN_SPMM_CASE
}

void dispatch_filtered(const SpmmParams& p, cudaStream_t s) {
    const int64_t units = p.idx_end - p.idx_begin;
    if (units <= 0) return;
    const unsigned blocks = (unsigned)((units + 255) / 256);   // 8 warps x 32 records
    const int vpl = (((p.w + 3) >> 2) + 31) / 32;
    switch (vpl) {
#define MIXGCN_SPMM_CASE(V) case V: spmm_filtered_kernel<V><<<blocks, 256, 0, s>>>(p); break;
        MIXGCN_SPMM_CASE(1) MIXGCN_SPMM_CASE(2) MIXGCN_SPMM_CASE(3) MIXGCN_SPMM_CASE(4)
        MIXGCN_SPMM_CASE(5) MIXGCN_SPMM_CASE(6) MIXGCN_SPMM_CASE(7) MIXGCN_SPMM_CASE(8)
#undef MIXGCN_SPMM_CASE
        default: break;
    }
}

constexpr int MAX_SLICE = 1024;      // columns per launch at most: 8 float4 per lane
constexpr int DEFAULT_SLICE = 256;   // widths above this run as slices of this many columns (2 float4 per lane, four CTAs per SM)

}  // namespace

namespace mixgcn {

// Aggregation of all rows (chunks <= 1) or of row chunk k of `chunks` (the pipeline's chunks), each
// with its own schedule: long rows as column-ordered segments, then rows longest first, short rows packed.
mixgcn_status launch_spmm(mixgcn_ctx* ctx, const mixgcn_graph* g, const CsrView& A, int chunks, int k,
                          int32_t w, const float* Y, int64_t ldy, float* Z, int64_t ldz,
                          const mixgcn_epilogue* epi, cudaStream_t s, const SpmmOpts& opts) {
    const SpmmRowSparse* sparse = opts.sparse;
    const LossFuse* lf = opts.loss;
    const uint8_t* row_filter = opts.row_filter;
    const int phase = opts.phase;
    const int64_t row_limit = opts.row_limit;
    if (w <= 0) return MIXGCN_OK;
    if (!Z && !opts.Z_lp) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: no output");
    if (sparse && row_filter) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "spmm: a row filter cannot be combined with a row-sparse input");
    if (epi && epi->sign_bits && (row_filter || opts.row_limit >= 0 || lf || !Z))
        MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "spmm: the sign bitmap needs every row of a plain fp32 result");
    if (lf) {
        if (sparse || row_filter || chunks > 1 || opts.out_bits || opts.Z_lp || opts.row_limit >= 0 || !Z || w > 256 ||
            (epi && (epi->relu || epi->drop_mask || epi->gate || epi->residual)))
            MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "spmm: the loss epilogue takes a plain aggregation of at most 256 columns with a bias");
    }
    if (chunks > 1) {
        MIXGCN_TRY(ensure_chunk_schedules(g, A, chunks));
        if (k < 0 || k >= A.n_chunk) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: chunk %d of %d does not exist", k, chunks);
    }
    const SpmmSchedule& S = chunks > 1 ? A.chunk[k] : A.full;
    if (S.n_rows <= 0) return MIXGCN_OK;
    SpmmParams p{};
    p.rowptr = A.rowptr; p.col = A.col; p.val = A.val;
    p.Y = Y; p.ldy = ldy; p.Z = Z; p.ldz = ldz; p.w_total = w;
    p.Z_lp = opts.Z_lp; p.ldz_lp = opts.ldz_lp;
    p.out_bits = opts.out_bits; p.ld_bits = opts.ld_bits; p.bits_scale = 1.0f; p.bits_skip = 1;
    if (epi && epi->gate_bits) {
        // a bit-packed gate goes through the same bitmap path as the sampled aggregation's output mask
        if (opts.out_bits) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "spmm: a sampled aggregation takes no bit-packed gate as well");
        p.out_bits = epi->gate_bits; p.ld_bits = epi->ld_gate_bits; p.bits_scale = epi->gate_scale; p.bits_skip = 0;
    }
    if (epi) {
        p.bias = epi->bias; p.relu = epi->relu; p.drop = epi->drop_mask; p.keep_scale = epi->keep_scale;
        p.gate = epi->gate_bits ? nullptr : epi->gate; p.ld_gate = epi->ld_gate; p.gate_scale = epi->gate_scale;
        p.residual = epi->residual; p.ld_residual = epi->ld_residual; p.residual_scale = epi->residual_scale;
    }
    p.status = ctx->d_status;
    p.n_out = g->n; p.n_cols = g->n; p.y_rows = opts.y_rows >= 0 ? opts.y_rows : g->n;
    p.nnz = opts.nnz >= 0 ? opts.nnz : g->nnz;
    p.n_long = S.n_long; p.n_partial = S.total_segs;
    p.rec = S.rec;
    if (sparse) { p.in_mask = sparse->in_mask; p.in_pos = sparse->in_pos; p.out_mask = sparse->out_mask; }
    p.row_filter = row_filter;
    if (lf) {
        p.loss_labels = lf->labels; p.loss_mask = lf->train_mask; p.loss_count = lf->count;
        p.loss_row = lf->row_loss; p.loss_pred = lf->pred; p.loss_zero_rows = lf->zero_rows;
    }
    const int slice = lf ? MAX_SLICE : ctx->spmm_slice_cols > 0 ? (ctx->spmm_slice_cols < MAX_SLICE ? ctx->spmm_slice_cols : MAX_SLICE) : DEFAULT_SLICE;
    for (int j0 = 0; j0 < w; j0 += slice) {
        p.j0 = j0;
        p.w = (w - j0) < slice ? (w - j0) : slice;
        if (sparse) {
            // same units, sparse-input kernel: long-row segments to scratch + combine, then every other row
            if (S.total_segs > 0) {
                const int64_t ldp = ((int64_t)p.w + 3) / 4 * 4;
                MIXGCN_TRY(ensure_workspace_spmm(ctx, S.total_segs * ldp * (int64_t)sizeof(float)));
                p.partial = reinterpret_cast<float*>(ctx->workspace_spmm); p.ldp = ldp;
                {
                    LaunchScope scope(ctx, PH_SPMM_SPARSE, s);
                    p.idx_begin = 0; p.idx_end = S.total_segs;
                    dispatch_sparse(p, 1, s);
                }
                {
                    LaunchScope scope(ctx, PH_SPMM_SPARSE, s);
                    const int64_t blocks = (S.n_long * 32 + 255) / 256;
                    spmm_combine_kernel<false><<<(unsigned)blocks, 256, 0, s>>>(p, S.n_long, S.seg_off, S.seg_pos, S.perm);
                }
                p.partial = nullptr;
            }
            {
                // ordinary rows by degree bucket, short rows packed 2/4/8 per warp as in the dense path
                int64_t bnd[5];
                bnd[0] = S.n_long;
                for (int q = 0; q < 3; ++q) bnd[q + 1] = S.rows_above[q] > S.n_long ? S.rows_above[q] : S.n_long;
                bnd[4] = S.n_rows;
                int64_t begin = bnd[0];
                int fold = 1;
                for (int q = 0; q < 4; ++q, fold <<= 1) {
                    const int64_t end = bnd[q + 1];
                    if (end <= begin) continue;
                    p.idx_begin = S.total_segs + (begin - S.n_long);
                    p.idx_end = S.total_segs + (end - S.n_long);
                    LaunchScope scope(ctx, PH_SPMM_SPARSE, s);
                    dispatch_sparse(p, fold, s);
                    begin = end;
                }
            }
            continue;
        }
        if (row_filter) {
            // kept rows only: segments of kept long rows, their combination, then every other kept row
            if (S.total_segs > 0) {
                const int64_t ldp = ((int64_t)p.w + 3) / 4 * 4;
                MIXGCN_TRY(ensure_workspace_spmm(ctx, S.total_segs * ldp * (int64_t)sizeof(float)));
                p.partial = reinterpret_cast<float*>(ctx->workspace_spmm); p.ldp = ldp;
                {
                    LaunchScope scope(ctx, PH_SPMM_SPARSE, s);
                    p.idx_begin = 0; p.idx_end = S.total_segs;
                    p.seg_perm = S.perm;
                    dispatch_filtered(p, s);
                    p.seg_perm = nullptr;
                }
                {
                    LaunchScope scope(ctx, PH_SPMM_SPARSE, s);
                    const int64_t blocks = (S.n_long * 32 + 255) / 256;
                    spmm_combine_kernel<false><<<(unsigned)blocks, 256, 0, s>>>(p, S.n_long, S.seg_off, S.seg_pos, S.perm);
                }
                p.partial = nullptr;
            }
            if (S.n_rows > S.n_long) {
                LaunchScope scope(ctx, PH_SPMM_SPARSE, s);
                p.idx_begin = S.total_segs; p.idx_end = S.total_segs + (S.n_rows - S.n_long);
                dispatch_filtered(p, s);
            }
            continue;
        }
        if (S.total_segs > 0) {
            const int64_t ldp = ((int64_t)p.w + 3) / 4 * 4;
            MIXGCN_TRY(ensure_workspace_spmm(ctx, S.total_segs * ldp * (int64_t)sizeof(float)));
            p.partial = reinterpret_cast<float*>(ctx->workspace_spmm); p.ldp = ldp;
            {
                LaunchScope scope(ctx, phase, s);
                p.idx_begin = 0; p.idx_end = S.total_segs;
                if (p.out_bits && p.bits_skip) p.seg_perm = S.perm;       // a segment's record names its long row by ordinal
                dispatch(p, p.w <= SPMM_FOLD_WMAX ? SPMM_FOLD_SEG : 1, s);
                p.seg_perm = nullptr;
            }
            {
                LaunchScope scope(ctx, phase, s);
                const int64_t blocks = (S.n_long * 32 + 255) / 256;
                if (lf) spmm_combine_kernel<true><<<(unsigned)blocks, 256, 0, s>>>(p, S.n_long, S.seg_off, S.seg_pos, S.perm);
                else spmm_combine_kernel<false><<<(unsigned)blocks, 256, 0, s>>>(p, S.n_long, S.seg_off, S.seg_pos, S.perm);
            }
            p.partial = nullptr;
        }
        // ordinary rows, in perm order: [n_long, n_rows) -> records [total_segs, total_segs + n_rows - n_long)
        int64_t bound[5];
        bound[0] = S.n_long;
        for (int q = 0; q < 3; ++q) bound[q + 1] = S.rows_above[q] > S.n_long ? S.rows_above[q] : S.n_long;
        bound[4] = S.n_rows;
        if (row_limit >= 0 && row_limit < S.n_rows) {
            // rows come longest first: only the first row_limit of them are wanted (the rest are empty)
            const int64_t lim = row_limit > S.n_long ? row_limit : S.n_long;
            for (int q = 1; q < 5; ++q) if (bound[q] > lim) bound[q] = lim;
        }
        int64_t begin = bound[0];
        int fold = 1;
        for (int q = 0; q < 4; ++q, fold <<= 1) {
            int64_t end = bound[q + 1];
            if (end <= begin) continue;
            p.idx_begin = S.total_segs + (begin - S.n_long);
            p.idx_end = S.total_segs + (end - S.n_long);
            LaunchScope scope(ctx, phase, s);
            if (lf) {
                if (!dispatch_loss(p, q == 0 ? (p.w <= SPMM_FOLD_WMAX ? SPMM_FOLD_MED : 1) : fold, s)) MIXGCN_FAIL(MIXGCN_EUNSUPPORTED, "spmm: no loss-epilogue kernel for width %d", p.w);
            } else if (q == 3 && p.w <= 128 && SPMM_PACK_DEG[2] <= SPMM_SHORT_MAXE) {
                // rows of at most SPMM_PACK_DEG[2] entries: several rows per warp, whole-warp gathers
                constexpr int RB = SPMM_SHORT_RB, MAXE = SPMM_SHORT_MAXE;
                const int64_t units = p.idx_end - p.idx_begin;
                const int64_t warps = (units + RB - 1) / RB;
                const unsigned grid_short = (unsigned)((warps + 7) / 8);
                const int epi_short = pick_epi(p);
                if (epi_short == EPI_PLAIN) spmm_short_kernel<RB, MAXE, EPI_PLAIN><<<grid_short, 256, 0, s>>>(p);
                else if (epi_short == EPI_BITS) spmm_short_kernel<RB, MAXE, EPI_BITS><<<grid_short, 256, 0, s>>>(p);
                else if (epi_short == EPI_BIAS) spmm_short_kernel<RB, MAXE, EPI_BIAS><<<grid_short, 256, 0, s>>>(p);
                else if (epi_short == EPI_GATE) spmm_short_kernel<RB, MAXE, EPI_GATE><<<grid_short, 256, 0, s>>>(p);
                else spmm_short_kernel<RB, MAXE, EPI_ANY><<<grid_short, 256, 0, s>>>(p);
            } else if (q == 3 && p.w <= 256 && SPMM_PACK_DEG[2] <= SPMM_SHORT_MAXE) {
                // the same for widths up to 256: two float4 per lane, two rows per warp
                constexpr int RB = SPMM_SHORT_RB / 2, MAXE = SPMM_SHORT_MAXE;
                const int64_t units = p.idx_end - p.idx_begin;
                const int64_t warps = (units + RB - 1) / RB;
                const unsigned grid_short = (unsigned)((warps + 7) / 8);
                const int epi_short = pick_epi(p);
                if (epi_short == EPI_PLAIN) spmm_short_kernel<RB, MAXE, EPI_PLAIN, 2><<<grid_short, 256, 0, s>>>(p);
                else if (epi_short == EPI_BITS) spmm_short_kernel<RB, MAXE, EPI_BITS, 2><<<grid_short, 256, 0, s>>>(p);
                else if (epi_short == EPI_BIAS) spmm_short_kernel<RB, MAXE, EPI_BIAS, 2><<<grid_short, 256, 0, s>>>(p);
                else if (epi_short == EPI_GATE) spmm_short_kernel<RB, MAXE, EPI_GATE, 2><<<grid_short, 256, 0, s>>>(p);
                else spmm_short_kernel<RB, MAXE, EPI_ANY, 2><<<grid_short, 256, 0, s>>>(p);
            } else {
                dispatch(p, q == 0 ? (p.w <= SPMM_FOLD_WMAX ? SPMM_FOLD_MED : 1) : fold, s);
            }
            begin = end;
        }
    }
    MIXGCN_CUDA(cudaGetLastError());
    // sign bitmap of the result: one more pass over the rows this call wrote
    if (epi && epi->sign_bits)
        MIXGCN_TRY(launch_mask_pack(ctx, S.n_rows, w, Z + S.row0 * ldz, ldz, nullptr, epi->sign_bits + S.row0 * epi->ld_sign_bits,
                                    epi->ld_sign_bits, s));
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
    if (epi && epi->residual && (epi->ld_residual < w || epi->residual == Z)) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: residual needs ld_residual >= w and must not be the output");
    if (epi && ((epi->gate_bits && epi->ld_gate_bits < (w + 31) / 32) || (epi->sign_bits && epi->ld_sign_bits < (w + 31) / 32)))
        MIXGCN_FAIL(MIXGCN_EINVAL, "spmm: a bit-packed mask needs ld >= ceil(w / 32) words");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    return launch_spmm(ctx, g, transposed ? g->bwd : g->fwd, 1, 0, w, Y, ldy, Z, ldz, epi, (cudaStream_t)stream);
}

namespace {

// bits[u][j] = (X == null || X[u][j] > 0) && (bytes == null || bytes[u*w + j] != 0): one thread per 32-bit word
__global__ void mask_pack_kernel(int64_t n, int w, const float* __restrict__ X, int64_t ldx, const uint8_t* __restrict__ bytes,
                                 uint32_t* __restrict__ bits, int64_t ld_bits) {
    const int words = (w + 31) >> 5;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n * words) return;
    const int64_t u = t / words; const int wd = (int)(t % words);
    uint32_t out = 0;
    for (int b = 0; b < 32; ++b) {
        const int j = wd * 32 + b;
        if (j >= w) break;
        bool on = true;
        if (X) on = X[u * ldx + j] > 0.0f;
        if (bytes) on = on && bytes[u * (int64_t)w + j] != 0;
        out |= (on ? 1u : 0u) << b;
    }
    bits[u * ld_bits + wd] = out;
}

}  // namespace

namespace mixgcn {
mixgcn_status launch_mask_pack(mixgcn_ctx* ctx, int64_t n, int32_t w, const float* X, int64_t ldx, const uint8_t* bytes,
                               uint32_t* bits, int64_t ld_bits, cudaStream_t s) {
    if (n <= 0 || w <= 0) return MIXGCN_OK;
    const int64_t total = n * ((w + 31) / 32);
    LaunchScope scope(ctx, PH_ELEM, s);
    mask_pack_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(n, w, X, ldx, bytes, bits, ld_bits);
    MIXGCN_CUDA(cudaGetLastError());
    return MIXGCN_OK;
}
}  // namespace mixgcn

extern "C" mixgcn_status mixgcn_mask_pack(mixgcn_ctx* ctx, int64_t n, int32_t w, const float* X, int64_t ldx,
                                          const uint8_t* bytes, uint32_t* bits, int64_t ld_bits, void* stream) {
    if (!ctx || !bits || (!X && !bytes)) MIXGCN_FAIL(MIXGCN_EINVAL, "mask_pack: null argument");
    if (n <= 0 || w <= 0 || ld_bits < (w + 31) / 32 || (X && ldx < w)) MIXGCN_FAIL(MIXGCN_EINVAL, "mask_pack: need n, w > 0, ld_bits >= ceil(w/32), ldx >= w");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    return launch_mask_pack(ctx, n, w, X, ldx, bytes, bits, ld_bits, (cudaStream_t)stream);
}

extern "C" mixgcn_status mixgcn_spmm_sampled(mixgcn_ctx* ctx, const mixgcn_graph* g, int transposed, int32_t w,
                                             const float* Y, int64_t ldy, float* Z, int64_t ldz, const uint32_t* mask_bits,
                                             int64_t ld_bits, const mixgcn_epilogue* epi, void* stream) {
    if (!ctx || !g || !Y || !Z || !mask_bits) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_sampled: null argument");
    if (w <= 0) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_sampled: w must be positive (got %d)", w);
    if (ldy < w || ldz < w || (ldy & 3) || (ldz & 3) || ld_bits < (w + 31) / 32)
        MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_sampled: leading dimensions must be multiples of 4 and >= w, ld_bits >= ceil(w/32)");
    if (!aligned16(Y) || !aligned16(Z)) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_sampled: Y and Z must be 16-byte aligned");
    if (Y == Z) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_sampled: Y and Z must not overlap");
    if (epi && epi->gate && epi->ld_gate < w) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_sampled: gate leading dimension < w");
    if (epi && epi->residual && (epi->ld_residual < w || epi->residual == Z)) MIXGCN_FAIL(MIXGCN_EINVAL, "spmm_sampled: residual needs ld_residual >= w and must not be the output");
    MIXGCN_CUDA(cudaSetDevice(ctx->device));
    SpmmOpts opts; opts.out_bits = mask_bits; opts.ld_bits = ld_bits;
    return launch_spmm(ctx, g, transposed ? g->bwd : g->fwd, 1, 0, w, Y, ldy, Z, ldz, epi, (cudaStream_t)stream, opts);
}
