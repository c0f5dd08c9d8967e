/*
 * gcn_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, obviously-correct CPU statement of full-graph GCN training as the MixGCN
 * paper defines it: propagation matrix (Section 2.1), layer forward (Eq. 3; Algorithm 2,
 * aggregation line then update line), loss / backward / weight update (Algorithm 2, last two
 * lines of the iteration body).  Every tensor is fp64; loops are written in definition order
 * with no blocking, fusion or reordering.  `#pragma omp parallel for` over independent output
 * rows is the only concession to speed (it does not change any sum's order).
 *
 * Only tests, the smoke check and the benchmark's cpu-baseline leg may call this file.  It
 * shares no code, header, table or helper with the CUDA library and never reads its outputs.
 *
 * Notation: node-major X = H^T (n x d, row-major, leading dimension given), W_l = [W^(l)]^T
 * (d_in x d_out, row-major).  Eq. 3 then reads X' = sigma(A_hat X W + 1 b^T).
 *
 * Pins (tests/test_oracle_pins.py): dense brute force on graphs of <= 64 nodes, closed forms
 * (complete graph => J/n, regular graphs, star, path, edgeless), scipy/numpy library routines,
 * adjoint identity, ln C loss, finite-difference gradients, closed-form Adam steps.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_SYMMETRISE 1u
#define ORACLE_ADD_SELF_LOOPS 2u

static int cmp_i32(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

/*
 * A_tilde = A + I (Section 2.1) from an edge list.  Input self-loops are ignored, each edge
 * (src,dst) = (u,v) stores entry (u,v) [and (v,u) when symmetrising], duplicates collapse
 * (A is binary), and one diagonal entry per node is added.  Output is row-wise sorted
 * neighbour lists, i.e. CSR.  Call with col == NULL to obtain rowptr and the entry count
 * first.  Returns nnz, or -1 on an id outside [0,n), -2 on allocation failure.
 */
int64_t oracle_graph_build(int64_t n, int64_t m, const int32_t* src, const int32_t* dst,
                           uint32_t flags, int64_t* rowptr, int32_t* col) {
    const int sym = (flags & ORACLE_SYMMETRISE) != 0, self = (flags & ORACLE_ADD_SELF_LOOPS) != 0;
    int64_t* cnt = (int64_t*)calloc((size_t)n + 1, sizeof(int64_t));
    if (!cnt) return -2;
    for (int64_t e = 0; e < m; ++e) {
        int32_t u = src[e], v = dst[e];
        if (u < 0 || v < 0 || u >= n || v >= n) { free(cnt); return -1; }
        if (u == v) continue;
        cnt[u + 1]++;
        if (sym) cnt[v + 1]++;
    }
    if (self) for (int64_t u = 0; u < n; ++u) cnt[u + 1]++;
    for (int64_t u = 0; u < n; ++u) cnt[u + 1] += cnt[u];
    int64_t total = cnt[n];
    int32_t* raw = (int32_t*)malloc((size_t)(total > 0 ? total : 1) * sizeof(int32_t));
    int64_t* pos = (int64_t*)malloc((size_t)(n + 1) * sizeof(int64_t));
    if (!raw || !pos) { free(cnt); free(raw); free(pos); return -2; }
    memcpy(pos, cnt, (size_t)(n + 1) * sizeof(int64_t));
    for (int64_t e = 0; e < m; ++e) {
        int32_t u = src[e], v = dst[e];
        if (u == v) continue;
        raw[pos[u]++] = v;
        if (sym) raw[pos[v]++] = u;
    }
    if (self) for (int64_t u = 0; u < n; ++u) raw[pos[u]++] = (int32_t)u;
    int64_t nnz = 0;
    rowptr[0] = 0;
    for (int64_t u = 0; u < n; ++u) {
        int64_t b = cnt[u], e = cnt[u + 1];
        qsort(raw + b, (size_t)(e - b), sizeof(int32_t), cmp_i32);
        for (int64_t i = b; i < e; ++i) {
            if (i > b && raw[i] == raw[i - 1]) continue;
            if (col) col[nnz] = raw[i];
            nnz++;
        }
        rowptr[u + 1] = nnz;
    }
    free(cnt); free(raw); free(pos);
    return nnz;
}

/*
 * Structure of the transposed matrix, built on its own by a counting sort over columns (not
 * by assuming symmetry).  src_index[j] is the position in the original arrays of transposed
 * entry j, so a value array can be carried over.
 */
void oracle_transpose(int64_t n, const int64_t* rowptr, const int32_t* col,
                      int64_t* rowptr_t, int32_t* col_t, int64_t* src_index) {
    for (int64_t u = 0; u <= n; ++u) rowptr_t[u] = 0;
    for (int64_t i = 0; i < rowptr[n]; ++i) rowptr_t[col[i] + 1]++;
    for (int64_t u = 0; u < n; ++u) rowptr_t[u + 1] += rowptr_t[u];
    int64_t* pos = (int64_t*)malloc((size_t)(n + 1) * sizeof(int64_t));
    memcpy(pos, rowptr_t, (size_t)(n + 1) * sizeof(int64_t));
    for (int64_t u = 0; u < n; ++u)
        for (int64_t i = rowptr[u]; i < rowptr[u + 1]; ++i) {
            int64_t j = pos[col[i]]++;
            col_t[j] = (int32_t)u;
            src_index[j] = i;
        }
    free(pos);
}

/*
 * A_hat = D^-1/2 A_tilde D^-1/2 with D_uu = sum_v A_tilde_uv (Section 2.1): the row sum of a
 * binary matrix is the row's entry count.  val64 is the fp64 definition.  dinv32 / val32
 * follow the fp32 storage recipe (dinv = 1/sqrt(deg) rounded to fp32 after each IEEE
 * operation, val = dinv_u * dinv_v) for bit-level comparison of stored values.
 */
void oracle_normalise(int64_t n, const int64_t* rowptr, const int32_t* col,
                      double* val64, float* dinv32, float* val32, int32_t* deg) {
    for (int64_t u = 0; u < n; ++u) {
        int64_t d = rowptr[u + 1] - rowptr[u];
        if (deg) deg[u] = (int32_t)d;
        if (dinv32) {
            volatile float s = sqrtf((float)d);
            volatile float r = 1.0f / s;
            dinv32[u] = r;
        }
    }
    for (int64_t u = 0; u < n; ++u) {
        double du = (double)(rowptr[u + 1] - rowptr[u]);
        for (int64_t i = rowptr[u]; i < rowptr[u + 1]; ++i) {
            int64_t v = col[i];
            double dv = (double)(rowptr[v + 1] - rowptr[v]);
            if (val64) val64[i] = 1.0 / sqrt(du * dv);
            if (val32) { volatile float p = dinv32[u] * dinv32[v]; val32[i] = p; }
        }
    }
}

/* Other aggregators on the same stored structure.  The paper evaluates GraphSAGE and GIN besides
 * GCN (Section 5, "The Model and Datasets") without defining them; these are their textbook
 * aggregation matrices: mode 1 = row mean, val_uv = 1 / (entries in row u) (GraphSAGE's mean
 * aggregator), mode 2 = plain sum, val_uv = 1 (GIN's sum aggregator).  val32 follows the fp32
 * storage recipe: one IEEE division of 1 by the entry count. */
void oracle_normalise_mode(int64_t n, const int64_t* rowptr, int32_t mode, double* val64, float* val32) {
    for (int64_t u = 0; u < n; ++u) {
        int64_t d = rowptr[u + 1] - rowptr[u];
        for (int64_t i = rowptr[u]; i < rowptr[u + 1]; ++i) {
            if (mode == 1) {
                if (val64) val64[i] = 1.0 / (double)d;
                if (val32) { volatile float r = 1.0f / (float)d; val32[i] = r; }
            } else {
                if (val64) val64[i] = 1.0;
                if (val32) val32[i] = 1.0f;
            }
        }
    }
}

/* Neighbour aggregation Z = A_hat X (Algorithm 2, aggregation line): row u of Z is the
 * weighted sum of the rows of X listed in row u of the matrix, in ascending column order. */
void oracle_aggregate(int64_t n, const int64_t* rowptr, const int32_t* col, const double* val,
                      int64_t d, const double* X, int64_t ldx, double* Z, int64_t ldz) {
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t u = 0; u < n; ++u) {
        for (int64_t j = 0; j < d; ++j) Z[u * ldz + j] = 0.0;
        for (int64_t i = rowptr[u]; i < rowptr[u + 1]; ++i) {
            const double a = val[i];
            const double* x = X + (int64_t)col[i] * ldx;
            for (int64_t j = 0; j < d; ++j) Z[u * ldz + j] += a * x[j];
        }
    }
}

/* The same sum for a chosen list of rows only: out[r,:] = (A_hat X)[rows[r],:]. */
void oracle_aggregate_rows(int64_t nrows, const int64_t* rows, const int64_t* rowptr,
                           const int32_t* col, const double* val, int64_t d,
                           const double* X, int64_t ldx, double* out) {
    for (int64_t r = 0; r < nrows; ++r) {
        int64_t u = rows[r];
        for (int64_t j = 0; j < d; ++j) out[r * d + j] = 0.0;
        for (int64_t i = rowptr[u]; i < rowptr[u + 1]; ++i)
            for (int64_t j = 0; j < d; ++j) out[r * d + j] += val[i] * X[(int64_t)col[i] * ldx + j];
    }
}

/* Node update before the activation, P = Z W + 1 b^T (Algorithm 2, update line; bias is
 * optional and absent from Eq. 3). */
void oracle_update(int64_t n, int64_t d_in, int64_t d_out, const double* Z, const double* W,
                   const double* bias, double* P) {
#pragma omp parallel for schedule(static)
    for (int64_t u = 0; u < n; ++u)
        for (int64_t j = 0; j < d_out; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < d_in; ++k) acc += Z[u * d_in + k] * W[k * d_out + j];
            P[u * d_out + j] = acc + (bias ? bias[j] : 0.0);
        }
}

/* X' = mask * keep_scale * sigma(P) with sigma = ReLU (Eq. 3); relu == 0 gives X' = P on the
 * last layer.  mask (0/1 bytes, optional) is a caller-drawn dropout mask. */
void oracle_activation(int64_t n, int64_t d_out, const double* P, int relu, const uint8_t* mask,
                       double keep_scale, double* Xout) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n * d_out; ++i) {
        double x = P[i];
        if (relu && !(x > 0.0)) x = 0.0;
        if (mask) x = mask[i] ? x * keep_scale : 0.0;
        Xout[i] = x;
    }
}

/*
 * Masked softmax cross-entropy (the loss line of Algorithm 2, with the mean-over-train-nodes,
 * natural-log reading): loss = -(1/#T) sum_{v in T} log softmax(P_v)[y_v];
 * G_v = (softmax(P_v) - e_{y_v}) / #T on T, 0 elsewhere; pred_v = first index of the row
 * maximum.  Returns #T (0 => loss and G are left as zeros).
 */
int64_t oracle_loss(int64_t n, int64_t C, const double* P, const int32_t* labels,
                    const uint8_t* train_mask, double* loss, double* G, int32_t* pred,
                    int64_t* n_correct) {
    int64_t T = 0, correct = 0;
    for (int64_t v = 0; v < n; ++v) T += train_mask[v] ? 1 : 0;
    double total = 0.0;
    for (int64_t v = 0; v < n; ++v) {
        const double* p = P + v * C;
        int64_t arg = 0;
        double mx = p[0];
        for (int64_t c = 1; c < C; ++c) if (p[c] > mx) { mx = p[c]; arg = c; }
        if (pred) pred[v] = (int32_t)arg;
        if (G) for (int64_t c = 0; c < C; ++c) G[v * C + c] = 0.0;
        if (!train_mask[v] || T == 0) continue;
        if (arg == labels[v]) correct++;
        double s = 0.0;
        for (int64_t c = 0; c < C; ++c) s += exp(p[c] - mx);
        double lse = mx + log(s);
        total += lse - p[labels[v]];
        if (G) for (int64_t c = 0; c < C; ++c)
            G[v * C + c] = (exp(p[c] - lse) - (c == labels[v] ? 1.0 : 0.0)) / (double)T;
    }
    *loss = T ? total / (double)T : 0.0;
    if (n_correct) *n_correct = correct;
    return T;
}

/*
 * Backward of one layer's update by the chain rule on X' = mask*keep_scale*ReLU(P),
 * P = Z W + 1 b^T:  dP = G' * mask*keep_scale * 1[P>0];  dW = Z^T dP;  db = column sums of
 * dP;  dZ = dP W^T (skipped when dZ == NULL: the first layer needs no input gradient).
 * The input gradient dX = A_hat^T dZ is then an oracle_aggregate call on the transposed
 * structure.
 */
void oracle_update_bwd(int64_t n, int64_t d_in, int64_t d_out, const double* Z, const double* P,
                       const double* W, const double* Gout, int relu, const uint8_t* mask,
                       double keep_scale, double* dP, double* dW, double* db, double* dZ) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n * d_out; ++i) {
        double g = Gout[i];
        if (mask) g = mask[i] ? g * keep_scale : 0.0;
        if (relu && !(P[i] > 0.0)) g = 0.0;
        dP[i] = g;
    }
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < d_in; ++k)
        for (int64_t j = 0; j < d_out; ++j) {
            double acc = 0.0;
            for (int64_t u = 0; u < n; ++u) acc += Z[u * d_in + k] * dP[u * d_out + j];
            dW[k * d_out + j] = acc;
        }
    if (db)
        for (int64_t j = 0; j < d_out; ++j) {
            double acc = 0.0;
            for (int64_t u = 0; u < n; ++u) acc += dP[u * d_out + j];
            db[j] = acc;
        }
    if (dZ) {
#pragma omp parallel for schedule(static)
        for (int64_t u = 0; u < n; ++u)
            for (int64_t k = 0; k < d_in; ++k) {
                double acc = 0.0;
                for (int64_t j = 0; j < d_out; ++j) acc += dP[u * d_out + j] * W[k * d_out + j];
                dZ[u * d_in + k] = acc;
            }
    }
}

/* Adam, bias-corrected, epsilon added after the square root of the corrected second moment,
 * t counted from 1, no weight decay (the "update weight" step of Algorithm 2). */
void oracle_adam(int64_t numel, double* theta, const double* g, double* m, double* v, int64_t t,
                 double lr, double beta1, double beta2, double eps) {
    const double c1 = 1.0 - pow(beta1, (double)t), c2 = 1.0 - pow(beta2, (double)t);
    for (int64_t i = 0; i < numel; ++i) {
        m[i] = beta1 * m[i] + (1.0 - beta1) * g[i];
        v[i] = beta2 * v[i] + (1.0 - beta2) * g[i] * g[i];
        theta[i] -= lr * (m[i] / c1) / (sqrt(v[i] / c2) + eps);
    }
}

/* ------------------------------------------------------------------------------------------------
 * Node reordering for the fine-grain pipeline (Section 3.2.2).
 * ------------------------------------------------------------------------------------------------ */

/* Graph bandwidth b = max over stored entries (u,v) of p_v - p_u, p = position in the processing
 * sequence (pos == NULL: identity). */
int64_t oracle_bandwidth(int64_t n, const int64_t* rowptr, const int32_t* col, const int64_t* pos) {
    int64_t b = 0;
    for (int64_t u = 0; u < n; ++u)
        for (int64_t i = rowptr[u]; i < rowptr[u + 1]; ++i) {
            int64_t pu = pos ? pos[u] : u, pv = pos ? pos[col[i]] : col[i];
            if (pv - pu > b) b = pv - pu;
        }
    return b;
}

/* Reverse Cuthill-McKee on a symmetric structure: components are started from the unvisited node of
 * fewest entries (lowest id on ties); a dequeued node appends its unvisited neighbours by increasing
 * entry count (lowest id on ties); the resulting sequence is reversed.  order[k] = node at position k. */
void oracle_rcm(int64_t n, const int64_t* rowptr, const int32_t* col, int64_t* order) {
    char* seen = (char*)calloc((size_t)n, 1);
    int64_t* byd = (int64_t*)malloc((size_t)n * sizeof(int64_t));
    int64_t* tmp = (int64_t*)malloc((size_t)n * sizeof(int64_t));
    int64_t head = 0, tail = 0, next_start = 0;
    /* nodes by (entry count, id): counting sort on the entry count */
    int64_t maxd = 0;
    for (int64_t u = 0; u < n; ++u) { int64_t d = rowptr[u + 1] - rowptr[u]; if (d > maxd) maxd = d; }
    int64_t* cnt = (int64_t*)calloc((size_t)maxd + 2, sizeof(int64_t));
    for (int64_t u = 0; u < n; ++u) cnt[rowptr[u + 1] - rowptr[u] + 1]++;
    for (int64_t d = 0; d <= maxd; ++d) cnt[d + 1] += cnt[d];
    for (int64_t u = 0; u < n; ++u) byd[cnt[rowptr[u + 1] - rowptr[u]]++] = u;
    while (tail < n) {
        while (seen[byd[next_start]]) ++next_start;
        int64_t s = byd[next_start];
        seen[s] = 1; order[tail++] = s;
        while (head < tail) {
            int64_t x = order[head++];
            int64_t m = 0;
            for (int64_t i = rowptr[x]; i < rowptr[x + 1]; ++i) {
                int64_t y = col[i];
                if (!seen[y]) { seen[y] = 1; tmp[m++] = y; }
            }
            /* insertion sort by entry count; the list is in ascending id, so ties keep the lower id first */
            for (int64_t a = 1; a < m; ++a) {
                int64_t y = tmp[a], dy = rowptr[y + 1] - rowptr[y], b = a;
                while (b > 0 && rowptr[tmp[b - 1] + 1] - rowptr[tmp[b - 1]] > dy) { tmp[b] = tmp[b - 1]; --b; }
                tmp[b] = y;
            }
            for (int64_t a = 0; a < m; ++a) order[tail++] = tmp[a];
        }
    }
    for (int64_t a = 0, b = n - 1; a < b; ++a, --b) { int64_t t = order[a]; order[a] = order[b]; order[b] = t; }
    free(seen); free(byd); free(tmp); free(cnt);
}

/* Proposition 3.5: with s batches idleness disappears when (n - b) / (2n) >= 1 / s; the stage count
 * the evaluation uses is the smallest such s, ceil(2n / (n - b)).  Returns -1 when b >= n. */
int64_t oracle_pipeline_stages(int64_t n, int64_t b) {
    if (b >= n) return -1;
    return (2 * n + (n - b) - 1) / (n - b);
}
