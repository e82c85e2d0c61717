/*
 * CPU oracle for the GAD training epoch (arXiv 2110.02987).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, double-precision restatement of what
 * the paper's training loop computes, used only to check the CUDA library and to be timed
 * beside it as a CPU baseline.  It shares no code with the CUDA library and the library
 * never calls it.
 *
 * What it follows (all section / equation numbers are the paper's):
 *   - augmented subgraph g'_i = (v_i + v'_i, e_i + e'_i)            Algorithm 1, last step
 *   - layer  H^(l+1) = sigma(A~ . H^(l) . W^(l))                    Section 3.3, forward equation
 *   - two-layer stack with softmax on top                            Section 3.3, second equation
 *   - loss / gradient                                               Section 3.3, loss and gradient equations
 *   - global consensus (plain average)                              Definition 3
 *   - update W = W - eta * gradient                                 Section 3.3 update equation
 *   - variance-based importance zeta(g')                            Section 3.4.1 (with its worked example)
 *   - weighted global consensus                                     Section 3.4.2
 *   - whole loop                                                    Algorithm 2
 *
 * Readings taken where the paper is silent or garbled (each is also listed in the design notes):
 *   - A~ is the symmetric normalisation D~^-1/2 (A+I) D~^-1/2 of Kipf and Welling, with the degrees
 *     taken inside each augmented subgraph; the subgraph keeps every edge of G whose two endpoints
 *     are both in v_i + v'_i.
 *   - the loss is multi-class softmax cross-entropy, averaged over the training nodes among the
 *     subgraph's own (non-replicated) nodes; replicated nodes only feed aggregation.
 *   - p(v_i) = local degree / sum of local degrees, unordered pairs, beta = 1 (fixed by the worked
 *     example); the distance term is the p-weighted RMS pairwise Euclidean distance of the input
 *     features ("aggregate" reading), or the literal pairwise form ("pairwise" reading); with
 *     zeta_mode 2 the aggregate reading keeps the sum over the layers of the variance equation: the
 *     squared distance is summed over the inputs H^(0) .. H^(L-1) of all layers (the activations of the
 *     most recent forward pass).
 *   - each processor takes one SGD step on its own copy, then the copies are replaced by their
 *     zeta-weighted mean; from identical copies this equals applying the weighted mean gradient.
 *   - the ReLU of the forward equation has a kink at 0: a hidden unit whose pre-activation is zero
 *     within rounding may be "on" in one arithmetic and "off" in another, and both are valid results.
 *     A caller comparing another implementation with this one may prescribe the branch of such units
 *     (orc_set_relu_branch), so that both sides take that decision alike; nothing else is affected.
 *
 * Pins: see tests/test_oracle_*.py (dense brute force, finite differences, the paper's printed
 * zeta values, Property 2, closed forms, special cases).  Parity unpinned (readings, not facts):
 * the choice between the aggregate and pairwise distance term when distances differ, whether the sum
 * over layers is kept (zeta_mode 2) or not, local versus global degrees in A~, induced halo-halo edges,
 * loss on core nodes only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_RANGE (-2)
#define ORC_ERR_DUPLICATE (-4)
#define ORC_ERR_OOM (-5)

/* ------------------------------------------------------------------------------------------
 * a1.  Block-diagonal store of the K augmented subgraphs.
 * Local ids of subgraph k: its core nodes in the given order, then its replicated nodes in the
 * given order.  Row r of the store is (k, local id) with r = sub_off[k] + local id; columns are
 * stored as store-row ids, ascending inside a row.
 * ---------------------------------------------------------------------------------------- */

typedef struct { int32_t c; double w; } orc_ent;

static int ent_cmp(const void* a, const void* b) {
    int32_t x = ((const orc_ent*)a)->c, y = ((const orc_ent*)b)->c;
    return (x > y) - (x < y);
}

/* Entries of one local row of (A'_k + I): neighbours inside the subgraph, parallel edges summed,
 * a unit self-loop added only if the row has none.  Returns the count; *offdiag = distinct
 * neighbours other than the node itself. */
static int64_t row_entries(int32_t u, int32_t lu, const int64_t* rowptr, const int32_t* col, const float* w,
                           const int32_t* local_of, orc_ent* tmp, int32_t* offdiag) {
    int64_t m = 0;
    for (int64_t e = rowptr[u]; e < rowptr[u + 1]; ++e) {
        int32_t lv = local_of[col[e]];
        if (lv < 0) continue;
        tmp[m].c = lv;
        tmp[m].w = w ? (double)w[e] : 1.0;
        ++m;
    }
    qsort(tmp, (size_t)m, sizeof(orc_ent), ent_cmp);
    int64_t o = 0;
    for (int64_t i = 0; i < m; ++i) {
        if (o > 0 && tmp[o - 1].c == tmp[i].c) tmp[o - 1].w += tmp[i].w;
        else tmp[o++] = tmp[i];
    }
    int has_self = 0;
    for (int64_t i = 0; i < o; ++i) if (tmp[i].c == lu) has_self = 1;
    *offdiag = (int32_t)(o - has_self);
    if (!has_self) {
        int64_t pos = o;
        while (pos > 0 && tmp[pos - 1].c > lu) { tmp[pos] = tmp[pos - 1]; --pos; }
        tmp[pos].c = lu;
        tmp[pos].w = 1.0;
        ++o;
    }
    return o;
}

static int fill_local_map(int32_t n, int32_t k, const int64_t* core_ptr, const int32_t* core_nodes,
                          const int64_t* halo_ptr, const int32_t* halo_nodes, int32_t* local_of, int set) {
    int32_t l = 0;
    for (int64_t i = core_ptr[k]; i < core_ptr[k + 1]; ++i, ++l) {
        int32_t u = core_nodes[i];
        if (u < 0 || u >= n) return ORC_ERR_RANGE;
        if (set) { if (local_of[u] >= 0) return ORC_ERR_DUPLICATE; local_of[u] = l; } else local_of[u] = -1;
    }
    for (int64_t i = halo_ptr[k]; i < halo_ptr[k + 1]; ++i, ++l) {
        int32_t u = halo_nodes[i];
        if (u < 0 || u >= n) return ORC_ERR_RANGE;
        if (set) { if (local_of[u] >= 0) return ORC_ERR_DUPLICATE; local_of[u] = l; } else local_of[u] = -1;
    }
    return ORC_OK;
}

/* pass = 0: sizes only (s_* may be NULL); pass = 1: fill.  */
static int store_pass(int pass, int32_t n, const int64_t* rowptr, const int32_t* col, const float* w, int32_t K,
                      const int64_t* core_ptr, const int32_t* core_nodes, const int64_t* halo_ptr,
                      const int32_t* halo_nodes, int64_t* n_prime, int64_t* nnz_prime, int64_t* s_rowptr,
                      int32_t* s_col, double* s_val, int32_t* sub_off, int32_t* gid, int32_t* deg) {
    int32_t* local_of = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    int64_t maxdeg = 1;
    for (int32_t u = 0; u < n; ++u) if (rowptr[u + 1] - rowptr[u] > maxdeg) maxdeg = rowptr[u + 1] - rowptr[u];
    orc_ent* tmp = (orc_ent*)malloc(sizeof(orc_ent) * (size_t)(maxdeg + 1));
    if (!local_of || !tmp) { free(local_of); free(tmp); return ORC_ERR_OOM; }
    for (int32_t u = 0; u < n; ++u) local_of[u] = -1;
    int64_t r = 0, z = 0;
    int rc = ORC_OK;
    if (pass) { s_rowptr[0] = 0; sub_off[0] = 0; }
    for (int32_t k = 0; k < K && rc == ORC_OK; ++k) {
        rc = fill_local_map(n, k, core_ptr, core_nodes, halo_ptr, halo_nodes, local_of, 1);
        if (rc != ORC_OK) break;
        int64_t nc = core_ptr[k + 1] - core_ptr[k], nh = halo_ptr[k + 1] - halo_ptr[k];
        int64_t off = r;
        for (int64_t l = 0; l < nc + nh; ++l, ++r) {
            int32_t u = l < nc ? core_nodes[core_ptr[k] + l] : halo_nodes[halo_ptr[k] + (l - nc)];
            int32_t od;
            int64_t m = row_entries(u, (int32_t)l, rowptr, col, w, local_of, tmp, &od);
            if (pass) {
                gid[r] = u;
                deg[r] = od;
                for (int64_t i = 0; i < m; ++i) {
                    s_col[z + i] = (int32_t)(off + tmp[i].c);
                    s_val[z + i] = tmp[i].w;
                }
                s_rowptr[r + 1] = z + m;
            }
            z += m;
        }
        if (pass) sub_off[k + 1] = (int32_t)r;
        fill_local_map(n, k, core_ptr, core_nodes, halo_ptr, halo_nodes, local_of, 0);
    }
    free(local_of);
    free(tmp);
    if (rc != ORC_OK) return rc;
    if (pass) {
        /* A~_ij = a_ij / sqrt(d~_i d~_j),  d~_i = sum_j (A'_k + I)_ij   (Section 3.3, forward equation) */
        double* dt = (double*)malloc(sizeof(double) * (size_t)(r > 0 ? r : 1));
        if (!dt) return ORC_ERR_OOM;
        for (int64_t i = 0; i < r; ++i) {
            double s = 0.0;
            for (int64_t e = s_rowptr[i]; e < s_rowptr[i + 1]; ++e) s += s_val[e];
            dt[i] = s;
        }
        for (int64_t i = 0; i < r; ++i)
            for (int64_t e = s_rowptr[i]; e < s_rowptr[i + 1]; ++e)
                s_val[e] = s_val[e] / sqrt(dt[i] * dt[s_col[e]]);
        free(dt);
    }
    *n_prime = r;
    *nnz_prime = z;
    return ORC_OK;
}

int orc_store_sizes(int32_t n, const int64_t* rowptr, const int32_t* col, int32_t K, const int64_t* core_ptr,
                    const int32_t* core_nodes, const int64_t* halo_ptr, const int32_t* halo_nodes,
                    int64_t* n_prime, int64_t* nnz_prime) {
    return store_pass(0, n, rowptr, col, NULL, K, core_ptr, core_nodes, halo_ptr, halo_nodes, n_prime, nnz_prime,
                      NULL, NULL, NULL, NULL, NULL, NULL);
}

int orc_store_build(int32_t n, const int64_t* rowptr, const int32_t* col, const float* w, int32_t K,
                    const int64_t* core_ptr, const int32_t* core_nodes, const int64_t* halo_ptr,
                    const int32_t* halo_nodes, int64_t* s_rowptr, int32_t* s_col, double* s_val,
                    int32_t* sub_off, int32_t* gid, int32_t* deg) {
    int64_t a, b;
    return store_pass(1, n, rowptr, col, w, K, core_ptr, core_nodes, halo_ptr, halo_nodes, &a, &b, s_rowptr, s_col,
                      s_val, sub_off, gid, deg);
}

/* ------------------------------------------------------------------------------------------
 * The model: K replicas, one per augmented subgraph (Algorithm 2 with one subgraph per processor).
 * ---------------------------------------------------------------------------------------- */

typedef struct {
    int64_t Np, nnz, P;
    int32_t K, L;
    int32_t* dims;            /* L+1 */
    int64_t* rowptr;          /* Np+1 */
    int32_t* col;             /* nnz  */
    double* val;              /* nnz  */
    int32_t* sub_off;         /* K+1  */
    int32_t* deg;             /* Np: local degree without the self-loop */
    int32_t* label;           /* Np   */
    uint8_t* train;           /* Np: 1 for core nodes whose split is "train" */
    int64_t* ntrain;          /* K    */
    double** H;               /* L+1 activations, H[0] = input features, H[L] = logits */
    double* Z;                /* scratch, Np x max width */
    double* dPre;             /* scratch */
    double* dZ;               /* scratch */
    double* params;           /* K x P */
    double* grads;            /* K x P */
    double lr, dropout, beta;
    uint64_t seed;
    int32_t weighted, zeta_mode;
    int64_t epoch;
    int8_t** branch;          /* L+1 maps [Np x dims[l]] or NULL: 0 = ReLU decides, 1 = unit taken as on, 2 = as off */
} orc_model;

static int64_t w_off(const orc_model* m, int l) {
    int64_t o = 0;
    for (int i = 0; i < l; ++i) o += (int64_t)m->dims[i] * m->dims[i + 1] + m->dims[i + 1];
    return o;
}
static int64_t b_off(const orc_model* m, int l) { return w_off(m, l) + (int64_t)m->dims[l] * m->dims[l + 1]; }

void orc_destroy(orc_model* m) {
    if (!m) return;
    if (m->H) { for (int l = 0; l <= m->L; ++l) free(m->H[l]); free(m->H); }
    if (m->branch) { for (int l = 0; l <= m->L; ++l) free(m->branch[l]); free(m->branch); }
    free(m->dims); free(m->rowptr); free(m->col); free(m->val); free(m->sub_off); free(m->deg); free(m->label);
    free(m->train); free(m->ntrain); free(m->Z); free(m->dPre); free(m->dZ); free(m->params); free(m->grads);
    free(m);
}

/* X is the whole graph's feature matrix [n x dims[0]] (float); labels / split are per graph node;
 * is_core[r] = 1 when store row r is one of its subgraph's own nodes.  params0: one replica's
 * parameters, copied to all K replicas (Algorithm 2: every processor starts from the same model). */
orc_model* orc_create(int64_t Np, int64_t nnz, const int64_t* s_rowptr, const int32_t* s_col, const double* s_val,
                      int32_t K, const int32_t* sub_off, const int32_t* gid, const int32_t* deg,
                      const int64_t* core_count, const float* X, const int32_t* labels, const uint8_t* split,
                      int32_t L, const int32_t* dims, double lr, double dropout, uint64_t seed, double beta,
                      int32_t weighted, int32_t zeta_mode, const float* params0) {
    orc_model* m = (orc_model*)calloc(1, sizeof(orc_model));
    if (!m) return NULL;
    m->Np = Np; m->nnz = nnz; m->K = K; m->L = L;
    m->lr = lr; m->dropout = dropout; m->seed = seed; m->beta = beta; m->weighted = weighted; m->zeta_mode = zeta_mode;
    m->dims = (int32_t*)malloc(sizeof(int32_t) * (size_t)(L + 1));
    memcpy(m->dims, dims, sizeof(int32_t) * (size_t)(L + 1));
    m->P = w_off(m, L);
    int maxw = 0;
    for (int l = 0; l <= L; ++l) if (dims[l] > maxw) maxw = dims[l];
    size_t rows = (size_t)(Np > 0 ? Np : 1);
    m->rowptr = (int64_t*)malloc(sizeof(int64_t) * (rows + 1));
    m->col = (int32_t*)malloc(sizeof(int32_t) * (size_t)(nnz > 0 ? nnz : 1));
    m->val = (double*)malloc(sizeof(double) * (size_t)(nnz > 0 ? nnz : 1));
    m->sub_off = (int32_t*)malloc(sizeof(int32_t) * (size_t)(K + 1));
    m->deg = (int32_t*)malloc(sizeof(int32_t) * rows);
    m->label = (int32_t*)malloc(sizeof(int32_t) * rows);
    m->train = (uint8_t*)malloc(rows);
    m->ntrain = (int64_t*)calloc((size_t)K, sizeof(int64_t));
    m->H = (double**)calloc((size_t)(L + 1), sizeof(double*));
    m->Z = (double*)malloc(sizeof(double) * rows * (size_t)maxw);
    m->dPre = (double*)malloc(sizeof(double) * rows * (size_t)maxw);
    m->dZ = (double*)malloc(sizeof(double) * rows * (size_t)maxw);
    m->params = (double*)malloc(sizeof(double) * (size_t)K * (size_t)m->P);
    m->grads = (double*)calloc((size_t)K * (size_t)m->P, sizeof(double));
    int ok = m->rowptr && m->col && m->val && m->sub_off && m->deg && m->label && m->train && m->ntrain && m->H &&
             m->Z && m->dPre && m->dZ && m->params && m->grads;
    if (ok) for (int l = 0; l <= L; ++l) {
        m->H[l] = (double*)calloc(rows * (size_t)dims[l], sizeof(double));
        if (!m->H[l]) ok = 0;
    }
    if (!ok) { orc_destroy(m); return NULL; }
    memcpy(m->rowptr, s_rowptr, sizeof(int64_t) * (size_t)(Np + 1));
    memcpy(m->col, s_col, sizeof(int32_t) * (size_t)nnz);
    memcpy(m->val, s_val, sizeof(double) * (size_t)nnz);
    memcpy(m->sub_off, sub_off, sizeof(int32_t) * (size_t)(K + 1));
    memcpy(m->deg, deg, sizeof(int32_t) * (size_t)Np);
    int F0 = dims[0];
    for (int32_t k = 0; k < K; ++k) {
        for (int64_t r = sub_off[k]; r < sub_off[k + 1]; ++r) {
            int32_t u = gid[r];
            for (int f = 0; f < F0; ++f) m->H[0][r * F0 + f] = (double)X[(int64_t)u * F0 + f];
            m->label[r] = labels[u];
            int core = (r - sub_off[k]) < core_count[k];
            m->train[r] = (uint8_t)(core && split[u] == 0);
            m->ntrain[k] += m->train[r];
        }
    }
    for (int32_t k = 0; k < K; ++k)
        for (int64_t i = 0; i < m->P; ++i) m->params[k * m->P + i] = (double)params0[i];
    return m;
}

/* Dropout keep decision: a pure function of (seed, epoch, layer, store row, column), built from the
 * splitmix64 output mixer (Steele, Lea, Flood 2014).  keep iff the top 24 bits are >= floor(p * 2^24). */
static uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
    return z ^ (z >> 31);
}
static int keep_unit(uint64_t seed, int64_t epoch, int layer, int64_t row, int colm, double p) {
    const uint64_t G = 0x9e3779b97f4a7c15ULL;
    uint64_t h = mix64(seed + G * (uint64_t)(1 + epoch));
    h = mix64(h + G * (uint64_t)(1 + layer));
    h = mix64(h + G * (uint64_t)(1 + row));
    h = mix64(h + G * (uint64_t)(1 + colm));
    uint32_t thr = (uint32_t)floor(p * 16777216.0);
    return (uint32_t)(h >> 40) >= thr;
}

/* Forward propagation, H^(l+1) = sigma(A~_k (H^(l) W_k^(l)) + b_k^(l)), sigma = ReLU except on the
 * last layer (Section 3.3, forward equations).  train != 0 applies dropout after the ReLU. */
static void forward(orc_model* m, int train) {
    for (int l = 0; l < m->L; ++l) {
        int fi = m->dims[l], fo = m->dims[l + 1];
        const double* Hin = m->H[l];
        double* Hout = m->H[l + 1];
        int64_t wo = w_off(m, l), bo = b_off(m, l);
        for (int32_t k = 0; k < m->K; ++k) {
            const double* W = m->params + (int64_t)k * m->P + wo;
            const double* b = m->params + (int64_t)k * m->P + bo;
            int64_t r0 = m->sub_off[k], r1 = m->sub_off[k + 1];
#pragma omp parallel for schedule(static)
            for (int64_t r = r0; r < r1; ++r)
                for (int j = 0; j < fo; ++j) {
                    double s = 0.0;
                    for (int f = 0; f < fi; ++f) s += Hin[r * fi + f] * W[(int64_t)f * fo + j];
                    m->Z[r * fo + j] = s;
                }
#pragma omp parallel for schedule(dynamic, 64)
            for (int64_t r = r0; r < r1; ++r)
                for (int j = 0; j < fo; ++j) {
                    double s = 0.0;
                    for (int64_t e = m->rowptr[r]; e < m->rowptr[r + 1]; ++e)
                        s += m->val[e] * m->Z[(int64_t)m->col[e] * fo + j];
                    s += b[j];
                    if (l < m->L - 1) {
                        int br = (m->branch && m->branch[l + 1]) ? m->branch[l + 1][r * fo + j] : 0;
                        s = br == 1 ? s : (br == 2 ? 0.0 : (s > 0.0 ? s : 0.0));
                        if (train && m->dropout > 0.0)
                            s = keep_unit(m->seed, m->epoch, l, r, j, m->dropout) ? s / (1.0 - m->dropout) : 0.0;
                    }
                    Hout[r * fo + j] = s;
                }
        }
    }
}

/* Softmax cross-entropy of subgraph k, mean over its training nodes, and d(loss)/d(logits) into dPre. */
static void loss_and_dlogits(orc_model* m, double* loss_k) {
    int C = m->dims[m->L];
    const double* logit = m->H[m->L];
    for (int32_t k = 0; k < m->K; ++k) {
        double tot = 0.0;
        double nt = (double)m->ntrain[k];
        for (int64_t r = m->sub_off[k]; r < m->sub_off[k + 1]; ++r) {
            double* g = m->dPre + r * C;
            if (!m->train[r]) { for (int c = 0; c < C; ++c) g[c] = 0.0; continue; }
            const double* z = logit + r * C;
            double mx = z[0];
            for (int c = 1; c < C; ++c) if (z[c] > mx) mx = z[c];
            double se = 0.0;
            for (int c = 0; c < C; ++c) se += exp(z[c] - mx);
            double lse = mx + log(se);
            tot += lse - z[m->label[r]];
            for (int c = 0; c < C; ++c) g[c] = (exp(z[c] - lse) - (c == m->label[r] ? 1.0 : 0.0)) / nt;
        }
        loss_k[k] = m->ntrain[k] > 0 ? tot / nt : 0.0;
    }
}

/* Backward propagation by the chain rule through the forward equations; on entry dPre holds
 * d(loss)/d(pre-activation of the last layer).  Fills grads[k] = d L_k / d theta_k. */
static void backward(orc_model* m) {
    for (int l = m->L - 1; l >= 0; --l) {
        int fi = m->dims[l], fo = m->dims[l + 1];
        int64_t wo = w_off(m, l), bo = b_off(m, l);
        for (int32_t k = 0; k < m->K; ++k) {
            int64_t r0 = m->sub_off[k], r1 = m->sub_off[k + 1];
            double* gW = m->grads + (int64_t)k * m->P + wo;
            double* gb = m->grads + (int64_t)k * m->P + bo;
            /* bias: column sums of dPre */
            for (int j = 0; j < fo; ++j) {
                double s = 0.0;
                for (int64_t r = r0; r < r1; ++r) s += m->dPre[r * fo + j];
                gb[j] = s;
            }
            /* dZ = A~_k^T dPre : scatter row i of dPre along row i of A~ */
            for (int64_t r = r0; r < r1; ++r) for (int j = 0; j < fo; ++j) m->dZ[r * fo + j] = 0.0;
#pragma omp parallel for schedule(static)
            for (int j = 0; j < fo; ++j)
                for (int64_t r = r0; r < r1; ++r) {
                    double g = m->dPre[r * fo + j];
                    if (g == 0.0) continue;
                    for (int64_t e = m->rowptr[r]; e < m->rowptr[r + 1]; ++e)
                        m->dZ[(int64_t)m->col[e] * fo + j] += m->val[e] * g;
                }
            /* dW = H^(l)^T dZ */
#pragma omp parallel for schedule(static)
            for (int f = 0; f < fi; ++f)
                for (int j = 0; j < fo; ++j) {
                    double s = 0.0;
                    for (int64_t r = r0; r < r1; ++r) s += m->H[l][r * fi + f] * m->dZ[r * fo + j];
                    gW[(int64_t)f * fo + j] = s;
                }
        }
        if (l == 0) break;
        /* dH^(l) = dZ W^T, then through the ReLU (and dropout scale) of layer l-1 into dPre; a second
         * sweep over k, once every gradient of this layer is done, because dPre is overwritten */
        double* next = (double*)malloc(sizeof(double) * (size_t)m->Np * (size_t)fi);
        for (int32_t k = 0; k < m->K; ++k) {
            const double* W = m->params + (int64_t)k * m->P + wo;
            int64_t r0 = m->sub_off[k], r1 = m->sub_off[k + 1];
#pragma omp parallel for schedule(static)
            for (int64_t r = r0; r < r1; ++r)
                for (int f = 0; f < fi; ++f) {
                    double s = 0.0;
                    for (int j = 0; j < fo; ++j) s += m->dZ[r * fo + j] * W[(int64_t)f * fo + j];
                    double h = m->H[l][r * fi + f];
                    double scale = m->dropout > 0.0 ? 1.0 / (1.0 - m->dropout) : 1.0;
                    int br = (m->branch && m->branch[l]) ? m->branch[l][r * fi + f] : 0;
                    int on = h > 0.0;
                    if (br == 1) on = !(m->dropout > 0.0) || keep_unit(m->seed, m->epoch, l - 1, r, f, m->dropout);
                    if (br == 2) on = 0;
                    next[r * fi + f] = on ? s * scale : 0.0;
                }
        }
        memcpy(m->dPre, next, sizeof(double) * (size_t)m->Np * (size_t)fi);
        free(next);
    }
}

/* ------------------------------------------------------------------------------------------
 * a7.  Variance-based subgraph importance (Section 3.4.1).
 * ---------------------------------------------------------------------------------------- */

/* p(v_i) of a subgraph: local degree over the sum of local degrees; uniform when there are no edges. */
static void node_prob(const int32_t* deg, int64_t n, double* p) {
    double tot = 0.0;
    for (int64_t i = 0; i < n; ++i) tot += (double)deg[i];
    for (int64_t i = 0; i < n; ++i) p[i] = tot > 0.0 ? (double)deg[i] / tot : 1.0 / (double)n;
}

/* "aggregate" reading: zeta = S / (D + beta), S = sum_{i<j} p_i p_j = (1 - sum p_i^2)/2,
 * D = sqrt( sum_{i<j} p_i p_j |x_i - x_j|^2 / S ), the numerator evaluated one feature dimension at
 * a time as the p-weighted variance of that dimension. */
double orc_zeta_aggregate(const int32_t* deg, const double* X, int64_t n, int F, double beta) {
    if (n <= 0) return 0.0;
    double* p = (double*)malloc(sizeof(double) * (size_t)n);
    node_prob(deg, n, p);
    double sq = 0.0;
    for (int64_t i = 0; i < n; ++i) sq += p[i] * p[i];
    double S = 0.5 * (1.0 - sq);
    double Q = 0.0;
    for (int f = 0; f < F; ++f) {
        double m1 = 0.0;
        for (int64_t i = 0; i < n; ++i) m1 += p[i] * X[i * F + f];
        double v = 0.0;
        for (int64_t i = 0; i < n; ++i) { double d = X[i * F + f] - m1; v += p[i] * d * d; }
        Q += v;
    }
    free(p);
    if (!(S > 0.0)) return 0.0;
    return S / (sqrt(Q / S) + beta);
}

/* "pairwise" reading, the printed formula taken literally: sum_{i<j} p_i p_j / (|x_i - x_j| + beta). O(n^2 F). */
double orc_zeta_pairwise(const int32_t* deg, const double* X, int64_t n, int F, double beta) {
    if (n <= 0) return 0.0;
    double* p = (double*)malloc(sizeof(double) * (size_t)n);
    node_prob(deg, n, p);
    double z = 0.0;
    for (int64_t i = 0; i < n; ++i)
        for (int64_t j = i + 1; j < n; ++j) {
            double d2 = 0.0;
            for (int f = 0; f < F; ++f) { double d = X[i * F + f] - X[j * F + f]; d2 += d * d; }
            z += p[i] * p[j] / (sqrt(d2) + beta);
        }
    free(p);
    return z;
}

/* The two sums of the aggregate reading straight from their pair definitions (O(n^2 F)); used to pin the
 * closed forms above.  out[0] = sum_{i<j} p_i p_j, out[1] = sum_{i<j} p_i p_j |x_i - x_j|^2. */
void orc_zeta_pair_sums(const int32_t* deg, const double* X, int64_t n, int F, double* out) {
    double* p = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    node_prob(deg, n, p);
    double S = 0.0, Q = 0.0;
    for (int64_t i = 0; i < n; ++i)
        for (int64_t j = i + 1; j < n; ++j) {
            double d2 = 0.0;
            for (int f = 0; f < F; ++f) { double d = X[i * F + f] - X[j * F + f]; d2 += d * d; }
            S += p[i] * p[j];
            Q += p[i] * p[j] * d2;
        }
    free(p);
    out[0] = S;
    out[1] = Q;
}

/* zeta_k for every subgraph and the consensus weights w_k = zeta_k / sum_j zeta_j (Section 3.4.2);
 * with weighted == 0 the weights are 1/K (Definition 3). */
void orc_subgraph_weights(orc_model* m, double* zeta, double* w) {
    int F = m->dims[0];
    double tot = 0.0;
    for (int32_t k = 0; k < m->K; ++k) {
        int64_t r0 = m->sub_off[k], n = m->sub_off[k + 1] - r0;
        if (m->zeta_mode == 2) {
            /* The sum over the layers l of the variance equation (Section 3.4.1) kept: the squared distance of two
             * nodes is summed over the inputs H^(0) .. H^(L-1) of all layers, i.e. it is the squared distance of the
             * rows of [H^(0) | H^(1) | ... | H^(L-1)], as they stand after the most recent forward pass. */
            int Ft = 0;
            for (int l = 0; l < m->L; ++l) Ft += m->dims[l];
            double* cat = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1) * (size_t)Ft);
            for (int64_t i = 0; i < n; ++i) {
                int o = 0;
                for (int l = 0; l < m->L; ++l) {
                    for (int f = 0; f < m->dims[l]; ++f) cat[i * Ft + o + f] = m->H[l][(r0 + i) * m->dims[l] + f];
                    o += m->dims[l];
                }
            }
            zeta[k] = orc_zeta_aggregate(m->deg + r0, cat, n, Ft, m->beta);
            free(cat);
        } else {
            zeta[k] = m->zeta_mode == 1 ? orc_zeta_pairwise(m->deg + r0, m->H[0] + r0 * F, n, F, m->beta)
                                        : orc_zeta_aggregate(m->deg + r0, m->H[0] + r0 * F, n, F, m->beta);
        }
        tot += zeta[k];
    }
    for (int32_t k = 0; k < m->K; ++k)
        w[k] = (m->weighted && tot > 0.0) ? zeta[k] / tot : 1.0 / (double)m->K;
}

/* a8.  Weighted global consensus over the K parameter copies: theta_k <- sum_j w_j theta_j for all k. */
void orc_consensus(orc_model* m) {
    double* zeta = (double*)malloc(sizeof(double) * (size_t)m->K * 2);
    double* w = zeta + m->K;
    orc_subgraph_weights(m, zeta, w);
    for (int64_t i = 0; i < m->P; ++i) {
        double s = 0.0;
        for (int32_t k = 0; k < m->K; ++k) s += w[k] * m->params[(int64_t)k * m->P + i];
        for (int32_t k = 0; k < m->K; ++k) m->params[(int64_t)k * m->P + i] = s;
    }
    free(zeta);
}

/* Inference-mode forward (no dropout); logits of every store row are then in H[L]. */
void orc_forward(orc_model* m) { forward(m, 0); }

/* Training-mode forward and the K per-subgraph losses, nothing else (used by finite differences). */
void orc_forward_loss(orc_model* m, double* loss_k) {
    forward(m, 1);
    loss_and_dlogits(m, loss_k);
}

/* Forward, loss, backward: fills grads without touching the parameters. */
void orc_forward_backward(orc_model* m, double* loss_k) {
    forward(m, 1);
    loss_and_dlogits(m, loss_k);
    backward(m);
}

/* One pass of Algorithm 2 with one subgraph per processor: every replica does forward, loss and
 * backward on its subgraph, takes its SGD step, and the copies are merged by the weighted
 * consensus.  loss_out: K subgraph losses, then sum_k |T_k| L_k / sum_k |T_k|, all before the update. */
void orc_train_epoch(orc_model* m, double* loss_out) {
    orc_forward_backward(m, loss_out);
    double num = 0.0, den = 0.0;
    for (int32_t k = 0; k < m->K; ++k) { num += (double)m->ntrain[k] * loss_out[k]; den += (double)m->ntrain[k]; }
    loss_out[m->K] = den > 0.0 ? num / den : 0.0;
    for (int64_t i = 0; i < (int64_t)m->K * m->P; ++i) m->params[i] -= m->lr * m->grads[i];
    orc_consensus(m);
    m->epoch += 1;
}

/* Prescribes the ReLU branch of n hidden units of H^(layer), 1 <= layer <= L-1 (side 1: on, 2: off, 0: let the ReLU
 * decide again); n < 0 forgets every prescription of that layer.  For units at the kink, see the header comment. */
int orc_set_relu_branch(orc_model* m, int32_t layer, int64_t n, const int64_t* rows, const int32_t* cols, int32_t side) {
    if (!m || layer < 1 || layer > m->L - 1 || side < 0 || side > 2) return ORC_ERR_ARG;
    if (!m->branch) {
        m->branch = (int8_t**)calloc((size_t)(m->L + 1), sizeof(int8_t*));
        if (!m->branch) return ORC_ERR_OOM;
    }
    size_t cells = (size_t)(m->Np > 0 ? m->Np : 1) * (size_t)m->dims[layer];
    if (n < 0) { free(m->branch[layer]); m->branch[layer] = NULL; return ORC_OK; }
    if (!m->branch[layer]) {
        m->branch[layer] = (int8_t*)calloc(cells, 1);
        if (!m->branch[layer]) return ORC_ERR_OOM;
    }
    for (int64_t i = 0; i < n; ++i) {
        if (rows[i] < 0 || rows[i] >= m->Np || cols[i] < 0 || cols[i] >= m->dims[layer]) return ORC_ERR_RANGE;
        m->branch[layer][rows[i] * m->dims[layer] + cols[i]] = (int8_t)side;
    }
    return ORC_OK;
}

/* accessors */
int64_t orc_param_count(const orc_model* m) { return m->P; }
void orc_get_params(const orc_model* m, int32_t k, double* out) { memcpy(out, m->params + (int64_t)k * m->P, sizeof(double) * (size_t)m->P); }
void orc_set_params(orc_model* m, int32_t k, const double* in) { memcpy(m->params + (int64_t)k * m->P, in, sizeof(double) * (size_t)m->P); }
void orc_get_grads(const orc_model* m, int32_t k, double* out) { memcpy(out, m->grads + (int64_t)k * m->P, sizeof(double) * (size_t)m->P); }
void orc_get_activation(const orc_model* m, int32_t l, double* out) { memcpy(out, m->H[l], sizeof(double) * (size_t)m->Np * (size_t)m->dims[l]); }
void orc_get_ntrain(const orc_model* m, int64_t* out) { memcpy(out, m->ntrain, sizeof(int64_t) * (size_t)m->K); }
int64_t orc_get_epoch(const orc_model* m) { return m->epoch; }
void orc_set_epoch(orc_model* m, int64_t e) { m->epoch = e; }
int orc_keep_unit(uint64_t seed, int64_t epoch, int layer, int64_t row, int colm, double p) { return keep_unit(seed, epoch, layer, row, colm, p); }
uint64_t orc_mix64(uint64_t z) { return mix64(z); }
