// Create-time host code: input validation and the block-diagonal store of the augmented subgraphs
// g'_k = (v_k + v'_k, e_k + e'_k) (Algorithm 1 of the paper, last step) with the normalised adjacency
// A~_k = D~^-1/2 (A'_k + I) D~^-1/2 of the forward equation (Section 3.3).  Not on the timed path.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <utility>

#include "gad_internal.h"

namespace gad {

static int validate(const gad_csr* g, const gad_partition* part, std::string& err) {
    if (!g || !part) { err = "graph or partition is NULL"; return GAD_ERR_ARG; }
    if (g->n < 0 || g->nnz < 0 || !g->rowptr || (g->nnz > 0 && !g->col)) { err = "bad CSR header"; return GAD_ERR_ARG; }
    if (g->rowptr[0] != 0 || g->rowptr[g->n] != g->nnz) { err = "rowptr[0] != 0 or rowptr[n] != nnz"; return GAD_ERR_ARG; }
    for (int32_t u = 0; u < g->n; ++u)
        if (g->rowptr[u + 1] < g->rowptr[u]) { err = "rowptr decreases at row " + std::to_string(u); return GAD_ERR_UNSORTED; }
    for (int64_t e = 0; e < g->nnz; ++e)
        if (g->col[e] < 0 || g->col[e] >= g->n) { err = "column out of range at entry " + std::to_string(e); return GAD_ERR_RANGE; }
    if (part->K < 1 || !part->core_ptr || !part->halo_ptr) { err = "partition needs K >= 1 and both pointer arrays"; return GAD_ERR_ARG; }
    if (part->core_ptr[0] != 0 || part->halo_ptr[0] != 0) { err = "core_ptr[0] / halo_ptr[0] must be 0"; return GAD_ERR_ARG; }
    for (int32_t k = 0; k < part->K; ++k)
        if (part->core_ptr[k + 1] < part->core_ptr[k] || part->halo_ptr[k + 1] < part->halo_ptr[k]) {
            err = "core_ptr / halo_ptr decreases at subgraph " + std::to_string(k);
            return GAD_ERR_UNSORTED;
        }
    if ((part->core_ptr[part->K] > 0 && !part->core_nodes) || (part->halo_ptr[part->K] > 0 && !part->halo_nodes)) {
        err = "node list is NULL";
        return GAD_ERR_ARG;
    }
    int64_t rows = part->core_ptr[part->K] + part->halo_ptr[part->K];
    if (rows >= (int64_t)1 << 31) { err = "more than 2^31-1 store rows"; return GAD_ERR_RANGE; }
    std::vector<uint8_t> owned((size_t)g->n, 0);
    for (int64_t i = 0; i < part->core_ptr[part->K]; ++i) {
        int32_t u = part->core_nodes[i];
        if (u < 0 || u >= g->n) { err = "core node out of range"; return GAD_ERR_RANGE; }
        if (owned[u]) { err = "node " + std::to_string(u) + " is a core node twice"; return GAD_ERR_DUPLICATE; }
        owned[u] = 1;
    }
    for (int64_t i = 0; i < part->halo_ptr[part->K]; ++i) {
        int32_t u = part->halo_nodes[i];
        if (u < 0 || u >= g->n) { err = "replicated node out of range"; return GAD_ERR_RANGE; }
    }
    return GAD_OK;
}

// local id of every graph node inside subgraph k, or -1
static int fill_local(const gad_partition* part, int32_t k, std::vector<int32_t>& local_of, std::string& err) {
    int32_t l = 0;
    for (int64_t i = part->core_ptr[k]; i < part->core_ptr[k + 1]; ++i) local_of[part->core_nodes[i]] = l++;
    for (int64_t i = part->halo_ptr[k]; i < part->halo_ptr[k + 1]; ++i) {
        int32_t u = part->halo_nodes[i];
        if (local_of[u] >= 0) {
            err = "node " + std::to_string(u) + " listed twice in subgraph " + std::to_string(k);
            return GAD_ERR_DUPLICATE;
        }
        local_of[u] = l++;
    }
    return GAD_OK;
}
static void clear_local(const gad_partition* part, int32_t k, std::vector<int32_t>& local_of) {
    for (int64_t i = part->core_ptr[k]; i < part->core_ptr[k + 1]; ++i) local_of[part->core_nodes[i]] = -1;
    for (int64_t i = part->halo_ptr[k]; i < part->halo_ptr[k + 1]; ++i) local_of[part->halo_nodes[i]] = -1;
}
static inline int32_t node_of(const gad_partition* part, int32_t k, int64_t local) {
    int64_t nc = part->core_ptr[k + 1] - part->core_ptr[k];
    return local < nc ? part->core_nodes[part->core_ptr[k] + local] : part->halo_nodes[part->halo_ptr[k] + (local - nc)];
}

int store_sizes(const gad_csr* g, const gad_partition* part, int64_t* Np, int64_t* nnz, int64_t* slots, std::string& err) {
    HostStore tmp;
    int rc = build_store(g, part, false, tmp, err);
    if (rc != GAD_OK) return rc;
    *Np = tmp.Np;
    *nnz = tmp.nnz;
    *slots = std::max(count_slots(tmp.rowptr), count_slots(tmp.t_rowptr));
    return GAD_OK;
}

int build_store(const gad_csr* g, const gad_partition* part, bool values, HostStore& st, std::string& err) {
    int rc = validate(g, part, err);
    if (rc != GAD_OK) return rc;
    const int32_t K = part->K;
    st.K = K;
    st.Np = part->core_ptr[K] + part->halo_ptr[K];
    st.sub_off.assign((size_t)K + 1, 0);
    st.core_count.assign((size_t)K, 0);
    for (int32_t k = 0; k < K; ++k) {
        st.core_count[k] = part->core_ptr[k + 1] - part->core_ptr[k];
        st.sub_off[k + 1] = st.sub_off[k] + (int32_t)(st.core_count[k] + part->halo_ptr[k + 1] - part->halo_ptr[k]);
    }
    const int64_t Np = st.Np;
    std::vector<int32_t> local_of((size_t)g->n, -1);

    // Pass 1: an upper bound of every row's length (neighbours inside the subgraph + a possible self-loop).
    std::vector<int64_t> ub((size_t)Np + 1, 0);
    for (int32_t k = 0; k < K; ++k) {
        rc = fill_local(part, k, local_of, err);
        if (rc != GAD_OK) return rc;
        const int64_t r0 = st.sub_off[k], nk = st.sub_off[k + 1] - r0;
#pragma omp parallel for schedule(static)
        for (int64_t l = 0; l < nk; ++l) {
            int32_t u = node_of(part, k, l);
            int64_t c = 1;
            for (int64_t e = g->rowptr[u]; e < g->rowptr[u + 1]; ++e) c += local_of[g->col[e]] >= 0;
            ub[r0 + l + 1] = c;
        }
        clear_local(part, k, local_of);
    }
    for (int64_t r = 0; r < Np; ++r) ub[r + 1] += ub[r];

    // Pass 2: every row gathered into its slot, sorted by local column, duplicates merged, self-loop ensured.
    std::vector<int32_t> tcol((size_t)ub[Np]);
    std::vector<double> tval(values ? (size_t)ub[Np] : 0);
    std::vector<int64_t> len((size_t)Np + 1, 0);
    st.gid.assign((size_t)Np, 0);
    st.deg.assign((size_t)Np, 0);
    for (int32_t k = 0; k < K; ++k) {
        fill_local(part, k, local_of, err);
        const int64_t r0 = st.sub_off[k], nk = st.sub_off[k + 1] - r0;
#pragma omp parallel
        {
            std::vector<std::pair<int32_t, double>> row;
#pragma omp for schedule(dynamic, 256)
            for (int64_t l = 0; l < nk; ++l) {
                int32_t u = node_of(part, k, l);
                row.clear();
                for (int64_t e = g->rowptr[u]; e < g->rowptr[u + 1]; ++e) {
                    int32_t lv = local_of[g->col[e]];
                    if (lv >= 0) row.emplace_back(lv, g->w ? (double)g->w[e] : 1.0);
                }
                bool sorted = true;
                for (size_t i = 1; i < row.size(); ++i) if (row[i - 1].first >= row[i].first) { sorted = false; break; }
                if (!sorted)
                    std::stable_sort(row.begin(), row.end(),
                                     [](const std::pair<int32_t, double>& a, const std::pair<int32_t, double>& b) { return a.first < b.first; });
                int64_t base = ub[r0 + l], o = 0;
                bool self = false, placed = false;
                for (size_t i = 0; i < row.size(); ++i) self = self || row[i].first == (int32_t)l;
                int32_t distinct = 0;
                for (size_t i = 0; i < row.size(); ++i) {
                    if (!self && !placed && row[i].first > (int32_t)l) {
                        tcol[base + o] = (int32_t)(r0 + l);
                        if (values) tval[base + o] = 1.0;
                        ++o;
                        placed = true;
                    }
                    if (i > 0 && row[i].first == row[i - 1].first) {
                        if (values) tval[base + o - 1] += row[i].second;
                        continue;
                    }
                    tcol[base + o] = (int32_t)(r0 + row[i].first);
                    if (values) tval[base + o] = row[i].second;
                    ++o;
                    ++distinct;
                }
                if (!self && !placed) {
                    tcol[base + o] = (int32_t)(r0 + l);
                    if (values) tval[base + o] = 1.0;
                    ++o;
                }
                len[r0 + l + 1] = o;
                st.gid[r0 + l] = u;
                st.deg[r0 + l] = distinct - (self ? 1 : 0);
            }
        }
        clear_local(part, k, local_of);
    }
    st.rowptr.assign((size_t)Np + 1, 0);
    for (int64_t r = 0; r < Np; ++r) st.rowptr[r + 1] = st.rowptr[r] + len[r + 1];
    st.nnz = st.rowptr[Np];
    if (!values) {
        // sizes only: the row lengths of the transposed store are the column counts
        st.t_rowptr.assign((size_t)Np + 1, 0);
        for (int64_t r = 0; r < Np; ++r)
            for (int64_t i = 0; i < len[r + 1]; ++i) st.t_rowptr[tcol[ub[r] + i] + 1]++;
        for (int64_t r = 0; r < Np; ++r) st.t_rowptr[r + 1] += st.t_rowptr[r];
        return GAD_OK;
    }

    // Compaction and normalisation: d~_i = row sum of (A'_k + I); A~_ij = a_ij / sqrt(d~_i d~_j).
    std::vector<double> dt((size_t)Np);
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < Np; ++r) {
        double s = 0.0;
        for (int64_t i = 0; i < len[r + 1]; ++i) s += tval[ub[r] + i];
        dt[r] = s;
    }
    st.col.resize((size_t)st.nnz);
    st.val.resize((size_t)st.nnz);
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < Np; ++r) {
        int64_t src = ub[r], dst = st.rowptr[r];
        for (int64_t i = 0; i < len[r + 1]; ++i) {
            int32_t c = tcol[src + i];
            st.col[dst + i] = c;
            st.val[dst + i] = (float)(tval[src + i] / std::sqrt(dt[r] * dt[c]));
        }
    }
    tcol.clear(); tcol.shrink_to_fit();
    tval.clear(); tval.shrink_to_fit();

    // Transposed store by counting sort; rows are visited in ascending order, so every transposed row comes
    // out with ascending columns.
    st.t_rowptr.assign((size_t)Np + 1, 0);
    for (int64_t e = 0; e < st.nnz; ++e) st.t_rowptr[st.col[e] + 1]++;
    for (int64_t r = 0; r < Np; ++r) st.t_rowptr[r + 1] += st.t_rowptr[r];
    st.t_col.resize((size_t)st.nnz);
    st.t_val.resize((size_t)st.nnz);
    {
        std::vector<int64_t> cur(st.t_rowptr.begin(), st.t_rowptr.end() - 1);
        for (int64_t r = 0; r < Np; ++r)
            for (int64_t e = st.rowptr[r]; e < st.rowptr[r + 1]; ++e) {
                int64_t p = cur[st.col[e]]++;
                st.t_col[p] = (int32_t)r;
                st.t_val[p] = st.val[e];
            }
    }
    st.symmetric = st.t_rowptr == st.rowptr && st.t_col == st.col &&
                   std::memcmp(st.t_val.data(), st.val.data(), sizeof(float) * (size_t)st.nnz) == 0;
    if (st.symmetric) {
        st.t_rowptr.clear(); st.t_rowptr.shrink_to_fit();
        st.t_col.clear(); st.t_col.shrink_to_fit();
        st.t_val.clear(); st.t_val.shrink_to_fit();
    }
    return GAD_OK;
}

int64_t part_entries_for(const std::vector<int64_t>& rowptr) {
    const int64_t Np = (int64_t)rowptr.size() - 1;
    // No shorter than a quarter of the entries an average resident warp gets (148 SMs x 64 warps): cutting rows finer than
    // that buys no balance and costs a scratch row (written, read back, added) per part.  Measured on 2.5 M rows of mean
    // degree 39: parts of 2048 instead of 64 entries take 8 % off the 256-wide aggregation; on 110 000 rows (2.3 M
    // entries) anything above 64 is slower, and this floor stays at 64 there.
    int64_t part = kMinPart;
    while (2 * part <= std::min<int64_t>(kMaxPart, rowptr[Np] / (4 * 148 * 64))) part *= 2;
    for (; part < kMaxPart; part *= 2) {
        int64_t slots = 0;
        for (int64_t r = 0; r < Np; ++r) {
            const int64_t len = rowptr[r + 1] - rowptr[r];
            if (len > part) slots += (len + part - 1) / part;
        }
        if (2 * slots <= Np) break;
    }
    return part;
}

// Part length of one cut row: the store's part length, or longer so that the row has at most kMaxSlotsPerRow parts
// (the parts of a hub row then end inside the main kernel instead of as a long serial sum in the finishing one).
static int64_t row_part_entries(int64_t len, int64_t part) {
    const int64_t want = round_up((len + kMaxSlotsPerRow - 1) / kMaxSlotsPerRow, 32);
    return std::min<int64_t>(std::max(part, want), 65535 / 32 * 32);
}

int64_t count_slots(const std::vector<int64_t>& rowptr) {
    const int64_t part = part_entries_for(rowptr);
    int64_t slots = 0;
    for (size_t r = 0; r + 1 < rowptr.size(); ++r) {
        const int64_t len = rowptr[r + 1] - rowptr[r];
        if (len > part) { const int64_t pl = row_part_entries(len, part); slots += (len + pl - 1) / pl; }
    }
    return slots;
}

void bin_rows(const std::vector<int64_t>& rowptr, const std::vector<int32_t>& sub_off, RowWork& out, int64_t forced_part) {
    const int64_t Np = (int64_t)rowptr.size() - 1;
    const int64_t part = forced_part > 0 ? forced_part : part_entries_for(rowptr);
    out.perm.clear(); out.parts.clear(); out.fin.clear(); out.items.clear(); out.slots = 0; out.part_entries = part;
    std::vector<int64_t> count(64, 0);
    auto bin_of = [](int64_t len) { int b = 0; while (len > 1) { len >>= 1; ++b; } return b; };
    for (int64_t r = 0; r < Np; ++r) {
        const int64_t len = rowptr[r + 1] - rowptr[r];
        if (len <= part) count[bin_of(len)]++;
    }
    std::vector<int64_t> start(64, 0);
    int64_t acc = 0;
    for (int b = 63; b >= 0; --b) { start[b] = acc; acc += count[b]; }
    out.perm.resize((size_t)acc);
    for (int64_t r = 0; r < Np; ++r) {
        const int64_t len = rowptr[r + 1] - rowptr[r];
        if (len <= part) { out.perm[(size_t)start[bin_of(len)]++] = (int32_t)r; continue; }
        const int64_t pl = row_part_entries(len, part);
        const int64_t np = (len + pl - 1) / pl;
        out.fin.push_back(make_int4((int)r, (int)out.slots, (int)np, 0));   // the subgraph is filled in below
        for (int64_t q = 0; q < np; ++q)
            out.parts.push_back(make_int4((int)r, (int)(q * pl), (int)std::min(pl, len - q * pl), (int)(out.slots + q)));
        out.slots += np;
    }
    // the unified list: subgraph by subgraph (the operand rows one subgraph gathers stay together in L2), parts
    // and uncut rows of a subgraph longest first
    auto pack = [&](int64_t row, int64_t e0, int64_t len, int64_t slot) {
        return make_int4((int)row, (int)(uint32_t)(e0 & 0xFFFFFFFFll), (int)(uint32_t)(((e0 >> 32) << 16) | len), (int)slot);
    };
    const int64_t K = (int64_t)sub_off.size() - 1;
    std::vector<int32_t> sub_of((size_t)Np);
    for (int64_t k = 0; k < K; ++k)
        for (int64_t r = sub_off[k]; r < sub_off[k + 1]; ++r) sub_of[(size_t)r] = (int32_t)k;
    for (int4& f : out.fin) f.w = sub_of[(size_t)f.x];
    auto key = [&](int64_t row, int64_t len) { return (size_t)(sub_of[(size_t)row] * 64 + (63 - bin_of(len))); };
    std::vector<int64_t> istart((size_t)K * 64 + 1, 0);
    for (const int4& pt : out.parts) istart[key(pt.x, pt.z) + 1]++;
    for (int32_t r : out.perm) istart[key(r, rowptr[r + 1] - rowptr[r]) + 1]++;
    for (size_t i = 1; i < istart.size(); ++i) istart[i] += istart[i - 1];
    out.items.resize((size_t)istart.back());
    for (const int4& pt : out.parts) out.items[(size_t)istart[key(pt.x, pt.z)]++] = pack(pt.x, rowptr[pt.x] + pt.y, pt.z, pt.w);
    for (int32_t r : out.perm) {
        const int64_t len = rowptr[r + 1] - rowptr[r];
        out.items[(size_t)istart[key(r, len)]++] = pack(r, rowptr[r], len, -1);
    }
}

}  // namespace gad
