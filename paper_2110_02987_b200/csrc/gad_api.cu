// The C boundary (include/gad.h): context, workspace plan, create, and the per-epoch launch sequence.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>

#include "gad_internal.h"

using namespace gad;

#include <mutex>
#include <set>

namespace gad {

std::atomic<int64_t> g_kernel_launches{0};

cudaError_t configure_kernel_once(const void* kernel, int smem_bytes, bool max_carveout) {
    static std::mutex lock;
    static std::set<std::pair<int, const void*>> done;   // (device, kernel)
    std::lock_guard<std::mutex> guard(lock);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const std::pair<int, const void*> key(dev, kernel);
    if (done.count(key)) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    if (max_carveout) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
    }
    done.insert(key);
    return cudaSuccess;
}

}  // namespace gad

// TMA descriptors kept per layer: forward A, B_hi, B_lo; input-gradient A, B_hi, B_lo; weight-gradient H, dZ.
constexpr int kMapsPerLayer = 8;

namespace {

struct ProfEntry {
    std::string name;
    int64_t launches = 0;
    double ms = 0.0, bytes = 0.0, flops = 0.0;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> pending;
};

// Everything whose size follows from (n, K, subgraph sizes, nnz', dims): used by gad_workspace_bytes and by
// gad_create, so both agree byte for byte.
struct Plan {
    int32_t n = 0, K = 0, L = 0;
    int64_t Np = 0, nnz = 0, P = 0, Pint = 0, pstride = 0, slots = 0;
    std::vector<int32_t> dims;
    std::vector<Layer> layers;
    std::vector<int32_t> ld;          // [L+1]
    int32_t maxld = 0;
    std::vector<RowSpan> tiles, chunks, dw_chunks, core_spans;
    std::vector<int32_t> chunk_ptr, dw_chunk_ptr;   // [K+1]
    std::vector<int64_t> pair_ptr;    // [K+1] tiles of pairs per subgraph (zeta_mode 1 on the FP32 ALUs), else empty
    size_t o_pair_ptr = 0, o_pair_partial = 0;
    std::vector<int64_t> gram_ptr;    // [K+1] 128 x 128 tiles of pairs per subgraph (zeta_mode 1 on the tensor cores)
    size_t o_gram_ptr = 0, o_gram_partial = 0, o_norm2 = 0, o_xhi = 0, o_xlo = 0;
    bool pair_alu_ok = false;         // every subgraph is small enough for the FP32-ALU pairwise kernel
    int64_t dw_partial = 0;           // floats per chunk
    std::vector<uint8_t> agg_first;   // [L] the layer aggregates before it transforms: sigma((A~ H^(l)) W + b)
    std::vector<size_t> o_P;          // [L] A~ H^(l)  [Np x ld_l] of those layers
    size_t o_counters = 0;            // arrival counters: [loss | K column sums | K zeta]
    // layers l >= 1 of at most 16 output columns take the streaming FP32 kernel on the way back (flag bit 2 switches it off)
    std::vector<uint8_t> narrow;      // [L]
    std::vector<RowSpan> nchunks;     // their row chunks: about three CTAs per SM, never across subgraphs
    std::vector<int32_t> nchunk_ptr;  // [K+1]
    size_t o_nchunks = 0, o_nchunk_ptr = 0, o_nw_partial = 0;
    size_t o_zeta_q = 0;              // [K] doubles: distance sums carried from layer to layer (zeta_mode 2)
    size_t o_bf16 = 0;                // [Np x widest SpMM operand] bfloat16 copy of the operand (gemm_mode 1), else unused
    size_t bytes = 0;
    // offsets into the workspace
    size_t o_growptr = 0, o_gecv = 0, o_gfin = 0, o_gitems = 0;   // the loss rows' store (see gad_ctx::Ag)
    size_t o_rowptr, o_ecv, o_fin, o_items, o_trowptr, o_tecv, o_tfin, o_titems, o_spmm_scratch, o_sub_off, o_gid, o_deg, o_label, o_train,
        o_deg_sum, o_deg_sq, o_inv_ntrain, o_tiles, o_chunks, o_chunk_ptr, o_dw_chunks, o_dw_chunk_ptr, o_core_spans, o_G1, o_G2, o_params, o_grads,
        o_dw_partial, o_cs_partial, o_loss_partial, o_zeta_partial, o_zeta, o_loss, o_flags, o_zeta_f, o_w_f, o_stage,
        o_stage_lab, o_stage2, o_stage_lab2;
    std::vector<size_t> o_H, o_w_hi, o_w_lo, o_wt_hi, o_wt_lo;   // per layer
};

size_t take(size_t& cur, size_t bytes) {
    size_t o = cur;
    cur += (size_t)round_up((int64_t)std::max<size_t>(bytes, 4), 256);
    return o;
}

int make_plan(Plan& p, int32_t n, int32_t K, const std::vector<int32_t>& sub_off, const std::vector<int64_t>& core_count,
              int64_t nnz, int64_t slots, const gad_config* cfg, std::string& err) {
    if (!cfg || cfg->L < 1 || !cfg->dims) { err = "config needs L >= 1 and dims"; return GAD_ERR_ARG; }
    for (int l = 0; l <= cfg->L; ++l)
        if (cfg->dims[l] < 1) { err = "layer size must be positive"; return GAD_ERR_ARG; }
    if (!(cfg->dropout >= 0.f && cfg->dropout < 1.f)) { err = "dropout must be in [0,1)"; return GAD_ERR_ARG; }
    if (cfg->gemm_mode != 0 && cfg->gemm_mode != 1) { err = "gemm_mode must be 0 or 1"; return GAD_ERR_ARG; }
    if (cfg->zeta_mode < 0 || cfg->zeta_mode > 2) { err = "zeta_mode must be 0, 1 or 2"; return GAD_ERR_ARG; }
    p.pair_alu_ok = true;
    for (int32_t k = 0; k < K; ++k)
        if (sub_off[k + 1] - sub_off[k] > kZetaPairMaxRows) p.pair_alu_ok = false;
    if (cfg->zeta_mode == 1 && (cfg->flags & (1 | 16)) != 0 && !p.pair_alu_ok) {   // the FP32-ALU form was asked for
        err = "zeta_mode 1 on the FP32 ALUs (flag bits 0 / 4) takes subgraphs of at most " + std::to_string(kZetaPairMaxRows) + " rows";
        return GAD_ERR_UNSUPPORTED;
    }
    if (!(cfg->beta > 0.f)) { err = "beta must be positive"; return GAD_ERR_ARG; }
    p.n = n; p.K = K; p.L = cfg->L; p.nnz = nnz; p.Np = sub_off[K]; p.slots = slots;
    p.dims.assign(cfg->dims, cfg->dims + cfg->L + 1);
    p.ld.resize(p.L + 1);
    p.maxld = 0;
    for (int l = 0; l <= p.L; ++l) { p.ld[l] = (int32_t)round_up(p.dims[l], 4); p.maxld = std::max(p.maxld, p.ld[l]); }
    // Layer 0 needs no gradient with respect to its input, so aggregating first costs one SpMM at the width F_0 where
    // transforming first costs two at F_1; keeping A~ H^(0) across epochs (flag bit 1) removes that one as well.
    // A layer l >= 1 needs the gradient with respect to its input either way, so it costs two SpMMs in both orders: at
    // the width F_l when it aggregates first, at F_{l+1} when it transforms first.  It aggregates first when its input is
    // the narrower side (flag bit 5 keeps the layers l >= 1 on the transform-first order, for comparison).
    p.agg_first.assign(p.L, 0);
    p.agg_first[0] = (cfg->flags & 2) != 0 || p.dims[0] <= 2 * p.dims[1];
    for (int l = 1; l < p.L; ++l) p.agg_first[l] = (cfg->flags & 32) == 0 && p.dims[l] < p.dims[l + 1];
    p.layers.resize(p.L);
    int64_t oi = 0, oe = 0;
    p.dw_partial = 0;
    for (int l = 0; l < p.L; ++l) {
        Layer& y = p.layers[l];
        y.fi = p.dims[l]; y.fo = p.dims[l + 1]; y.ldi = p.ld[l]; y.ldo = p.ld[l + 1]; y.ldw = p.ld[l + 1];
        y.w_int = oi; oi += (int64_t)y.fi * y.ldw;
        y.b_int = oi; oi += y.ldo;
        y.w_ext = oe; oe += (int64_t)y.fi * y.fo;
        y.b_ext = oe; oe += y.fo;
        p.dw_partial = std::max(p.dw_partial, (int64_t)y.fi * y.ldw);
    }
    p.P = oe; p.Pint = oi; p.pstride = round_up(oi, 64);
    // row tiles of the grouped transforms (128 rows, never across subgraphs) and reduction chunks
    const int64_t target = 592;
    int64_t R = round_up(std::max<int64_t>(1, (p.Np + target - 1) / target), 32);
    R = std::min<int64_t>(std::max<int64_t>(R, 128), 16384);
    // The weight gradient has a long reduction per output tile, so it gets longer chunks: about one CTA per SM (a
    // single wave: every CTA pays the pipeline fill once) over the layer with the most output tiles (128 rows x up to 256 columns each).
    int64_t max_tiles = 1;
    for (const Layer& y : p.layers) {
        const int bn = tc_bn_for(y.fo);
        max_tiles = std::max<int64_t>(max_tiles, ((y.fi + 127) / 128) * (int64_t)((y.ldw + bn - 1) / bn));
    }
    int64_t Rdw = round_up(std::max<int64_t>(1, p.Np * max_tiles / std::max<int64_t>(74, 148 - K)), 32);
    // (not longer than 4096 rows: the CTAs that share a chunk then stay close enough to share it in L2)
    Rdw = std::min<int64_t>(std::max<int64_t>(Rdw, 256), 4096);
    p.chunk_ptr.assign(K + 1, 0);
    p.dw_chunk_ptr.assign(K + 1, 0);
    for (int32_t k = 0; k < K; ++k) {
        for (int64_t r = sub_off[k]; r < sub_off[k + 1]; r += Rdw)
            p.dw_chunks.push_back(RowSpan{(int32_t)r, (int32_t)std::min<int64_t>(Rdw, sub_off[k + 1] - r), k, 0});
        p.dw_chunk_ptr[k + 1] = (int32_t)p.dw_chunks.size();
        for (int32_t r = sub_off[k]; r < sub_off[k + 1]; r += 128)
            p.tiles.push_back(RowSpan{r, std::min<int32_t>(128, sub_off[k + 1] - r), k, 0});
        for (int64_t r = sub_off[k]; r < sub_off[k + 1]; r += R)
            p.chunks.push_back(RowSpan{(int32_t)r, (int32_t)std::min<int64_t>(R, sub_off[k + 1] - r), k, 0});
        p.chunk_ptr[k + 1] = (int32_t)p.chunks.size();
        for (int64_t r = 0; r < core_count[k]; r += 256)
            p.core_spans.push_back(RowSpan{(int32_t)(sub_off[k] + r), (int32_t)std::min<int64_t>(256, core_count[k] - r), k, 0});
    }
    const size_t Np = (size_t)p.Np, nc = p.chunks.size();
    size_t cur = 0;
    p.o_rowptr = take(cur, 8 * (Np + 1)); p.o_ecv = take(cur, 8 * (size_t)nnz);
    // work lists: one part per scratch slot, at most one cut row per kMinPart entries
    const size_t max_parts = (size_t)(slots + 1), max_fin = (size_t)(nnz / kMinPart + 1);
    p.o_fin = take(cur, 16 * max_fin);
    p.o_items = take(cur, 16 * (Np + max_parts));
    p.o_trowptr = take(cur, 8 * (Np + 1)); p.o_tecv = take(cur, 8 * (size_t)nnz);
    p.o_tfin = take(cur, 16 * max_fin);
    p.o_titems = take(cur, 16 * (Np + max_parts));
    if (!(cfg->flags & 64)) {
        p.o_growptr = take(cur, 8 * (Np + 1)); p.o_gecv = take(cur, 8 * (size_t)nnz);
        p.o_gfin = take(cur, 16 * max_fin);
        p.o_gitems = take(cur, 16 * (Np + max_parts));
    }
    p.o_sub_off = take(cur, 4 * (size_t)(K + 1)); p.o_gid = take(cur, 4 * Np); p.o_deg = take(cur, 4 * Np);
    p.o_label = take(cur, 4 * Np); p.o_train = take(cur, Np);
    p.o_deg_sum = take(cur, 8 * (size_t)K); p.o_deg_sq = take(cur, 8 * (size_t)K); p.o_inv_ntrain = take(cur, 4 * (size_t)K);
    p.o_tiles = take(cur, sizeof(RowSpan) * p.tiles.size()); p.o_chunks = take(cur, sizeof(RowSpan) * nc);
    p.o_chunk_ptr = take(cur, 4 * (size_t)(K + 1));
    p.o_dw_chunks = take(cur, sizeof(RowSpan) * p.dw_chunks.size()); p.o_dw_chunk_ptr = take(cur, 4 * (size_t)(K + 1));
    p.o_core_spans = take(cur, sizeof(RowSpan) * p.core_spans.size());
    p.o_H.resize(p.L + 1);
    for (int l = 0; l <= p.L; ++l) p.o_H[l] = take(cur, 4 * Np * (size_t)p.ld[l]);
    int32_t max_spmm_ld = 4;   // a layer's SpMMs run at its input width when it aggregates first, else at its output width
    for (int l = 0; l < p.L; ++l) max_spmm_ld = std::max(max_spmm_ld, p.ld[p.agg_first[l] ? l : l + 1]);
    p.o_spmm_scratch = take(cur, 4 * (size_t)slots * (size_t)max_spmm_ld);
    if (cfg->gemm_mode == 1) p.o_bf16 = take(cur, 2 * Np * (size_t)max_spmm_ld);
    p.o_G1 = take(cur, 4 * Np * (size_t)p.maxld); p.o_G2 = take(cur, 4 * Np * (size_t)p.maxld);
    p.o_params = take(cur, 4 * (size_t)K * (size_t)p.pstride); p.o_grads = take(cur, 4 * (size_t)K * (size_t)p.pstride);
    p.o_dw_partial = take(cur, 4 * p.dw_chunks.size() * (size_t)p.dw_partial); p.o_cs_partial = take(cur, 4 * nc * (size_t)p.maxld);
    int32_t zeta_ld = p.ld[0];   // widest matrix the importance statistics run over: H^(0), or every layer's input (zeta_mode 2)
    if (cfg->zeta_mode == 2)
        for (int l = 0; l < p.L; ++l) zeta_ld = std::max(zeta_ld, p.ld[l]);
    p.o_loss_partial = take(cur, 4 * nc); p.o_zeta_partial = take(cur, 8 * nc * 2 * (size_t)zeta_ld);
    p.o_zeta_q = take(cur, 8 * (size_t)K);
    p.o_zeta = take(cur, 8 * (size_t)K); p.o_loss = take(cur, 4 * (size_t)(K + 1)); p.o_flags = take(cur, 16);
    p.o_zeta_f = take(cur, 4 * (size_t)K); p.o_w_f = take(cur, 4 * (size_t)K);
    p.o_stage = take(cur, 4 * (size_t)n * (size_t)std::max(p.dims[0], p.dims[p.L])); p.o_stage_lab = take(cur, 4 * (size_t)n);
    // second staging pair: the copy of the next inputs may run while the previous ones are still being gathered
    p.o_stage2 = take(cur, 4 * (size_t)n * (size_t)p.dims[0]); p.o_stage_lab2 = take(cur, 4 * (size_t)n);
    p.o_w_hi.resize(p.L); p.o_w_lo.resize(p.L); p.o_wt_hi.resize(p.L); p.o_wt_lo.resize(p.L);
    for (int l = 0; l < p.L; ++l) {
        const Layer& y = p.layers[l];
        p.o_w_hi[l] = take(cur, 4 * (size_t)K * y.fi * y.ldw); p.o_w_lo[l] = take(cur, 4 * (size_t)K * y.fi * y.ldw);
        p.o_wt_hi[l] = take(cur, 4 * (size_t)K * y.fo * y.ldi); p.o_wt_lo[l] = take(cur, 4 * (size_t)K * y.fo * y.ldi);
    }
    p.o_counters = take(cur, 4 * (size_t)(1 + 2 * K));
    p.o_P.assign(p.L, 0);
    for (int l = 0; l < p.L; ++l)
        if (p.agg_first[l]) p.o_P[l] = take(cur, 4 * Np * (size_t)p.ld[l]);
    p.narrow.assign(p.L, 0);
    int64_t narrow_partial = 0;
    for (int l = 0; l < p.L; ++l) {
        const Layer& y = p.layers[l];
        p.narrow[l] = (cfg->flags & 5) == 0 && l > 0 && !p.agg_first[l] && narrow_supported(y.ldi, y.ldo);
        if (p.narrow[l]) narrow_partial = std::max(narrow_partial, (int64_t)y.fi * y.ldw + y.ldi);
    }
    if (narrow_partial > 0) {
        const int64_t Rn = std::max<int64_t>(64, round_up((p.Np + 443) / 444, 32));
        p.nchunk_ptr.assign(K + 1, 0);
        for (int32_t k = 0; k < K; ++k) {
            for (int64_t r = sub_off[k]; r < sub_off[k + 1]; r += Rn)
                p.nchunks.push_back(RowSpan{(int32_t)r, (int32_t)std::min<int64_t>(Rn, sub_off[k + 1] - r), k, 0});
            p.nchunk_ptr[k + 1] = (int32_t)p.nchunks.size();
        }
        p.o_nchunks = take(cur, sizeof(RowSpan) * p.nchunks.size());
        p.o_nchunk_ptr = take(cur, 4 * (size_t)(K + 1));
        p.o_nw_partial = take(cur, 4 * p.nchunks.size() * (size_t)narrow_partial);
    }
    if (cfg->zeta_mode == 1 && p.pair_alu_ok) {
        p.pair_ptr.assign(K + 1, 0);
        for (int32_t k = 0; k < K; ++k) p.pair_ptr[k + 1] = p.pair_ptr[k] + zeta_pair_tiles(sub_off[k + 1] - sub_off[k]);
        p.o_pair_ptr = take(cur, 8 * (size_t)(K + 1));
        p.o_pair_partial = take(cur, 8 * (size_t)p.pair_ptr[K]);
    }
    if (cfg->zeta_mode == 1 && (cfg->flags & (1 | 16)) == 0) {
        p.gram_ptr.assign(K + 1, 0);
        for (int32_t k = 0; k < K; ++k) p.gram_ptr[k + 1] = p.gram_ptr[k] + zeta_gram_tiles(sub_off[k + 1] - sub_off[k]);
        p.o_gram_ptr = take(cur, 8 * (size_t)(K + 1));
        p.o_gram_partial = take(cur, 8 * (size_t)zeta_gram_partials(kGramMaxCtas, K));
        p.o_norm2 = take(cur, 4 * Np);
        p.o_xhi = take(cur, 4 * Np * (size_t)p.ld[0]); p.o_xlo = take(cur, 4 * Np * (size_t)p.ld[0]);
    }
    p.bytes = cur;
    return GAD_OK;
}

}  // namespace

struct gad_ctx {
    struct alignas(64) TMap { unsigned char bytes[128]; };
    cudaStream_t stream = nullptr;
    char* ws = nullptr;
    Plan p;
    gad_config cfg{};
    std::string err;
    bool symmetric = false;
    SparseDev A, At;
    // The transposed store without the entries that read a row carrying no loss (a replicated node, or a core node that
    // is not a training node): d loss / d logits is zero there, so the backward aggregation of the last layer gathers
    // only the rest and adds the same numbers in the same order.  Built once (the split is fixed at creation).
    SparseDev Ag;
    bool use_loss_rows = false;
    int64_t nnz_loss_rows = 0;
    int64_t epoch = 0;
    std::vector<int32_t> sub_off, gid;
    std::vector<int64_t> ntrain;
    int64_t ntrain_total = 0;
    bool profiling = false;
    std::vector<ProfEntry> prof;
    std::vector<float> host_block;  // staging for parameter pack / unpack
    cudaStream_t copy_stream = nullptr;   // host -> device copies of gad_set_inputs
    cudaStream_t side_stream = nullptr;   // small kernels of an epoch that depend on little (operand split, zeta, bias gradients)
    cudaEvent_t ev_fork = nullptr, ev_split = nullptr, ev_g1 = nullptr, ev_bias = nullptr, ev_join = nullptr;
    cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_gathered[2] = {nullptr, nullptr};
    int stage_idx = 0;              // staging pair the next gad_set_inputs uses
    bool hoist = false;             // keep A~ H^(0) across epochs (config flag bit 1)
    bool P_valid = false;           // A~ H^(0) matches the current features
    bool acts_valid = false;        // a forward pass has filled H^(1) .. H^(L)
    // The launches of an epoch captured once and replayed (index 0: gad_train_epoch_local, 1: gad_train_epoch).
    struct EpochGraph { cudaGraphExec_t exec = nullptr; int64_t kernels = 0; bool failed = false; } graphs[2];
    int64_t direct_epochs = 0;      // epochs enqueued launch by launch so far (the first one also sets up the kernels)
    bool use_tc = false;            // tensor-core transforms (tcgen05) instead of the SIMT ones
    bool use_gram = false;          // zeta_mode 1 through the Gram-matrix kernel on the tensor cores
    TMap map_xhi, map_xlo;          // the TF32 split of H^(0) as 128-row boxes, for that kernel
    int num_sms = 1;
    std::vector<TMap> maps;         // per layer: forward A, B_hi, B_lo; input-gradient A, B_hi, B_lo

    template <class T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
    float* H(int l) const { return at<float>(p.o_H[l]); }
};

namespace {

thread_local std::string g_last_error;  // also readable after a failed gad_create, when there is no context

int fail(gad_ctx* c, int code, const std::string& msg) {
    if (c) c->err = msg;
    g_last_error = msg;
    return code;
}
#define GAD_CK(call)                                                                                       \
    do {                                                                                                   \
        cudaError_t e_ = (call);                                                                           \
        if (e_ != cudaSuccess)                                                                             \
            return fail(ctx, GAD_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_));            \
    } while (0)

ProfEntry& prof_entry(gad_ctx* c, const char* name, int layer, double bytes, double flops) {
    char buf[64];
    if (layer >= 0) snprintf(buf, sizeof buf, "%s_l%d", name, layer); else snprintf(buf, sizeof buf, "%s", name);
    for (auto& e : c->prof) if (e.name == buf) return e;
    c->prof.push_back(ProfEntry{});
    c->prof.back().name = buf;
    c->prof.back().bytes = bytes;
    c->prof.back().flops = flops;
    return c->prof.back();
}

// Runs one launcher, optionally bracketed by events on the context's stream.
template <class F>
int run(gad_ctx* ctx, const char* name, int layer, double bytes, double flops, F&& launch) {
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (ctx->profiling) {
        GAD_CK(cudaEventCreate(&e0));
        GAD_CK(cudaEventCreate(&e1));
        GAD_CK(cudaEventRecord(e0, ctx->stream));
    }
    cudaError_t e = launch();
    if (e != cudaSuccess) return fail(ctx, GAD_ERR_CUDA, std::string(name) + ": " + cudaGetErrorString(e));
    if (ctx->profiling) {
        GAD_CK(cudaEventRecord(e1, ctx->stream));
        prof_entry(ctx, name, layer, bytes, flops).pending.emplace_back(e0, e1);
    }
    return GAD_OK;
}
#define GAD_RUN(...)                            \
    do {                                        \
        int rc_ = run(ctx, __VA_ARGS__);        \
        if (rc_ != GAD_OK) return rc_;          \
    } while (0)

// Room for the bfloat16 copy of an aggregation's operand: the reduced-precision mode gathers from that copy.
void* bf16_of(gad_ctx* ctx) { return ctx->cfg.gemm_mode == 1 ? (void*)(ctx->ws + ctx->p.o_bf16) : nullptr; }

double spmm_bytes(const Plan& p, int F, int64_t nnz = -1) { return 8.0 * (nnz < 0 ? p.nnz : nnz) + 8.0 * p.Np + 8.0 * (double)p.Np * F; }

// Inside a training epoch the kernels that depend on little (operand split of the weights, zeta, bias gradients) go
// to a second stream and run beside the aggregation / transform sequence; events order them against it.  While
// per-kernel timing is on everything stays on the context's stream, where the timing events are recorded.
cudaStream_t side_of(gad_ctx* ctx) { return ctx->profiling ? ctx->stream : ctx->side_stream; }
// Work enqueued on `to` after this call starts only when the work enqueued on `from` so far has finished.
int hand_over(gad_ctx* ctx, cudaStream_t from, cudaStream_t to, cudaEvent_t ev) {
    if (from == to) return GAD_OK;
    GAD_CK(cudaEventRecord(ev, from));
    GAD_CK(cudaStreamWaitEvent(to, ev, 0));
    return GAD_OK;
}

int forward_pass(gad_ctx* ctx, bool train, cudaStream_t ss) {
    const Plan& p = ctx->p;
    float* Z = ctx->at<float>(p.o_G2);
    const float* params = ctx->at<float>(p.o_params);
    const int passes = ctx->cfg.gemm_mode == 0 ? 3 : 1;
    if (ctx->use_tc)
        for (int l = 0; l < p.L; ++l) {
            const Layer& y = p.layers[l];
            GAD_RUN("split_weights", l, 20.0 * p.K * y.fi * y.fo, 0.0, [&] {
                return launch_split_weights(params, p.pstride, y.w_int, y.fi, y.fo, y.ldw, y.ldi, p.K, ctx->at<float>(p.o_w_hi[l]),
                                            ctx->at<float>(p.o_w_lo[l]), ctx->at<float>(p.o_wt_hi[l]), ctx->at<float>(p.o_wt_lo[l]),
                                            ss);
            });
        }
    bool split_pending = ctx->use_tc && ss != ctx->stream;   // the first transform waits for the split operands
    if (split_pending) GAD_CK(cudaEventRecord(ctx->ev_split, ss));
    for (int l = 0; l < p.L; ++l) {
        const Layer& y = p.layers[l];
        Epilogue ep{params, p.pstride, y.b_int, ctx->at<int32_t>(p.o_sub_off), p.K, l < p.L - 1 ? 1 : 0,
                    train ? ctx->cfg.dropout : 0.f, ctx->cfg.seed, ctx->epoch, l};
        if (p.agg_first[l]) {
            // A~ (H W) = (A~ H) W: aggregate at the input width, finish the layer in the transform's epilogue
            if (!(l == 0 && ctx->hoist && ctx->P_valid)) {
                GAD_RUN("spmm_fwd", l, spmm_bytes(p, y.fi), 2.0 * p.nnz * y.fi,
                        [&] { return launch_spmm(ctx->A, ctx->H(l), y.ldi, ctx->at<float>(p.o_P[l]), y.ldi, y.fi, nullptr, bf16_of(ctx), false, ctx->stream); });
                if (l == 0) ctx->P_valid = true;
            }
            const ActEpi act = make_act(ep, 0);
            if (split_pending) { GAD_CK(cudaStreamWaitEvent(ctx->stream, ctx->ev_split, 0)); split_pending = false; }
            GAD_RUN("gemm_fwd", l, 4.0 * p.Np * (y.fi + y.fo) + 4.0 * p.K * y.fi * y.fo, 2.0 * p.Np * y.fi * y.fo, [&] {
                if (ctx->use_tc)
                    return launch_gemm_rows_tc(&ctx->maps[kMapsPerLayer * l + 0], &ctx->maps[kMapsPerLayer * l + 1], &ctx->maps[kMapsPerLayer * l + 2], 2, passes, y.fi, y.fo,
                                               ctx->H(l + 1), y.ldo, ctx->at<RowSpan>(p.o_tiles), (int)p.tiles.size(), nullptr, 0, 1.f, &act,
                                               ctx->at<int32_t>(p.o_flags) + 1, ctx->num_sms, ctx->stream);
                return launch_gemm_rows_simt(2, ctx->at<float>(p.o_P[l]), y.ldi, y.fi, params, p.pstride, y.w_int, y.ldw, y.fo, ctx->H(l + 1), y.ldo,
                                             ctx->at<RowSpan>(p.o_tiles), (int)p.tiles.size(), nullptr, 0, 1.f, &act, ctx->stream);
            });
            continue;
        }
        if (split_pending) { GAD_CK(cudaStreamWaitEvent(ctx->stream, ctx->ev_split, 0)); split_pending = false; }
        // reduced-precision mode: the transform writes the bfloat16 operand copy the aggregation gathers, and nothing else
        void* zb = ctx->use_tc ? bf16_of(ctx) : nullptr;
        GAD_RUN("gemm_fwd", l, 4.0 * p.Np * (y.fi + y.fo) + 4.0 * p.K * y.fi * y.fo, 2.0 * p.Np * y.fi * y.fo, [&] {
            if (ctx->use_tc)
                return launch_gemm_rows_tc(&ctx->maps[kMapsPerLayer * l + 0], &ctx->maps[kMapsPerLayer * l + 1], &ctx->maps[kMapsPerLayer * l + 2], 0, passes, y.fi, y.fo, Z,
                                           y.ldo, ctx->at<RowSpan>(p.o_tiles), (int)p.tiles.size(), nullptr, 0, 1.f, nullptr,
                                           ctx->at<int32_t>(p.o_flags) + 1, ctx->num_sms, ctx->stream, zb);
            return launch_gemm_rows_simt(0, ctx->H(l), y.ldi, y.fi, params, p.pstride, y.w_int, y.ldw, y.fo, Z, y.ldo,
                                         ctx->at<RowSpan>(p.o_tiles), (int)p.tiles.size(), nullptr, 0, 1.f, nullptr, ctx->stream);
        });
        GAD_RUN("spmm_fwd", l, spmm_bytes(p, y.fo), 2.0 * p.nnz * y.fo,
                [&] { return launch_spmm(ctx->A, Z, y.ldo, ctx->H(l + 1), y.ldo, y.fo, &ep, bf16_of(ctx), zb != nullptr, ctx->stream); });
    }
    ctx->acts_valid = true;
    return GAD_OK;
}

int zeta_pass(gad_ctx* ctx, cudaStream_t s) {
    const Plan& p = ctx->p;
    if (ctx->cfg.zeta_mode == 2 && !ctx->acts_valid) {   // asked for before any pass has run: an inference pass provides the activations
        int rc = forward_pass(ctx, false, ctx->stream);
        if (rc != GAD_OK) return rc;
    }
    if (ctx->cfg.zeta_mode == 1 && ctx->use_gram) {
        const double pairs = 128.0 * 128.0 * (double)p.gram_ptr[p.K];
        GAD_RUN("zeta", -1, 4.0 * p.Np * (p.dims[0] + 2), 2.0 * pairs * p.dims[0], [&] {
            return launch_zeta_gram(&ctx->map_xhi, &ctx->map_xlo, ctx->H(0), p.ld[0], p.dims[0], p.Np, ctx->at<int32_t>(p.o_deg),
                                    ctx->at<int32_t>(p.o_sub_off), ctx->at<int64_t>(p.o_deg_sum), ctx->at<int64_t>(p.o_gram_ptr),
                                    p.gram_ptr[p.K], p.K, ctx->cfg.beta, ctx->at<float>(p.o_xhi), ctx->at<float>(p.o_xlo),
                                    ctx->at<float>(p.o_norm2), ctx->at<double>(p.o_gram_partial), ctx->at<double>(p.o_zeta),
                                    ctx->at<int32_t>(p.o_flags) + 1, std::min(ctx->num_sms, kGramMaxCtas), s);
        });
        return GAD_OK;
    }
    if (ctx->cfg.zeta_mode == 1) {
        const double pairs = 64.0 * 64.0 * (double)p.pair_ptr[p.K];
        GAD_RUN("zeta", -1, 4.0 * p.Np * (p.dims[0] + 1), 3.0 * pairs * p.dims[0], [&] {
            return launch_zeta_pair(ctx->H(0), p.ld[0], p.dims[0], ctx->at<int32_t>(p.o_deg), ctx->at<int32_t>(p.o_sub_off),
                                    ctx->at<int64_t>(p.o_deg_sum), ctx->at<int64_t>(p.o_pair_ptr), p.pair_ptr[p.K], p.K, ctx->cfg.beta,
                                    ctx->at<double>(p.o_pair_partial), ctx->at<unsigned>(p.o_counters) + 1 + p.K,
                                    ctx->at<double>(p.o_zeta), s);
        });
        return GAD_OK;
    }
    // zeta_mode 2 keeps the sum over the layers of the variance equation (Section 3.4.1): the statistics run over the
    // input H^(l) of every layer (activations of the most recent forward pass), their distance sums added up
    const int nl = ctx->cfg.zeta_mode == 2 ? p.L : 1;
    double cols = 0.0;
    for (int l = 0; l < nl; ++l) cols += p.dims[l];
    GAD_RUN("zeta", -1, 4.0 * p.Np * (cols + nl), 4.0 * p.Np * cols, [&] {
        for (int l = 0; l < nl; ++l) {
            const int phase = nl == 1 ? 0 : (l == 0 ? 1 : (l == nl - 1 ? 3 : 2));
            cudaError_t e = launch_zeta(ctx->H(l), p.ld[l], p.dims[l], ctx->at<int32_t>(p.o_deg), ctx->at<RowSpan>(p.o_chunks),
                                        (int)p.chunks.size(), ctx->at<int32_t>(p.o_chunk_ptr), ctx->at<int32_t>(p.o_sub_off),
                                        ctx->at<int64_t>(p.o_deg_sum), ctx->at<int64_t>(p.o_deg_sq), ctx->cfg.beta,
                                        ctx->at<double>(p.o_zeta_partial), ctx->at<unsigned>(p.o_counters) + 1 + p.K,
                                        ctx->at<double>(p.o_zeta), ctx->at<double>(p.o_zeta_q), phase, s);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    });
    return GAD_OK;
}

int backward_pass(gad_ctx* ctx, cudaStream_t ss) {
    const Plan& p = ctx->p;
    float* G1 = ctx->at<float>(p.o_G1);
    float* G2 = ctx->at<float>(p.o_G2);
    float* grads = ctx->at<float>(p.o_grads);
    const float* params = ctx->at<float>(p.o_params);
    const RowSpan* chunks = ctx->at<RowSpan>(p.o_chunks);
    const int nc = (int)p.chunks.size();
    const int32_t* chunk_ptr = ctx->at<int32_t>(p.o_chunk_ptr);
    const RowSpan* dw_chunks = ctx->at<RowSpan>(p.o_dw_chunks);
    const int ndw = (int)p.dw_chunks.size();
    const int32_t* dw_chunk_ptr = ctx->at<int32_t>(p.o_dw_chunk_ptr);
    const float scale = ctx->cfg.dropout > 0.f ? 1.f / (1.f - ctx->cfg.dropout) : 1.f;
    bool bias_done = false;   // the layer above was narrow: its fused kernel has already summed this layer's dPre columns
    for (int l = p.L - 1; l >= 0; --l) {
        const Layer& y = p.layers[l];
        // the store of this layer's backward aggregation, and its entries
        const bool loss_rows = ctx->use_loss_rows && l == p.L - 1;
        const SparseDev& Ab = loss_rows ? ctx->Ag : (ctx->symmetric ? ctx->A : ctx->At);
        const int64_t nnz_b = loss_rows ? ctx->nnz_loss_rows : p.nnz;
        if (!bias_done) {
            // db reads dPre (G1) beside the kernels that follow; the next writer of G1 waits for it
            int rc = hand_over(ctx, ctx->stream, ss, ctx->ev_g1);
            if (rc != GAD_OK) return rc;
            GAD_RUN("bias_grad", l, 4.0 * p.Np * y.fo, 1.0 * p.Np * y.fo, [&] {
                return launch_colsum_chunks(G1, y.ldo, chunks, nc, ctx->at<float>(p.o_cs_partial), p.maxld, chunk_ptr,
                                            ctx->at<unsigned>(p.o_counters) + 1, grads, p.pstride, y.b_int, ss);
            });
            if (ss != ctx->stream) GAD_CK(cudaEventRecord(ctx->ev_bias, ss));
        }
        bias_done = false;
        const bool agg_first = p.agg_first[l] != 0;   // then dW = (A~ H^(l))^T dPre, and dH^(l) = A~^T (dPre W^T)
        if (!agg_first)
            GAD_RUN("spmm_bwd", l, spmm_bytes(p, y.fo, nnz_b), 2.0 * nnz_b * y.fo,
                    [&] { return launch_spmm(Ab, G1, y.ldo, G2, y.ldo, y.fo, nullptr, bf16_of(ctx), false, ctx->stream); });
        if (ctx->use_tc && p.narrow[l]) {
            // one pass over H^(l) and dZ gives both dW and dPre of the layer below (it writes G1: the column sums come first)
            if (ss != ctx->stream) GAD_CK(cudaStreamWaitEvent(ctx->stream, ctx->ev_bias, 0));
            // the chunk results hold db of layer l-1 and then dW of layer l, which is also their order in the parameter block
            const int64_t plen = (int64_t)y.ldi + (int64_t)y.fi * y.ldw;
            GAD_RUN("gemm_dwdh", l, 4.0 * p.Np * (2.0 * y.fi + y.fo) + 8.0 * p.K * y.fi * y.fo, 4.0 * p.Np * y.fi * y.fo, [&] {
                return launch_narrow_bwd(ctx->H(l), y.ldi, y.fi, G2, y.ldo, params, p.pstride, y.w_int, y.ldw,
                                         ctx->at<RowSpan>(p.o_nchunks), (int)p.nchunks.size(), scale, G1,
                                         ctx->at<float>(p.o_nw_partial), plen, ctx->at<int32_t>(p.o_flags) + 1, ctx->stream);
            });
            // the sum over the chunks is needed only by the update at the end of the epoch: beside the kernels that follow
            int rc2 = hand_over(ctx, ctx->stream, ss, ctx->ev_g1);
            if (rc2 != GAD_OK) return rc2;
            GAD_RUN("reduce_dwdh", l, 4.0 * (double)p.nchunks.size() * (double)plen, 1.0 * (double)p.nchunks.size() * (double)plen, [&] {
                return launch_reduce_chunks(ctx->at<float>(p.o_nw_partial), plen, ctx->at<int32_t>(p.o_nchunk_ptr), p.K, grads, p.pstride,
                                            p.layers[l - 1].b_int, plen, ss);
            });
            if (ss != ctx->stream) GAD_CK(cudaEventRecord(ctx->ev_bias, ss));   // a later narrow layer reuses the chunk results' buffer
            bias_done = true;
            continue;
        }
        GAD_RUN("gemm_dw", l, 4.0 * p.Np * (y.fi + y.fo) + 4.0 * p.K * y.fi * y.fo, 2.0 * p.Np * y.fi * y.fo, [&] {
            cudaError_t e =
                ctx->use_tc ? launch_gemm_tn_tc(&ctx->maps[kMapsPerLayer * l + 6], &ctx->maps[kMapsPerLayer * l + 7],
                                                ctx->cfg.gemm_mode == 0 ? 3 : 1, y.fi, y.fo, y.ldw, dw_chunks, ndw,
                                                ctx->at<float>(p.o_dw_partial), ctx->at<int32_t>(p.o_flags) + 1, ctx->stream)
                            : launch_gemm_tn_simt(agg_first ? ctx->at<float>(p.o_P[l]) : ctx->H(l), y.ldi, y.fi, agg_first ? G1 : G2, y.ldo,
                                                  y.fo, dw_chunks, ndw, ctx->at<float>(p.o_dw_partial), y.ldw, ctx->stream);
            if (e != cudaSuccess) return e;
            return launch_reduce_chunks(ctx->at<float>(p.o_dw_partial), (int64_t)y.fi * y.ldw, dw_chunk_ptr, p.K, grads, p.pstride,
                                        y.w_int, (int64_t)y.fi * y.ldw, ctx->stream);
        });
        if (l > 0 && agg_first) {
            // dP = dPre W^T (no mask yet: the ReLU of layer l-1 sits below the aggregation), dH^(l) = A~^T dP, then the mask
            GAD_RUN("gemm_dh", l, 4.0 * p.Np * (y.fi + y.fo) + 4.0 * p.K * y.fi * y.fo, 2.0 * p.Np * y.fi * y.fo, [&] {
                if (ctx->use_tc)
                    return launch_gemm_rows_tc(&ctx->maps[kMapsPerLayer * l + 3], &ctx->maps[kMapsPerLayer * l + 4], &ctx->maps[kMapsPerLayer * l + 5], 1,
                                               ctx->cfg.gemm_mode == 0 ? 3 : 1, y.fo, y.fi, G2, y.ldi, ctx->at<RowSpan>(p.o_tiles),
                                               (int)p.tiles.size(), nullptr, 0, 1.f, nullptr, ctx->at<int32_t>(p.o_flags) + 1,
                                               ctx->num_sms, ctx->stream);
                return launch_gemm_rows_simt(1, G1, y.ldo, y.fo, params, p.pstride, y.w_int, y.ldw, y.fi, G2, y.ldi,
                                             ctx->at<RowSpan>(p.o_tiles), (int)p.tiles.size(), nullptr, 0, 1.f, nullptr, ctx->stream);
            });
            if (ss != ctx->stream) GAD_CK(cudaStreamWaitEvent(ctx->stream, ctx->ev_bias, 0));   // the column sums have read dPre
            GAD_RUN("spmm_bwd", l, spmm_bytes(p, y.fi, nnz_b), 2.0 * nnz_b * y.fi,
                    [&] { return launch_spmm(Ab, G2, y.ldi, G1, y.ldi, y.fi, nullptr, bf16_of(ctx), false, ctx->stream); });
            GAD_RUN("relu_mask", l, 12.0 * p.Np * y.fi, 1.0 * p.Np * y.fi,
                    [&] { return launch_relu_mask(G1, ctx->H(l), y.ldi, p.Np, scale, ctx->stream); });
            continue;
        }
        if (l > 0 && ss != ctx->stream) GAD_CK(cudaStreamWaitEvent(ctx->stream, ctx->ev_bias, 0));
        if (l > 0)
            GAD_RUN("gemm_dh", l, 4.0 * p.Np * (2.0 * y.fi + y.fo) + 4.0 * p.K * y.fi * y.fo, 2.0 * p.Np * y.fi * y.fo, [&] {
                if (ctx->use_tc)
                    return launch_gemm_rows_tc(&ctx->maps[kMapsPerLayer * l + 3], &ctx->maps[kMapsPerLayer * l + 4], &ctx->maps[kMapsPerLayer * l + 5], 1,
                                               ctx->cfg.gemm_mode == 0 ? 3 : 1, y.fo, y.fi, G1, y.ldi, ctx->at<RowSpan>(p.o_tiles),
                                               (int)p.tiles.size(), ctx->H(l), y.ldi, scale, nullptr, ctx->at<int32_t>(p.o_flags) + 1,
                                               ctx->num_sms, ctx->stream);
                return launch_gemm_rows_simt(1, G2, y.ldo, y.fo, params, p.pstride, y.w_int, y.ldw, y.fi, G1, y.ldi,
                                             ctx->at<RowSpan>(p.o_tiles), (int)p.tiles.size(), ctx->H(l), y.ldi, scale, nullptr,
                                             ctx->stream);
            });
    }
    return GAD_OK;
}

void pack_params(const Plan& p, const float* ext, float* blk) {
    std::fill(blk, blk + p.pstride, 0.f);
    for (const Layer& y : p.layers) {
        for (int i = 0; i < y.fi; ++i)
            std::memcpy(blk + y.w_int + (int64_t)i * y.ldw, ext + y.w_ext + (int64_t)i * y.fo, sizeof(float) * y.fo);
        std::memcpy(blk + y.b_int, ext + y.b_ext, sizeof(float) * y.fo);
    }
}
void unpack_params(const Plan& p, const float* blk, float* ext) {
    for (const Layer& y : p.layers) {
        for (int i = 0; i < y.fi; ++i)
            std::memcpy(ext + y.w_ext + (int64_t)i * y.fo, blk + y.w_int + (int64_t)i * y.ldw, sizeof(float) * y.fo);
        std::memcpy(ext + y.b_ext, blk + y.b_int, sizeof(float) * y.fo);
    }
}

uint64_t host_mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
    return z ^ (z >> 31);
}

// Default initialisation in the caller-visible layout [W_0, b_0, W_1, b_1, ...]: W_l uniform in (-a, a), a = sqrt(6 / (F_l +
// F_{l+1})) (Glorot), the i-th weight overall from the 53 top bits of mix(seed + G i) (splitmix64 stream); biases zero.
void default_params(const std::vector<int32_t>& dims, uint64_t seed, float* out) {
    uint64_t ctr = 0;
    int64_t o = 0;
    for (size_t l = 0; l + 1 < dims.size(); ++l) {
        const int64_t fi = dims[l], fo = dims[l + 1];
        const double a = std::sqrt(6.0 / (double)(fi + fo));
        for (int64_t i = 0; i < fi * fo; ++i) {
            const uint64_t h = host_mix64(seed + 0x9e3779b97f4a7c15ULL * (++ctr));
            out[o++] = (float)((2.0 * ((h >> 11) * (1.0 / 9007199254740992.0)) - 1.0) * a);
        }
        for (int64_t j = 0; j < fo; ++j) out[o++] = 0.f;
    }
}

int upload_sparse(gad_ctx* ctx, const std::vector<int32_t>& sub_off, const std::vector<int64_t>& rowptr, const std::vector<int32_t>& col,
                  const std::vector<float>& val,
                  size_t o_rowptr, size_t o_ecv, size_t o_fin, size_t o_items, SparseDev& out, int64_t forced_part = 0,
                  int64_t* part_entries = nullptr) {
    const Plan& p = ctx->p;
    std::vector<uint2> ecv(col.size());
    for (size_t e = 0; e < col.size(); ++e) {
        uint32_t bits;
        std::memcpy(&bits, &val[e], 4);
        ecv[e] = make_uint2((uint32_t)col[e], bits);
    }
    RowWork work;
    bin_rows(rowptr, sub_off, work, forced_part);
    if (part_entries) *part_entries = work.part_entries;
    if (work.slots > p.slots) return fail(ctx, GAD_ERR_OOM, "SpMM scratch slots exceed the planned count");
    GAD_CK(cudaMemcpyAsync(ctx->ws + o_rowptr, rowptr.data(), 8 * rowptr.size(), cudaMemcpyHostToDevice, ctx->stream));
    if (!ecv.empty()) GAD_CK(cudaMemcpyAsync(ctx->ws + o_ecv, ecv.data(), 8 * ecv.size(), cudaMemcpyHostToDevice, ctx->stream));
    if (!work.fin.empty())
        GAD_CK(cudaMemcpyAsync(ctx->ws + o_fin, work.fin.data(), 16 * work.fin.size(), cudaMemcpyHostToDevice, ctx->stream));
    if (!work.items.empty())
        GAD_CK(cudaMemcpyAsync(ctx->ws + o_items, work.items.data(), 16 * work.items.size(), cudaMemcpyHostToDevice, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));  // the host vectors above go out of scope
    out.rowptr = ctx->at<int64_t>(o_rowptr);
    out.ecv = ctx->at<uint2>(o_ecv);
    out.fin = ctx->at<int4>(o_fin);
    out.items = ctx->at<int4>(o_items);
    out.nitems = (int32_t)work.items.size();
    out.nrows = (int64_t)rowptr.size() - 1;
    out.scratch = ctx->at<float>(p.o_spmm_scratch);
    out.nfin = (int32_t)work.fin.size();
    return GAD_OK;
}

template <class T>
int upload(gad_ctx* ctx, size_t off, const std::vector<T>& v) {
    if (!v.empty()) GAD_CK(cudaMemcpyAsync(ctx->ws + off, v.data(), sizeof(T) * v.size(), cudaMemcpyHostToDevice, ctx->stream));
    return GAD_OK;
}

}  // namespace

extern "C" {

int gad_workspace_bytes(const gad_csr* g, const gad_partition* part, const gad_config* cfg, size_t* bytes) {
    if (!bytes) return GAD_ERR_ARG;
    std::string err;
    int64_t Np = 0, nnz = 0, slots = 0;
    int rc = store_sizes(g, part, &Np, &nnz, &slots, err);
    if (rc != GAD_OK) return fail(nullptr, rc, err);
    std::vector<int32_t> sub_off(part->K + 1, 0);
    std::vector<int64_t> core_count(part->K, 0);
    for (int32_t k = 0; k < part->K; ++k) {
        core_count[k] = part->core_ptr[k + 1] - part->core_ptr[k];
        sub_off[k + 1] = sub_off[k] + (int32_t)(core_count[k] + part->halo_ptr[k + 1] - part->halo_ptr[k]);
    }
    Plan p;
    rc = make_plan(p, g->n, part->K, sub_off, core_count, nnz, slots, cfg, err);
    if (rc != GAD_OK) return fail(nullptr, rc, err);
    *bytes = p.bytes;
    return GAD_OK;
}

int gad_create(gad_ctx** out, const gad_csr* g, const gad_partition* part, const float* X, const int32_t* labels,
               const uint8_t* split, const gad_config* cfg, const float* init_params, void* workspace, size_t workspace_bytes,
               void* stream) {
    if (!out) return GAD_ERR_ARG;
    *out = nullptr;
    if (!g || !part || !X || !labels || !split || !cfg || !workspace) return GAD_ERR_ARG;
    if (((uintptr_t)workspace & 255) != 0) return GAD_ERR_ARG;
    gad_ctx* ctx = new (std::nothrow) gad_ctx();
    if (!ctx) return GAD_ERR_OOM;
    struct Guard { gad_ctx*& c; bool ok = false; ~Guard() { if (!ok) { delete c; c = nullptr; } } } guard{ctx};
    ctx->stream = (cudaStream_t)stream;
    ctx->ws = (char*)workspace;
    ctx->cfg = *cfg;
    ctx->hoist = (cfg->flags & 2) != 0;
    GAD_CK(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    GAD_CK(cudaStreamCreateWithFlags(&ctx->side_stream, cudaStreamNonBlocking));
    for (cudaEvent_t* e : {&ctx->ev_fork, &ctx->ev_split, &ctx->ev_g1, &ctx->ev_bias, &ctx->ev_join})
        GAD_CK(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
    for (int i = 0; i < 2; ++i) {
        GAD_CK(cudaEventCreateWithFlags(&ctx->ev_copied[i], cudaEventDisableTiming));
        GAD_CK(cudaEventCreateWithFlags(&ctx->ev_gathered[i], cudaEventDisableTiming));
    }
    HostStore st;
    int rc = build_store(g, part, true, st, ctx->err);
    if (rc != GAD_OK) return fail(ctx, rc, ctx->err);
    const int64_t slots = std::max(count_slots(st.rowptr), st.symmetric ? 0 : count_slots(st.t_rowptr));
    rc = make_plan(ctx->p, g->n, part->K, st.sub_off, st.core_count, st.nnz, slots, cfg, ctx->err);
    if (rc != GAD_OK) return fail(ctx, rc, ctx->err);
    ctx->cfg.dims = ctx->p.dims.data();
    const Plan& p = ctx->p;
    if (workspace_bytes < p.bytes) return fail(ctx, GAD_ERR_OOM, "workspace smaller than gad_workspace_bytes");
    const int C = p.dims[p.L];
    for (int32_t u = 0; u < g->n; ++u) {
        if (labels[u] < 0 || labels[u] >= C) return fail(ctx, GAD_ERR_RANGE, "label out of range");
        if (split[u] > 2) return fail(ctx, GAD_ERR_RANGE, "split value out of range");
    }
    ctx->symmetric = st.symmetric;
    ctx->sub_off = st.sub_off;
    ctx->gid = st.gid;

    int64_t part_t = 0;   // part length of the store the backward aggregation reads
    rc = upload_sparse(ctx, st.sub_off, st.rowptr, st.col, st.val, p.o_rowptr, p.o_ecv, p.o_fin, p.o_items, ctx->A, 0, &part_t);
    if (rc != GAD_OK) return rc;
    if (!st.symmetric) {
        rc = upload_sparse(ctx, st.sub_off, st.t_rowptr, st.t_col, st.t_val, p.o_trowptr, p.o_tecv, p.o_tfin, p.o_titems, ctx->At, 0, &part_t);
        if (rc != GAD_OK) return rc;
    }
    // per-row labels and loss mask, per-subgraph degree sums and training counts
    std::vector<int32_t> label((size_t)p.Np);
    std::vector<uint8_t> train((size_t)p.Np);
    std::vector<int64_t> deg_sum(p.K, 0), deg_sq(p.K, 0);
    std::vector<float> inv_ntrain(p.K, 0.f);
    ctx->ntrain.assign(p.K, 0);
    ctx->ntrain_total = 0;
    for (int32_t k = 0; k < p.K; ++k) {
        for (int64_t r = st.sub_off[k]; r < st.sub_off[k + 1]; ++r) {
            const int32_t u = st.gid[r];
            label[r] = labels[u];
            const bool core = (r - st.sub_off[k]) < st.core_count[k];
            train[r] = (uint8_t)(core && split[u] == 0);
            ctx->ntrain[k] += train[r];
            deg_sum[k] += st.deg[r];
            deg_sq[k] += (int64_t)st.deg[r] * st.deg[r];
        }
        inv_ntrain[k] = ctx->ntrain[k] > 0 ? 1.f / (float)ctx->ntrain[k] : 0.f;
        ctx->ntrain_total += ctx->ntrain[k];
    }
    if (!(cfg->flags & 64)) {
        // the transposed store restricted to the columns that carry loss, rows cut as the full one cuts them (so its
        // scratch slots are no more than the planned ones)
        const std::vector<int64_t>& rp = st.symmetric ? st.rowptr : st.t_rowptr;
        const std::vector<int32_t>& cl = st.symmetric ? st.col : st.t_col;
        const std::vector<float>& vl = st.symmetric ? st.val : st.t_val;
        std::vector<int64_t> grp((size_t)p.Np + 1, 0);
        std::vector<int32_t> gcl;
        std::vector<float> gvl;
        for (int64_t r = 0; r < p.Np; ++r) {
            for (int64_t e = rp[r]; e < rp[r + 1]; ++e)
                if (train[(size_t)cl[e]]) { gcl.push_back(cl[e]); gvl.push_back(vl[e]); }
            grp[(size_t)r + 1] = (int64_t)gcl.size();
        }
        rc = upload_sparse(ctx, st.sub_off, grp, gcl, gvl, p.o_growptr, p.o_gecv, p.o_gfin, p.o_gitems, ctx->Ag, part_t);
        if (rc != GAD_OK) return rc;
        ctx->use_loss_rows = true;
        ctx->nnz_loss_rows = (int64_t)gcl.size();
    }
    if ((rc = upload(ctx, p.o_sub_off, st.sub_off)) || (rc = upload(ctx, p.o_gid, st.gid)) || (rc = upload(ctx, p.o_deg, st.deg)) ||
        (rc = upload(ctx, p.o_label, label)) || (rc = upload(ctx, p.o_train, train)) || (rc = upload(ctx, p.o_deg_sum, deg_sum)) ||
        (rc = upload(ctx, p.o_deg_sq, deg_sq)) || (rc = upload(ctx, p.o_inv_ntrain, inv_ntrain)) ||
        (rc = upload(ctx, p.o_tiles, p.tiles)) || (rc = upload(ctx, p.o_chunks, p.chunks)) ||
        (rc = upload(ctx, p.o_chunk_ptr, p.chunk_ptr)) || (rc = upload(ctx, p.o_dw_chunks, p.dw_chunks)) ||
        (rc = upload(ctx, p.o_dw_chunk_ptr, p.dw_chunk_ptr)) || (rc = upload(ctx, p.o_core_spans, p.core_spans)) ||
        (rc = upload(ctx, p.o_pair_ptr, p.pair_ptr)) || (rc = upload(ctx, p.o_gram_ptr, p.gram_ptr)) || (rc = upload(ctx, p.o_nchunks, p.nchunks)) ||
        (rc = upload(ctx, p.o_nchunk_ptr, p.nchunk_ptr)))
        return rc;
    // features: graph order -> staging -> store-row order with zero pad columns
    GAD_CK(cudaMemcpyAsync(ctx->ws + p.o_stage, X, 4 * (size_t)g->n * p.dims[0], cudaMemcpyHostToDevice, ctx->stream));
    GAD_CK(launch_gather_rows(ctx->at<float>(p.o_stage), p.dims[0], ctx->at<int32_t>(p.o_gid), p.Np, ctx->H(0), p.ld[0], ctx->stream));
    // parameters: K identical padded copies
    std::vector<float> ext((size_t)p.P);
    if (init_params) std::memcpy(ext.data(), init_params, sizeof(float) * (size_t)p.P);
    else default_params(p.dims, cfg->seed, ext.data());
    ctx->host_block.assign((size_t)p.pstride, 0.f);
    pack_params(p, ext.data(), ctx->host_block.data());
    for (int32_t k = 0; k < p.K; ++k)
        GAD_CK(cudaMemcpyAsync(ctx->at<float>(p.o_params) + (int64_t)k * p.pstride, ctx->host_block.data(), 4 * (size_t)p.pstride,
                               cudaMemcpyHostToDevice, ctx->stream));
    GAD_CK(cudaMemsetAsync(ctx->ws + p.o_grads, 0, 4 * (size_t)p.K * p.pstride, ctx->stream));
    GAD_CK(cudaMemsetAsync(ctx->ws + p.o_flags, 0, 16, ctx->stream));
    // tensor-core path: operand copies start at zero (their pad columns are never written) and get TMA descriptors
    {
        int dev = 0;
        GAD_CK(cudaGetDevice(&dev));
        cudaDeviceProp prop;
        GAD_CK(cudaGetDeviceProperties(&prop, dev));
        ctx->num_sms = prop.multiProcessorCount;
        ctx->use_tc = (cfg->flags & 1) == 0 && prop.major == 10 && p.Np > 0;
    }
    if (ctx->cfg.zeta_mode == 1) {
        ctx->use_gram = ctx->use_tc && !p.gram_ptr.empty();
        if (ctx->use_gram && !(tc_make_map(&ctx->map_xhi, ctx->at<float>(p.o_xhi), p.dims[0], p.Np, 0, 4ull * p.ld[0], 0, 128) &&
                               tc_make_map(&ctx->map_xlo, ctx->at<float>(p.o_xlo), p.dims[0], p.Np, 0, 4ull * p.ld[0], 0, 128)))
            return fail(ctx, GAD_ERR_CUDA, "cuTensorMapEncodeTiled failed");
        if (!ctx->use_gram && !p.pair_alu_ok)
            return fail(ctx, GAD_ERR_UNSUPPORTED, "zeta_mode 1 without the tensor-core kernel takes subgraphs of at most " +
                                                      std::to_string(kZetaPairMaxRows) + " rows");
    }
    if (ctx->use_tc) {
        ctx->maps.resize((size_t)kMapsPerLayer * p.L);
        bool ok = true;
        for (int l = 0; l < p.L && ok; ++l) {
            const Layer& y = p.layers[l];
            GAD_CK(cudaMemsetAsync(ctx->ws + p.o_w_hi[l], 0, 4 * (size_t)p.K * y.fi * y.ldw, ctx->stream));
            GAD_CK(cudaMemsetAsync(ctx->ws + p.o_w_lo[l], 0, 4 * (size_t)p.K * y.fi * y.ldw, ctx->stream));
            GAD_CK(cudaMemsetAsync(ctx->ws + p.o_wt_hi[l], 0, 4 * (size_t)p.K * y.fo * y.ldi, ctx->stream));
            GAD_CK(cudaMemsetAsync(ctx->ws + p.o_wt_lo[l], 0, 4 * (size_t)p.K * y.fo * y.ldi, ctx->stream));
            gad_ctx::TMap* m = &ctx->maps[(size_t)kMapsPerLayer * l];
            // forward: A = H^(l) [Np x fi], B = W^T copies [K][fo][fi]
            const bool agg_first = p.agg_first[l] != 0;   // then the transform and the weight gradient read A~ H^(l), dW and dH read dPre (G1)
            float* Hin = agg_first ? ctx->at<float>(p.o_P[l]) : ctx->H(l);
            ok = ok && tc_make_map(&m[0], Hin, y.fi, p.Np, 0, 4ull * y.ldi, 0, 128);
            ok = ok && tc_make_map(&m[1], ctx->at<float>(p.o_wt_hi[l]), y.fi, y.fo, p.K, 4ull * y.ldi, 4ull * y.fo * y.ldi, tc_bn_for(y.fo));
            ok = ok && tc_make_map(&m[2], ctx->at<float>(p.o_wt_lo[l]), y.fi, y.fo, p.K, 4ull * y.ldi, 4ull * y.fo * y.ldi, tc_bn_for(y.fo));
            // input gradient: A = dZ [Np x fo] (in G2), B = W copies [K][fi][fo]
            ok = ok && tc_make_map(&m[3], ctx->at<float>(agg_first ? p.o_G1 : p.o_G2), y.fo, p.Np, 0, 4ull * y.ldo, 0, 128);
            ok = ok && tc_make_map(&m[4], ctx->at<float>(p.o_w_hi[l]), y.fo, y.fi, p.K, 4ull * y.ldw, 4ull * y.fi * y.ldw, tc_bn_for(y.fi));
            ok = ok && tc_make_map(&m[5], ctx->at<float>(p.o_w_lo[l]), y.fo, y.fi, p.K, 4ull * y.ldw, 4ull * y.fi * y.ldw, tc_bn_for(y.fi));
            // weight gradient: 32-row tiles of H^(l) and of dZ (in G2)
            ok = ok && tc_make_map(&m[6], Hin, y.fi, p.Np, 0, 4ull * y.ldi, 0, tc_tn_rows(), true);
            ok = ok && tc_make_map(&m[7], ctx->at<float>(agg_first ? p.o_G1 : p.o_G2), y.fo, p.Np, 0, 4ull * y.ldo, 0, tc_tn_rows(), true);
        }
        if (!ok) return fail(ctx, GAD_ERR_CUDA, "cuTensorMapEncodeTiled failed");
    }
    GAD_CK(cudaMemsetAsync(ctx->ws + p.o_loss, 0, 4 * (size_t)(p.K + 1), ctx->stream));
    GAD_CK(cudaMemsetAsync(ctx->ws + p.o_zeta, 0, 8 * (size_t)p.K, ctx->stream));   // empty subgraphs keep zeta = 0
    GAD_CK(cudaMemsetAsync(ctx->ws + p.o_counters, 0, 4 * (size_t)(1 + 2 * p.K), ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    guard.ok = true;
    *out = ctx;
    return GAD_OK;
}

int gad_default_params(int32_t L, const int32_t* dims, uint64_t seed, float* out) {
    if (L < 1 || !dims || !out) return GAD_ERR_ARG;
    for (int l = 0; l <= L; ++l)
        if (dims[l] < 1) return GAD_ERR_ARG;
    default_params(std::vector<int32_t>(dims, dims + L + 1), seed, out);
    return GAD_OK;
}

int gad_get_loss(gad_ctx* ctx, float* loss_out) {
    if (!ctx || !loss_out) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    int32_t flags[2] = {0, 0};
    GAD_CK(cudaMemcpyAsync(loss_out, ctx->ws + p.o_loss, 4 * (size_t)(p.K + 1), cudaMemcpyDeviceToHost, ctx->stream));
    GAD_CK(cudaMemcpyAsync(flags, ctx->ws + p.o_flags, 8, cudaMemcpyDeviceToHost, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    const int32_t flag = flags[0];
    if (flags[1]) {
        GAD_CK(cudaMemsetAsync(ctx->ws + p.o_flags, 0, 8, ctx->stream));
        return fail(ctx, GAD_ERR_DEVICE_TIMEOUT, "a bounded device-side wait ran out (role " + std::to_string(flags[1]) + ")");
    }
    if (flag) {
        GAD_CK(cudaMemsetAsync(ctx->ws + p.o_flags, 0, 4, ctx->stream));
        return fail(ctx, GAD_ERR_NONFINITE, "a subgraph loss is NaN or infinite");
    }
    return GAD_OK;
}

static int train_epoch(gad_ctx* ctx, float* loss_out, bool consensus);

int gad_train_epoch(gad_ctx* ctx, float* loss_out) { return train_epoch(ctx, loss_out, true); }
int gad_train_epoch_local(gad_ctx* ctx, float* loss_out) { return train_epoch(ctx, loss_out, false); }

// Every launch of one epoch, on the context's two streams.
static int enqueue_epoch(gad_ctx* ctx, bool consensus) {
    const Plan& p = ctx->p;
    cudaStream_t ss = side_of(ctx);
    int rc = hand_over(ctx, ctx->stream, ss, ctx->ev_fork);   // this epoch's side work follows everything enqueued so far
    if (rc != GAD_OK) return rc;
    if ((rc = forward_pass(ctx, true, ss)) != GAD_OK) return rc;
    // zeta beside the forward pass; with zeta_mode 2 it reads this pass's activations, so it follows it (beside the backward pass)
    if (ctx->cfg.zeta_mode == 2 && (rc = hand_over(ctx, ctx->stream, ss, ctx->ev_fork)) != GAD_OK) return rc;
    if (ss != ctx->stream && (rc = zeta_pass(ctx, ss)) != GAD_OK) return rc;
    const int C = p.dims[p.L];
    GAD_RUN("softmax_xent", -1, 8.0 * p.Np * C, 0.0, [&] {
        return launch_softmax_xent(ctx->H(p.L), p.ld[p.L], C, ctx->at<int32_t>(p.o_label), ctx->at<uint8_t>(p.o_train),
                                   ctx->at<RowSpan>(p.o_chunks), (int)p.chunks.size(), ctx->at<float>(p.o_inv_ntrain),
                                   ctx->at<float>(p.o_G1), ctx->at<float>(p.o_loss_partial), ctx->at<int32_t>(p.o_chunk_ptr), p.K,
                                   ctx->ntrain_total > 0 ? 1.f / (float)ctx->ntrain_total : 0.f, ctx->at<float>(p.o_loss),
                                   ctx->at<int32_t>(p.o_flags), ctx->at<unsigned>(p.o_counters), ctx->stream);
    });
    if ((rc = backward_pass(ctx, ss)) != GAD_OK) return rc;
    if (ss == ctx->stream && (rc = zeta_pass(ctx, ss)) != GAD_OK) return rc;
    if ((rc = hand_over(ctx, ss, ctx->stream, ctx->ev_join)) != GAD_OK) return rc;
    if (consensus)
        GAD_RUN("sgd_consensus", -1, 12.0 * p.K * p.Pint, 4.0 * p.K * p.Pint, [&] {
            return launch_sgd_consensus(ctx->at<float>(p.o_params), ctx->at<float>(p.o_grads), p.pstride, p.pstride, p.K, ctx->cfg.lr,
                                        ctx->at<double>(p.o_zeta), ctx->cfg.weighted, 1, ctx->at<int32_t>(p.o_flags) + 1, ctx->stream);
        });
    return GAD_OK;
}

// An epoch's launch sequence depends on nothing that changes from epoch to epoch unless dropout is on (the mask is
// indexed by the epoch) or A~ H^(0) is being kept (its first epoch differs), so it can be captured into a CUDA graph
// once and replayed: one submission instead of about twenty, and no gaps between dependent kernels.  Needs a stream
// that can be captured (not the legacy default stream).
static bool graph_allowed(const gad_ctx* ctx) {
    return (ctx->cfg.flags & 8) == 0 && ctx->stream != nullptr && ctx->stream != cudaStreamLegacy && ctx->stream != cudaStreamPerThread &&
           !ctx->profiling && !ctx->hoist && !(ctx->cfg.dropout > 0.f) && ctx->direct_epochs >= 1;
}

static void capture_epoch(gad_ctx* ctx, bool consensus, gad_ctx::EpochGraph& eg) {
    if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        cudaGetLastError();
        eg.failed = true;   // e.g. the caller is capturing this stream already: the launches then go into that capture
        return;
    }
    const int64_t before = g_kernel_launches.load();
    const int rc = enqueue_epoch(ctx, consensus);
    cudaGraph_t graph = nullptr;
    const cudaError_t e = cudaStreamEndCapture(ctx->stream, &graph);
    // (a context belongs to one host thread, so the difference is this capture's own launches unless other threads
    // launched meanwhile; only this capture's share is taken back: nothing of it has run yet)
    const int64_t kernels = g_kernel_launches.load() - before;
    g_kernel_launches -= kernels;
    if (rc == GAD_OK && e == cudaSuccess && graph && cudaGraphInstantiate(&eg.exec, graph, 0) == cudaSuccess) {
        eg.kernels = kernels;
    } else {
        eg.exec = nullptr;
        eg.failed = true;
    }
    if (graph) cudaGraphDestroy(graph);
    cudaGetLastError();
}

static int train_epoch(gad_ctx* ctx, float* loss_out, bool consensus) {
    if (!ctx) return GAD_ERR_ARG;
    gad_ctx::EpochGraph& eg = ctx->graphs[consensus ? 1 : 0];
    bool done = false;
    cudaStreamCaptureStatus outer = cudaStreamCaptureStatusNone;   // a caller capturing the stream gets plain launches into its capture
    if (graph_allowed(ctx) && !eg.failed && cudaStreamIsCapturing(ctx->stream, &outer) == cudaSuccess &&
        outer == cudaStreamCaptureStatusNone) {
        if (!eg.exec) capture_epoch(ctx, consensus, eg);
        if (eg.exec) {
            GAD_CK(cudaGraphLaunch(eg.exec, ctx->stream));
            g_kernel_launches += eg.kernels;
            done = true;
        }
    }
    if (!done) {
        int rc = enqueue_epoch(ctx, consensus);
        if (rc != GAD_OK) return rc;
        ctx->direct_epochs += 1;
    }
    ctx->epoch += 1;
    if (loss_out) return gad_get_loss(ctx, loss_out);
    return GAD_OK;
}

int gad_forward(gad_ctx* ctx, float* logits_out) {
    if (!ctx || !logits_out) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    int rc = forward_pass(ctx, false, ctx->stream);
    if (rc != GAD_OK) return rc;
    const int C = p.dims[p.L];
    GAD_CK(cudaMemsetAsync(ctx->ws + p.o_stage, 0, 4 * (size_t)p.n * C, ctx->stream));
    GAD_CK(launch_scatter_core(ctx->H(p.L), p.ld[p.L], C, ctx->at<int32_t>(p.o_gid), ctx->at<RowSpan>(p.o_core_spans),
                               (int)p.core_spans.size(), ctx->at<float>(p.o_stage), ctx->stream));
    GAD_CK(cudaMemcpyAsync(logits_out, ctx->ws + p.o_stage, 4 * (size_t)p.n * C, cudaMemcpyDeviceToHost, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    return GAD_OK;
}

int gad_subgraph_weights(gad_ctx* ctx, float* zeta_out, float* w_out) {
    if (!ctx) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    int rc = zeta_pass(ctx, ctx->stream);
    if (rc != GAD_OK) return rc;
    GAD_CK(launch_weights(ctx->at<double>(p.o_zeta), p.K, ctx->cfg.weighted, ctx->at<float>(p.o_zeta_f), ctx->at<float>(p.o_w_f),
                          ctx->stream));
    if (zeta_out) GAD_CK(cudaMemcpyAsync(zeta_out, ctx->ws + p.o_zeta_f, 4 * (size_t)p.K, cudaMemcpyDeviceToHost, ctx->stream));
    if (w_out) GAD_CK(cudaMemcpyAsync(w_out, ctx->ws + p.o_w_f, 4 * (size_t)p.K, cudaMemcpyDeviceToHost, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    return GAD_OK;
}

int gad_consensus(gad_ctx* ctx) {
    if (!ctx) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    int rc = zeta_pass(ctx, ctx->stream);
    if (rc != GAD_OK) return rc;
    GAD_RUN("consensus", -1, 8.0 * p.K * p.Pint, 2.0 * p.K * p.Pint, [&] {
        return launch_sgd_consensus(ctx->at<float>(p.o_params), ctx->at<float>(p.o_grads), p.pstride, p.pstride, p.K, 0.f,
                                    ctx->at<double>(p.o_zeta), ctx->cfg.weighted, 0, ctx->at<int32_t>(p.o_flags) + 1, ctx->stream);
    });
    return GAD_OK;
}

int gad_get_train_counts(const gad_ctx* ctx, int64_t* counts) {
    if (!ctx || !counts) return GAD_ERR_ARG;
    for (int32_t k = 0; k < ctx->p.K; ++k) counts[k] = ctx->ntrain[(size_t)k];
    return GAD_OK;
}

int gad_consensus_floats(const gad_ctx* ctx, int64_t* count) {
    if (!ctx || !count) return GAD_ERR_ARG;
    *count = ctx->p.pstride;
    return GAD_OK;
}

int gad_consensus_partial(gad_ctx* ctx, double total, int32_t with_step, float* dev_out) {
    if (!ctx || !dev_out || !(total > 0.0) || ((uintptr_t)dev_out & 15) != 0) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    if (!with_step) {   // no epoch has necessarily run: evaluate zeta here
        int rc = zeta_pass(ctx, ctx->stream);
        if (rc != GAD_OK) return rc;
    }
    GAD_RUN("consensus_partial", -1, (with_step ? 8.0 : 4.0) * p.K * p.Pint + 4.0 * p.Pint, 4.0 * p.K * p.Pint, [&] {
        return launch_consensus_partial(ctx->at<float>(p.o_params), ctx->at<float>(p.o_grads), p.pstride, p.pstride, p.K, ctx->cfg.lr,
                                        ctx->at<double>(p.o_zeta), ctx->cfg.weighted, with_step ? 1 : 0, total, dev_out, ctx->at<int32_t>(p.o_flags) + 1,
                                        ctx->stream);
    });
    return GAD_OK;
}

int gad_consensus_apply(gad_ctx* ctx, const float* dev_in) {
    if (!ctx || !dev_in || ((uintptr_t)dev_in & 15) != 0) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    GAD_RUN("consensus_apply", -1, 4.0 * (p.K + 1) * p.Pint, 0.0, [&] {
        return launch_consensus_apply(ctx->at<float>(p.o_params), p.pstride, p.pstride, p.K, dev_in, ctx->at<int32_t>(p.o_flags) + 1, ctx->stream);
    });
    return GAD_OK;
}

int gad_export_params(gad_ctx* ctx, int32_t k, float* dev_out) {
    if (!ctx || !dev_out || k < 0 || k >= ctx->p.K) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    GAD_CK(cudaMemcpyAsync(dev_out, ctx->at<float>(p.o_params) + (int64_t)k * p.pstride, 4 * (size_t)p.pstride, cudaMemcpyDeviceToDevice,
                           ctx->stream));
    return GAD_OK;
}

int gad_param_count(const gad_ctx* ctx, int64_t* P) {
    if (!ctx || !P) return GAD_ERR_ARG;
    *P = ctx->p.P;
    return GAD_OK;
}

static int get_block(gad_ctx* ctx, size_t base, int32_t k, float* out) {
    if (!ctx || !out || k < 0 || k >= ctx->p.K) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    GAD_CK(cudaMemcpyAsync(ctx->host_block.data(), ctx->at<float>(base) + (int64_t)k * p.pstride, 4 * (size_t)p.pstride,
                           cudaMemcpyDeviceToHost, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    unpack_params(p, ctx->host_block.data(), out);
    return GAD_OK;
}
int gad_get_params(gad_ctx* ctx, int32_t k, float* out) { return get_block(ctx, ctx ? ctx->p.o_params : 0, k, out); }
int gad_get_grads(gad_ctx* ctx, int32_t k, float* out) { return get_block(ctx, ctx ? ctx->p.o_grads : 0, k, out); }

int gad_set_params(gad_ctx* ctx, int32_t k, const float* in) {
    if (!ctx || !in || k < 0 || k >= ctx->p.K) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    pack_params(p, in, ctx->host_block.data());
    GAD_CK(cudaMemcpyAsync(ctx->at<float>(p.o_params) + (int64_t)k * p.pstride, ctx->host_block.data(), 4 * (size_t)p.pstride,
                           cudaMemcpyHostToDevice, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    return GAD_OK;
}

int gad_store_sizes(const gad_ctx* ctx, int64_t* n_prime, int64_t* nnz_prime) {
    if (!ctx) return GAD_ERR_ARG;
    if (n_prime) *n_prime = ctx->p.Np;
    if (nnz_prime) *nnz_prime = ctx->p.nnz;
    return GAD_OK;
}

int gad_get_store(gad_ctx* ctx, int64_t* rowptr, int32_t* col, float* val, int32_t* sub_off, int32_t* gid, int32_t* deg) {
    if (!ctx) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    if (rowptr) GAD_CK(cudaMemcpyAsync(rowptr, ctx->ws + p.o_rowptr, 8 * (size_t)(p.Np + 1), cudaMemcpyDeviceToHost, ctx->stream));
    if (sub_off) GAD_CK(cudaMemcpyAsync(sub_off, ctx->ws + p.o_sub_off, 4 * (size_t)(p.K + 1), cudaMemcpyDeviceToHost, ctx->stream));
    if (gid && p.Np) GAD_CK(cudaMemcpyAsync(gid, ctx->ws + p.o_gid, 4 * (size_t)p.Np, cudaMemcpyDeviceToHost, ctx->stream));
    if (deg && p.Np) GAD_CK(cudaMemcpyAsync(deg, ctx->ws + p.o_deg, 4 * (size_t)p.Np, cudaMemcpyDeviceToHost, ctx->stream));
    std::vector<uint2> ecv;
    if ((col || val) && p.nnz) {
        ecv.resize((size_t)p.nnz);
        GAD_CK(cudaMemcpyAsync(ecv.data(), ctx->ws + p.o_ecv, 8 * (size_t)p.nnz, cudaMemcpyDeviceToHost, ctx->stream));
    }
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    for (size_t e = 0; e < ecv.size(); ++e) {
        if (col) col[e] = (int32_t)ecv[e].x;
        if (val) std::memcpy(&val[e], &ecv[e].y, 4);
    }
    return GAD_OK;
}

int gad_get_activation(gad_ctx* ctx, int32_t l, float* out) {
    if (!ctx || !out || l < 0 || l > ctx->p.L) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    if (p.Np == 0) return GAD_OK;
    GAD_CK(cudaMemcpy2DAsync(out, 4 * (size_t)p.dims[l], ctx->H(l), 4 * (size_t)p.ld[l], 4 * (size_t)p.dims[l], (size_t)p.Np,
                             cudaMemcpyDeviceToHost, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    return GAD_OK;
}

int gad_set_inputs(gad_ctx* ctx, const float* X, const int32_t* labels) {
    if (!ctx) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    if (!X && !labels) return GAD_OK;
    if (labels) {   // the loss kernel indexes a row of logits with the label: same range check as gad_create, before anything is enqueued
        const int C = p.dims[p.L];
        for (int32_t u = 0; u < p.n; ++u)
            if (labels[u] < 0 || labels[u] >= C) return fail(ctx, GAD_ERR_RANGE, "label out of range at node " + std::to_string(u));
    }
    // The copy goes out on its own stream into one of two staging pairs, so it can overlap the epoch that is still
    // running on the context's stream; the gathers then run on the context's stream, after the copy.
    const int b = ctx->stage_idx;
    const size_t o_x = b ? p.o_stage2 : p.o_stage, o_l = b ? p.o_stage_lab2 : p.o_stage_lab;
    GAD_CK(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_gathered[b], 0));   // the pair's previous contents have been consumed
    if (X) GAD_CK(cudaMemcpyAsync(ctx->ws + o_x, X, 4 * (size_t)p.n * p.dims[0], cudaMemcpyHostToDevice, ctx->copy_stream));
    if (labels) GAD_CK(cudaMemcpyAsync(ctx->ws + o_l, labels, 4 * (size_t)p.n, cudaMemcpyHostToDevice, ctx->copy_stream));
    GAD_CK(cudaEventRecord(ctx->ev_copied[b], ctx->copy_stream));
    GAD_CK(cudaStreamWaitEvent(ctx->stream, ctx->ev_copied[b], 0));
    if (X) {
        GAD_RUN("gather_features", -1, 8.0 * p.Np * p.dims[0], 0.0, [&] {
            return launch_gather_rows(ctx->at<float>(o_x), p.dims[0], ctx->at<int32_t>(p.o_gid), p.Np, ctx->H(0), p.ld[0],
                                      ctx->stream);
        });
        ctx->P_valid = false;   // A~ H^(0) is aggregated again by the next forward pass
    }
    if (labels) {
        GAD_RUN("gather_labels", -1, 8.0 * p.Np, 0.0, [&] {
            return launch_gather_labels(ctx->at<int32_t>(o_l), ctx->at<int32_t>(p.o_gid), p.Np, ctx->at<int32_t>(p.o_label),
                                        ctx->stream);
        });
    }
    GAD_CK(cudaEventRecord(ctx->ev_gathered[b], ctx->stream));
    ctx->stage_idx ^= 1;
    return GAD_OK;
}

int gad_read_loss_async(gad_ctx* ctx, float* loss_out) {
    if (!ctx || !loss_out) return GAD_ERR_ARG;
    GAD_CK(cudaMemcpyAsync(loss_out, ctx->ws + ctx->p.o_loss, 4 * (size_t)(ctx->p.K + 1), cudaMemcpyDeviceToHost, ctx->stream));
    return GAD_OK;
}

int gad_synchronize(gad_ctx* ctx) {
    if (!ctx) return GAD_ERR_ARG;
    GAD_CK(cudaStreamSynchronize(ctx->copy_stream));
    GAD_CK(cudaStreamSynchronize(ctx->side_stream));
    int32_t timed_out = 0;
    GAD_CK(cudaMemcpyAsync(&timed_out, ctx->ws + ctx->p.o_flags + 4, 4, cudaMemcpyDeviceToHost, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    if (timed_out) {
        GAD_CK(cudaMemsetAsync(ctx->ws + ctx->p.o_flags + 4, 0, 4, ctx->stream));
        return fail(ctx, GAD_ERR_DEVICE_TIMEOUT, "a bounded device-side wait ran out (role " + std::to_string(timed_out) + ")");
    }
    return GAD_OK;
}

int gad_check_store(gad_ctx* ctx, int64_t* violations) {
    if (!ctx || !violations) return GAD_ERR_ARG;
    const Plan& p = ctx->p;
    // two 64-bit words of the loss-partial buffer serve as the counters (nothing of an epoch is in flight after the wait below)
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    unsigned long long* bad = ctx->at<unsigned long long>(p.o_loss_partial);
    const unsigned long long init[2] = {0ull, ~0ull};
    GAD_CK(cudaMemcpyAsync(bad, init, 16, cudaMemcpyHostToDevice, ctx->stream));
    GAD_CK(launch_check_store(ctx->A, p.nnz, p.slots, ctx->at<int32_t>(p.o_sub_off), p.K, bad, ctx->stream));
    if (!ctx->symmetric) GAD_CK(launch_check_store(ctx->At, p.nnz, p.slots, ctx->at<int32_t>(p.o_sub_off), p.K, bad, ctx->stream));
    if (ctx->use_loss_rows)
        GAD_CK(launch_check_store(ctx->Ag, ctx->nnz_loss_rows, p.slots, ctx->at<int32_t>(p.o_sub_off), p.K, bad, ctx->stream));
    unsigned long long out[2] = {0, 0};
    GAD_CK(cudaMemcpyAsync(out, bad, 16, cudaMemcpyDeviceToHost, ctx->stream));
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    *violations = (int64_t)out[0];
    if (out[0]) return fail(ctx, GAD_ERR_RANGE, "store self-check: " + std::to_string(out[0]) + " index violations, first at work-list position " +
                                                    std::to_string(out[1] - 1));
    return GAD_OK;
}

int gad_debug_expire_wait(gad_ctx* ctx, uint32_t polls) {
    if (!ctx || polls < 1 || polls > 65536) return GAD_ERR_ARG;
    GAD_CK(launch_expire_wait(ctx->at<int32_t>(ctx->p.o_flags) + 1, polls, ctx->stream));
    return GAD_OK;
}

int gad_get_epoch(const gad_ctx* ctx, int64_t* epoch) {
    if (!ctx || !epoch) return GAD_ERR_ARG;
    *epoch = ctx->epoch;
    return GAD_OK;
}
int gad_set_epoch(gad_ctx* ctx, int64_t epoch) {
    if (!ctx || epoch < 0) return GAD_ERR_ARG;
    ctx->epoch = epoch;
    return GAD_OK;
}

static int prof_drain(gad_ctx* ctx) {
    GAD_CK(cudaStreamSynchronize(ctx->stream));
    for (auto& e : ctx->prof) {
        for (auto& pr : e.pending) {
            float ms = 0.f;
            GAD_CK(cudaEventElapsedTime(&ms, pr.first, pr.second));
            e.ms += ms;
            e.launches += 1;
            cudaEventDestroy(pr.first);
            cudaEventDestroy(pr.second);
        }
        e.pending.clear();
    }
    return GAD_OK;
}

int gad_profile_enable(gad_ctx* ctx, int32_t on) {
    if (!ctx) return GAD_ERR_ARG;
    ctx->profiling = on != 0;
    return GAD_OK;
}
int gad_profile_reset(gad_ctx* ctx) {
    if (!ctx) return GAD_ERR_ARG;
    int rc = prof_drain(ctx);
    ctx->prof.clear();
    return rc;
}
int gad_profile_count(const gad_ctx* ctx, int32_t* count) {
    if (!ctx || !count) return GAD_ERR_ARG;
    *count = (int32_t)ctx->prof.size();
    return GAD_OK;
}
int gad_profile_read(gad_ctx* ctx, int32_t i, char* name64, int64_t* launches, double* total_ms, double* bytes_per_launch,
                     double* flops_per_launch) {
    if (!ctx || i < 0 || i >= (int32_t)ctx->prof.size()) return GAD_ERR_ARG;
    int rc = prof_drain(ctx);
    if (rc != GAD_OK) return rc;
    const ProfEntry& e = ctx->prof[i];
    if (name64) { std::strncpy(name64, e.name.c_str(), 63); name64[63] = 0; }
    if (launches) *launches = e.launches;
    if (total_ms) *total_ms = e.ms;
    if (bytes_per_launch) *bytes_per_launch = e.bytes;
    if (flops_per_launch) *flops_per_launch = e.flops;
    return GAD_OK;
}

int gad_launch_count(int64_t* launches) {
    if (!launches) return GAD_ERR_ARG;
    *launches = gad::g_kernel_launches.load();
    return GAD_OK;
}

const char* gad_last_error(const gad_ctx* ctx) { return ctx ? ctx->err.c_str() : g_last_error.c_str(); }

void gad_destroy(gad_ctx* ctx) {
    if (!ctx) return;
    for (auto& eg : ctx->graphs)
        if (eg.exec) cudaGraphExecDestroy(eg.exec);
    for (auto& e : ctx->prof)
        for (auto& pr : e.pending) { cudaEventDestroy(pr.first); cudaEventDestroy(pr.second); }
    if (ctx->copy_stream) { cudaStreamSynchronize(ctx->copy_stream); cudaStreamDestroy(ctx->copy_stream); }
    if (ctx->side_stream) { cudaStreamSynchronize(ctx->side_stream); cudaStreamDestroy(ctx->side_stream); }
    for (cudaEvent_t e : {ctx->ev_fork, ctx->ev_split, ctx->ev_g1, ctx->ev_bias, ctx->ev_join})
        if (e) cudaEventDestroy(e);
    for (int i = 0; i < 2; ++i) {
        if (ctx->ev_copied[i]) cudaEventDestroy(ctx->ev_copied[i]);
        if (ctx->ev_gathered[i]) cudaEventDestroy(ctx->ev_gathered[i]);
    }
    delete ctx;
}

}  // extern "C"
