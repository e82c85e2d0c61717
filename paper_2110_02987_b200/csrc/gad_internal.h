// Internal declarations shared by the translation units of the library (not part of the boundary).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cmath>
#include <string>
#include <vector>

#include "../../include/gad.h"

namespace gad {

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

// Kernels launched by this library in this process (every <<<>>> adds one; contexts on several host threads share it).
extern std::atomic<int64_t> g_kernel_launches;

// Function attributes belong to a device: asks once per (current device, kernel) for `smem_bytes` of dynamic shared
// memory and, with `max_carveout`, for the largest shared-memory share of the SM.  Safe from several host threads.
cudaError_t configure_kernel_once(const void* kernel, int smem_bytes, bool max_carveout);

// ---------------------------------------------------------------------------------------------
// Host-side result of building the block-diagonal store (create-time, not on the timed path).
// ---------------------------------------------------------------------------------------------
struct HostStore {
    int32_t K = 0;
    int64_t Np = 0, nnz = 0;
    std::vector<int64_t> rowptr;   // [Np+1]
    std::vector<int32_t> col;      // [nnz] store-row ids, ascending inside a row
    std::vector<float> val;        // [nnz] A~ entries, computed in double and rounded once
    std::vector<int32_t> sub_off;  // [K+1]
    std::vector<int32_t> gid;      // [Np]
    std::vector<int32_t> deg;      // [Np] local degree, self-loop excluded
    std::vector<int64_t> core_count;  // [K]
    bool symmetric = false;        // A~ equals its transpose entry by entry
    std::vector<int64_t> t_rowptr; // transposed store (t_col, t_val empty when symmetric or when values were not asked for)
    std::vector<int32_t> t_col;
    std::vector<float> t_val;
};

// Validates the inputs and fills the store; returns a GAD_* status and a message.
int build_store(const gad_csr* g, const gad_partition* part, bool values, HostStore& out, std::string& err);
// Sizes only (for gad_workspace_bytes): rows, entries, and the SpMM scratch slots of the worse orientation.
int store_sizes(const gad_csr* g, const gad_partition* part, int64_t* Np, int64_t* nnz, int64_t* slots, std::string& err);

// Work lists of the SpMM launch (host side).  A row of at most `part_entries` entries is one item; a longer row is
// cut into parts of `part_entries` entries, each an item with a scratch slot of its own, and gets an entry
// fin = {row, first scratch slot, slots, subgraph of the row}.  The part length starts at kMinPart, or at a quarter of the
// entries an average resident warp gets if that is more, and doubles (up to kMaxPart) until the cut rows need at most one
// scratch slot per two store rows; a row that would still need more than kMaxSlotsPerRow parts gets longer parts of its own.
// items = {row, low 32 bits of the first entry's position in the store, (high bits << 16) | entries, scratch slot
// or -1 for an uncut row}, subgraph by subgraph and inside a subgraph binned by floor(log2(entries)), longest bin
// first, ascending row inside a bin.  `perm` (uncut rows in that order) and `parts` are the intermediate lists the
// items are built from.
constexpr int64_t kMinPart = 64, kMaxPart = 8192, kMaxSlotsPerRow = 32;
struct RowWork {
    std::vector<int32_t> perm;
    std::vector<int4> parts, fin, items;
    int64_t slots = 0, part_entries = kMinPart;
};
int64_t part_entries_for(const std::vector<int64_t>& rowptr);
// forced_part > 0: cut rows into parts of that many entries instead of the length part_entries_for would choose
void bin_rows(const std::vector<int64_t>& rowptr, const std::vector<int32_t>& sub_off, RowWork& out, int64_t forced_part = 0);
// Scratch slots bin_rows would use, from the row lengths alone.
int64_t count_slots(const std::vector<int64_t>& rowptr);

// ---------------------------------------------------------------------------------------------
// Device views
// ---------------------------------------------------------------------------------------------
struct SparseDev {
    const int64_t* rowptr = nullptr;  // [Np+1] (kept for the accessors; the kernels read the work list)
    const uint2* ecv = nullptr;       // [nnz] packed (column, value bits)
    const int4* fin = nullptr;        // rows made of several parts
    const int4* items = nullptr;      // parts and uncut rows together, longest first
    float* scratch = nullptr;         // [slots x leading dimension of the output] partial rows
    int32_t nfin = 0, nitems = 0;
    int64_t nrows = 0;                // rows (and columns) of the store
};

struct Layer {
    int32_t fi, fo;        // F_l, F_{l+1}
    int32_t ldi, ldo;      // leading dimensions of H^(l), H^(l+1) (multiples of 4 floats)
    int32_t ldw;           // leading dimension of W_l rows inside the padded parameter block
    int64_t w_int, b_int;  // offsets inside one replica's padded parameter block (multiples of 4 floats)
    int64_t w_ext, b_ext;  // offsets inside the caller-visible [P] layout
};

// A run of rows that belongs to one subgraph: {first row, row count, subgraph, unused}.
struct RowSpan { int32_t row0, nrows, k, pad; };

struct Epilogue {            // of the forward SpMM: bias, ReLU, dropout
    const float* params;     // padded parameter blocks
    int64_t pstride;         // floats between replicas
    int64_t b_int;           // bias offset inside a block
    const int32_t* sub_off;  // [K+1]
    int32_t K;
    int32_t relu;            // 0 on the last layer
    float dropout;
    uint64_t seed;
    int64_t epoch;
    int32_t layer;
};

// What a finishing kernel gets: where the biases are and how ReLU / dropout apply on this layer and epoch.
struct ActEpi {
    const float* params;   // padded parameter blocks
    long long pstride;     // floats between replicas
    long long b_int;       // bias offset inside a block
    int relu;              // 0 on the last layer
    int drop;              // dropout is applied (rate > 0 on a layer with ReLU)
    uint32_t thr;          // keep an element when the top 24 bits of its hash reach this
    float scale;           // 1 / (1 - rate)
    unsigned long long seed;
    long long epoch;
    int layer;
    int col0;              // column of the operand's first column (column slabs)
};
inline ActEpi make_act(const Epilogue& e, int col0) {
    ActEpi t{};
    t.params = e.params; t.pstride = e.pstride; t.b_int = e.b_int + col0;
    t.relu = e.relu; t.layer = e.layer;
    t.drop = e.dropout > 0.f && e.relu;
    t.thr = t.drop ? (uint32_t)std::floor((double)e.dropout * 16777216.0) : 0u;
    t.scale = t.drop ? 1.f / (1.f - e.dropout) : 1.f;
    t.seed = e.seed; t.epoch = e.epoch; t.col0 = col0;
    return t;
}

// ---------------------------------------------------------------------------------------------
// Kernel launchers (each enqueues on `s` and returns the cudaGetLastError of its launches)
// ---------------------------------------------------------------------------------------------
// bf16_scratch: null, or device room for nrows x ldz bfloat16 values: the operand is then copied there in bfloat16 and
// gathered from the copy (reduced-precision mode); with bf16_ready the copy is there already (written by the producer).
cudaError_t launch_spmm(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F,
                        const Epilogue* epi, void* bf16_scratch, bool bf16_ready, cudaStream_t s);

// Tests every index of a device store and its work lists against its range (see check_store_kernel); bad[0] += violations,
// bad[1] = min(bad[1], first offending work-list position + 1).
cudaError_t launch_check_store(const SparseDev& A, long long nnz, long long slots, const int32_t* sub_off, int K, unsigned long long* bad,
                               cudaStream_t s);

// mode 0: C = A * W_k (W row-major [Kd x N], ld ldw); mode 1: C = (A * W_k^T) masked by Hmask > 0, scaled
// (W row-major [N x Kd]); mode 2: C = sigma(A * W_k + b_k) with dropout as `act` says.  Tiles never cross a subgraph.
cudaError_t launch_gemm_rows_simt(int mode, const float* A, int lda, int Kd, const float* params, int64_t pstride,
                                  int64_t w_int, int ldw, int N, float* C, int ldc, const RowSpan* tiles,
                                  int ntiles, const float* Hmask, int ldh, float scale, const ActEpi* act, cudaStream_t s);

// Tensor-core (tcgen05) version of launch_gemm_rows_simt.  The operands come through TMA descriptors made by
// tc_make_map (A: [rows x Kd]; B, B_lo: [K][N][Kd] copies written by launch_split_weights); passes = 3 gives fp32
// accuracy by operand splitting, passes = 1 plain TF32 operands.  err receives a role code if a bounded wait runs out.
int tc_bn_for(int n_cols);
int tc_tn_rows();   // rows of the row-box descriptors the weight-gradient kernel reads (mapH / mapZ of launch_gemm_tn_tc)
bool tc_make_map(void* out_map, const void* base, uint64_t inner, uint64_t rows, uint64_t outer, uint64_t row_stride_bytes,
                 uint64_t outer_stride_bytes, uint32_t box_rows, bool mn_major = false);
cudaError_t launch_split_weights(const float* params, int64_t pstride, int64_t w_int, int fi, int fo, int ldw, int ldkt, int K,
                                 float* w_hi, float* w_lo, float* wt_hi, float* wt_lo, cudaStream_t s);
// Cbf16 (mode 0 only, may be null): the result goes there as bfloat16 [rows x ldc] INSTEAD of to C - the operand copy the
// reduced-precision aggregation gathers, written by its producer.
cudaError_t launch_gemm_rows_tc(const void* mapA, const void* mapB, const void* mapBlo, int mode, int passes, int Kd, int n_cols,
                                float* C, int ldc, const RowSpan* tiles, int ntiles, const float* Hmask, int ldh, float scale,
                                const ActEpi* act, int32_t* err, int num_sms, cudaStream_t s, void* Cbf16 = nullptr);

// Tensor-core version of launch_gemm_tn_simt; mapH / mapZ are row-box descriptors (tc_tn_rows rows) of H^(l) and dZ.
cudaError_t launch_gemm_tn_tc(const void* mapH, const void* mapZ, int passes, int M, int n_cols, int ldw, const RowSpan* chunks,
                              int nchunks, float* partial, int32_t* err, cudaStream_t s);

// Backward transforms of a layer with at most 16 output columns as one stream on the FP32 ALUs (narrow.cu).  `chunks`
// are runs of rows of one subgraph, one CTA each.  In one pass over H and dZ: dPre = (dZ W_k^T) masked by H > 0, times
// `scale`, and partial[chunk] = [column sums of those dPre rows (ldh floats)] [H[chunk rows]^T dZ[chunk rows] (fi x ldw)],
// to be added per subgraph by launch_reduce_chunks (the bias of a layer lies right before the weights of the next).  H and dZ must be contiguous (leading dimension = row length).  err receives 90 if a bounded wait runs out.
bool narrow_supported(int ldi, int ldo);
cudaError_t launch_narrow_bwd(const float* H, int ldh, int fi, const float* dZ, int ldz, const float* params, int64_t pstride,
                              int64_t w_int, int ldw, const RowSpan* chunks, int nchunks, float scale, float* dPre, float* partial,
                              int64_t partial_stride, int32_t* err, cudaStream_t s);

// partial[chunk] = H[chunk rows]^T * dZ[chunk rows]   ([M x ldw] each), one CTA column per chunk.
cudaError_t launch_gemm_tn_simt(const float* H, int ldh, int M, const float* dZ, int ldz, int N,
                                const RowSpan* chunks, int nchunks, float* partial, int ldw, cudaStream_t s);

// out[k][off + i] = sum over the chunks of subgraph k, in chunk order, of partial[chunk][i], i < len.
cudaError_t launch_reduce_chunks(const float* partial, int64_t pstride_chunk, const int32_t* chunk_ptr, int K,
                                 float* out, int64_t ostride, int64_t off, int64_t len, cudaStream_t s);

// The three launchers below are single kernels whose last-arriving CTA (per subgraph, or overall for the loss)
// finishes the reduction over the chunks in chunk order; `counters` are monotonic arrival counters, zero at creation.

// out[k][off + j] = sum over the rows of subgraph k of G[row][j], j < ld  (counters: one per subgraph).
cudaError_t launch_colsum_chunks(const float* G, int ld, const RowSpan* chunks, int nchunks, float* partial,
                                 int64_t pstride_chunk, const int32_t* chunk_ptr, unsigned* counters, float* out,
                                 int64_t ostride, int64_t off, cudaStream_t s);

// dlogits, and loss[0..K-1] = mean loss of each subgraph, loss[K] = mean over all training rows  (counter: one).
cudaError_t launch_softmax_xent(const float* logits, int ld, int C, const int32_t* label, const uint8_t* train,
                                const RowSpan* chunks, int nchunks, const float* inv_ntrain, float* dlogits,
                                float* loss_partial, const int32_t* chunk_ptr, int K, float inv_total, float* loss,
                                int32_t* nonfinite, unsigned* counter, cudaStream_t s);

// zeta[k] of every subgraph that has rows  (counters: one per subgraph).  phase 0: from the matrix X alone; phases 1, 2, 3:
// X is the first, a further, the last of several matrices whose squared distances add up (q_acc: one double per subgraph).
cudaError_t launch_zeta(const float* X, int ld, int F, const int32_t* deg, const RowSpan* chunks, int nchunks,
                        const int32_t* chunk_ptr, const int32_t* sub_off, const int64_t* deg_sum, const int64_t* deg_sq,
                        float beta, double* partial, unsigned* counters, double* zeta, double* q_acc, int phase, cudaStream_t s);

// zeta_k in the literal pairwise form, sum_{i<j} p_i p_j / (|x_i - x_j| + beta), 64 x 64 tiles of pairs (one CTA each,
// pair_ptr[k] = first tile of subgraph k); counters: one per subgraph; partial: one double per tile.
constexpr int64_t kZetaPairMaxRows = 32768;
int64_t zeta_pair_tiles(int64_t rows);
cudaError_t launch_zeta_pair(const float* X, int ld, int F, const int32_t* deg, const int32_t* sub_off, const int64_t* deg_sum,
                             const int64_t* pair_ptr, int64_t npairs, int K, float beta, double* partial, unsigned* counters,
                             double* zeta, cudaStream_t s);

// `err_word` (may be null): when a kernel of the epoch has reported a bounded wait that ran out, the gradients are not to
// be trusted and the three consensus kernels leave the parameters (and `out`) untouched.
// The same zeta_k with the squared distances from a Gram matrix on the tensor cores (zeta_gram.cu): tiles of 128 x 128 pairs,
// tile_ptr[k] = first tile of subgraph k, any subgraph size.  Xhi, Xlo: [rows x ld] floats each (TF32 split of X, written
// by the call; mapHi / mapLo are their 128-row-box descriptors); norm2: [rows] floats; partial: zeta_gram_partials doubles.
constexpr int kGramMaxCtas = 256;
int64_t zeta_gram_tiles(int64_t rows);
int64_t zeta_gram_partials(int num_ctas, int K);
cudaError_t launch_zeta_gram(const void* mapHi, const void* mapLo, const float* X, int ld, int F, long long rows, const int32_t* deg,
                             const int32_t* sub_off, const int64_t* deg_sum, const int64_t* tile_ptr, int64_t ntiles, int K, float beta,
                             float* Xhi, float* Xlo, float* norm2, double* partial, double* zeta, int32_t* err, int num_sms, cudaStream_t s);

cudaError_t launch_sgd_consensus(float* params, const float* grads, int64_t pstride, int64_t len, int K, float lr,
                                 const double* zeta, int weighted, int with_sgd, const int32_t* err_word, cudaStream_t s);
// One context's share of a consensus over several contexts: out = sum_k w_k (theta_k - lr grad_k) with w_k = zeta_k / total
// (or 1 / total), the parameters unchanged; and the finished sum written to every replica.
cudaError_t launch_consensus_partial(const float* params, const float* grads, int64_t pstride, int64_t len, int K, float lr,
                                     const double* zeta, int weighted, int with_sgd, double total, float* out, const int32_t* err_word, cudaStream_t s);
cudaError_t launch_consensus_apply(float* params, int64_t pstride, int64_t len, int K, const float* in, const int32_t* err_word, cudaStream_t s);

// One CTA waits, with the transforms' bounded wait and a limit of `polls` polls, on a barrier that nothing arrives at, and
// reports it in `err` like a transform would (role 99).  For testing the time-out path; returns at once.
cudaError_t launch_expire_wait(int32_t* err, uint32_t polls, cudaStream_t s);
cudaError_t launch_weights(const double* zeta, int K, int weighted, float* zeta_f, float* w_f, cudaStream_t s);

// G[r][c] = H[r][c] > 0 ? G[r][c] * scale : 0 over rows x ld values (the ReLU and dropout scale of the layer below, applied
// to an input gradient that was aggregated after its transform).
cudaError_t launch_relu_mask(float* G, const float* H, int ld, int64_t rows, float scale, cudaStream_t s);

cudaError_t launch_gather_rows(const float* Xg, int F, const int32_t* gid, int64_t Np, float* H0, int ld,
                               cudaStream_t s);
cudaError_t launch_gather_labels(const int32_t* yg, const int32_t* gid, int64_t Np, int32_t* label, cudaStream_t s);
cudaError_t launch_scatter_core(const float* logits, int ld, int C, const int32_t* gid, const RowSpan* core_spans,
                                int nspans, float* out, cudaStream_t s);

}  // namespace gad
