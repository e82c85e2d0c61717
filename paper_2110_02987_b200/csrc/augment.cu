// Importance-based subgraph augmentation (Algorithm 1 of the paper, Section 3.2.2): for every subgraph of a
// partition, Monte-Carlo random walks from its boundary nodes estimate how often each outside node is reached
// (importance equation), the number of walks follows the Monte-Carlo error equation, and the replication nodes are
// taken walk by walk in descending order of the walks' summed importance until the density-sized number n(g_i) is
// reached.  Its output (the replication-node lists) is what gad_create takes as `halo_nodes`.
//
// On the GPU: the boundary test, the walks with their visit counts, the count statistics and the walk scores, all in
// integers (the same draws, counts and scores as a CPU evaluation: every random number is a pure function
// mix(seed, subgraph, walk, step) of the splitmix64 output function).  Walks are never stored: the scoring kernel and
// the host's selection loop regenerate them from the generator.  On the host: the boundary list, the number of walks
// from the integer sums, the ranking of the walks and the selection loop, which is sequential by definition.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <functional>
#include <numeric>
#include <string>
#include <vector>

#include "gad_internal.h"

namespace gad {

namespace {

constexpr int kMaxSteps = 8;

__host__ __device__ inline uint64_t aug_mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
    return z ^ (z >> 31);
}
// key of (seed, subgraph, walk); the step is mixed in per draw
__host__ __device__ inline uint64_t walk_key(uint64_t seed, int sub, int64_t walk) {
    const uint64_t G = 0x9e3779b97f4a7c15ULL;
    const uint64_t h = aug_mix64(seed + G * (uint64_t)(1 + sub));
    return aug_mix64(h + G * (uint64_t)(1 + walk));
}
__host__ __device__ inline uint64_t walk_draw(uint64_t key, int step) {
    const uint64_t G = 0x9e3779b97f4a7c15ULL;
    return aug_mix64(key + G * (uint64_t)(1 + step));
}
// The node sequence of one walk: start at a uniformly drawn boundary node, every step to a uniformly drawn neighbour.
__host__ __device__ inline void make_walk(const int64_t* rowptr, const int32_t* col, const int32_t* B, int64_t nB, uint64_t seed, int sub,
                                          int64_t walk, int steps, int32_t* seq) {
    const uint64_t key = walk_key(seed, sub, walk);
    int32_t cur = B[walk_draw(key, 0) % (uint64_t)nB];
    seq[0] = cur;
    for (int s = 1; s <= steps; ++s) {
        const int64_t r0 = rowptr[cur], d = rowptr[cur + 1] - r0;
        if (d > 0) cur = col[r0 + (int64_t)(walk_draw(key, s) % (uint64_t)d)];
        seq[s] = cur;
    }
}
// v is outside the subgraph and does not occur earlier in the walk
__host__ __device__ inline bool first_outside(const uint8_t* inside, const int32_t* seq, int s) {
    const int32_t v = seq[s];
    if (inside[v]) return false;
    for (int t = 0; t < s; ++t)
        if (seq[t] == v) return false;
    return true;
}

// flag[t] = core node t has a neighbour outside the core set; *inner += directed entries between two different core nodes
// (2 |e_i| of the density definition; an integer sum, so the order of the additions does not matter).
__global__ void boundary_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, const int32_t* __restrict__ core,
                                int64_t ncore, const uint8_t* __restrict__ inside, uint8_t* __restrict__ flag,
                                unsigned long long* __restrict__ inner) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long mine = 0;
    if (t < ncore) {
        const int32_t v = core[t];
        uint8_t f = 0;
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            const int32_t c = col[e];
            if (!inside[c]) f = 1;
            else if (c != v) ++mine;
        }
        flag[t] = f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(inner, mine);
}
__global__ void mark_kernel(const int32_t* __restrict__ core, int64_t ncore, uint8_t* __restrict__ inside, uint8_t value) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < ncore) inside[core[t]] = value;
}
__global__ void walk_count_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, const int32_t* __restrict__ B,
                                  int64_t nB, const uint8_t* __restrict__ inside, uint64_t seed, int sub, int64_t j0, int64_t j1,
                                  int steps, int32_t* __restrict__ count) {
    const int64_t j = j0 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= j1) return;
    int32_t seq[kMaxSteps + 1];
    make_walk(rowptr, col, B, nB, seed, sub, j, steps, seq);
    for (int s = 0; s <= steps; ++s)
        if (first_outside(inside, seq, s)) atomicAdd(count + seq[s], 1);   // integer: the result does not depend on the order
}
__global__ void walk_score_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, const int32_t* __restrict__ B,
                                  int64_t nB, const uint8_t* __restrict__ inside, uint64_t seed, int sub, int64_t nwalks, int steps,
                                  const int32_t* __restrict__ count, int64_t* __restrict__ score, unsigned long long* __restrict__ key) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= nwalks) return;
    int32_t seq[kMaxSteps + 1];
    make_walk(rowptr, col, B, nB, seed, sub, j, steps, seq);
    int64_t sc = 0;
    for (int s = 0; s <= steps; ++s)
        if (first_outside(inside, seq, s)) sc += count[seq[s]];
    score[j] = sc;
    // ranking key: a better walk (higher score; equal scores: lower index) has the larger key, and no two walks share one
    if (key) key[j] = ((unsigned long long)sc << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)j);
}

// Selection of the S largest ranking keys without sorting them all: the keys are unique, so the S-th largest one is found
// digit by digit (13 bits at a time, from the top), each pass a histogram of the next digit over the keys that share the
// digits fixed so far; the host reads the 8192 counts and fixes the digit.  A last pass gathers the keys >= that one.
constexpr int kDigitBits = 13, kDigits = 1 << kDigitBits;
// sel = {digits fixed so far, their mask, rank still to find among the keys that share them}: kept on the device, so the passes
// follow each other without the host in between.
struct KeySelect { unsigned long long prefix, mask; long long remaining; };
__global__ void __launch_bounds__(256) key_hist_kernel(const unsigned long long* __restrict__ key, int64_t n, const KeySelect* __restrict__ sel,
                                                       int shift, unsigned* __restrict__ hist) {
    __shared__ unsigned h[kDigits];
    const unsigned long long prefix = sel->prefix, prefix_mask = sel->mask;
    for (int i = threadIdx.x; i < kDigits; i += blockDim.x) h[i] = 0u;
    __syncthreads();
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += (int64_t)gridDim.x * blockDim.x) {
        const unsigned long long k = key[j];
        if ((k & prefix_mask) == prefix) atomicAdd(&h[(unsigned)(k >> shift) & (kDigits - 1)], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kDigits; i += blockDim.x)
        if (h[i]) atomicAdd(hist + i, h[i]);
}
// One CTA of 1024 threads: the digit whose bin holds the key of rank `remaining` (counted from the largest digit down),
// fixed in *sel; the histogram is cleared for the next pass.
__global__ void __launch_bounds__(1024) key_digit_kernel(unsigned* __restrict__ hist, KeySelect* __restrict__ sel, int shift) {
    __shared__ long long part[1024];
    __shared__ int chosen;
    __shared__ long long chosen_rem;
    constexpr int PER = kDigits / 1024;
    const int t = threadIdx.x;                 // thread t owns the bins kDigits-1 - PER t .. kDigits - PER (t + 1), largest first
    unsigned mine[PER];
    long long s = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) { mine[i] = hist[kDigits - 1 - (PER * t + i)]; s += mine[i]; }
    part[t] = s;
    if (t == 0) { chosen = 0; chosen_rem = 1; }
    __syncthreads();
    // keys in the bins of the threads before this one (inclusive scan by doubling, then made exclusive)
    for (int o = 1; o < 1024; o <<= 1) {
        const long long add = t >= o ? part[t - o] : 0;
        __syncthreads();
        part[t] += add;
        __syncthreads();
    }
    const long long before = part[t] - s, remaining = sel->remaining;
    if (before < remaining && remaining <= before + s) {   // exactly one thread: the bins are disjoint and ordered
        long long r = remaining - before;
        int i = 0;
        for (; i < PER - 1 && (long long)mine[i] < r; ++i) r -= mine[i];
        chosen = kDigits - 1 - (PER * t + i);
        chosen_rem = r;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < PER; ++i) hist[PER * t + i] = 0u;
    if (t == 0) {
        sel->prefix |= (unsigned long long)chosen << shift;
        sel->mask |= (unsigned long long)(kDigits - 1) << shift;
        sel->remaining = chosen_rem;
    }
}
__global__ void __launch_bounds__(256) key_gather_kernel(const unsigned long long* __restrict__ key, int64_t n, const KeySelect* __restrict__ sel,
                                                         unsigned long long* __restrict__ out, unsigned long long* __restrict__ n_out, int64_t cap) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    const unsigned long long least = sel->prefix;
    const unsigned long long k = key[j];
    if (k >= least) {
        const unsigned long long at = atomicAdd(n_out, 1ull);   // the host sorts what it gets: the order here is free
        if ((int64_t)at < cap) out[at] = k;
    }
}
// m = visited candidates, S1 = sum of counts, S2 = sum of squared counts
__global__ void count_stats_kernel(const int32_t* __restrict__ count, int64_t n, unsigned long long* __restrict__ stats) {
    __shared__ unsigned long long sm[3][256];
    unsigned long long m = 0, s1 = 0, s2 = 0;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n; v += (int64_t)gridDim.x * blockDim.x) {
        const unsigned long long c = (unsigned long long)count[v];
        if (c) { ++m; s1 += c; s2 += c * c; }
    }
    sm[0][threadIdx.x] = m; sm[1][threadIdx.x] = s1; sm[2][threadIdx.x] = s2;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o)
            for (int q = 0; q < 3; ++q) sm[q][threadIdx.x] += sm[q][threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0)
        for (int q = 0; q < 3; ++q) atomicAdd(stats + q, sm[q][0]);
}

struct AugPlan {
    size_t o_rowptr, o_col, o_inside, o_core, o_flag, o_B, o_count, o_stats, o_score, o_key, o_hist, o_top, bytes;
    int64_t max_core, max_walks, max_top;   // max_top: most leading walks ever ranked on the device
};
// Leading walks whose order is established first: the selection loop rarely needs more (it then orders all of them).
inline int64_t leading_walks(int64_t nwalks, int64_t n_rep) { return std::min<int64_t>(nwalks, std::max<int64_t>(1024, 8 * n_rep)); }

size_t take(size_t& cur, size_t bytes) { size_t o = cur; cur += (size_t)round_up((int64_t)std::max<size_t>(bytes, 4), 256); return o; }

int plan_augment(const gad_csr* g, int32_t K, const int64_t* core_ptr, const int32_t* core_nodes, const gad_augment_config* cfg, AugPlan& p,
                 std::string& err) {
    if (!g || !g->rowptr || (g->nnz > 0 && !g->col) || g->n < 0 || K < 1 || !core_ptr || !cfg) { err = "bad arguments"; return GAD_ERR_ARG; }
    if (cfg->steps < 1 || cfg->steps > kMaxSteps) { err = "steps must be 1 .. 8"; return GAD_ERR_ARG; }
    if (!(cfg->alpha >= 0.0) || !(cfg->E > 0.0) || !(cfg->zc > 0.0) || cfg->cap < 1) { err = "alpha >= 0, E > 0, zc > 0, cap >= 1"; return GAD_ERR_ARG; }
    // the kernels index rowptr, col and the per-node arrays with the caller's values: check the whole CSR here, on the host
    if (g->nnz < 0 || g->rowptr[0] != 0) { err = "rowptr must start at 0 and nnz must not be negative"; return GAD_ERR_ARG; }
    for (int32_t v = 0; v < g->n; ++v)
        if (g->rowptr[v + 1] < g->rowptr[v]) { err = "rowptr decreases"; return GAD_ERR_UNSORTED; }
    if (g->rowptr[g->n] != g->nnz) { err = "rowptr[n] differs from nnz"; return GAD_ERR_ARG; }
    for (int64_t e = 0; e < g->nnz; ++e)
        if (g->col[e] < 0 || g->col[e] >= g->n) { err = "column out of range"; return GAD_ERR_RANGE; }
    p.max_core = 0; p.max_walks = 1;
    for (int32_t k = 0; k < K; ++k) {
        if (core_ptr[k + 1] < core_ptr[k]) { err = "core_ptr decreases"; return GAD_ERR_UNSORTED; }
        int64_t deg = 0;
        for (int64_t t = core_ptr[k]; t < core_ptr[k + 1]; ++t) {
            const int32_t v = core_nodes[t];
            if (v < 0 || v >= g->n) { err = "core node out of range"; return GAD_ERR_RANGE; }
            deg += g->rowptr[v + 1] - g->rowptr[v];
        }
        p.max_core = std::max(p.max_core, core_ptr[k + 1] - core_ptr[k]);
        p.max_walks = std::max(p.max_walks, deg * (int64_t)cfg->cap);   // n0 is at most the subgraph's degree sum
    }
    size_t cur = 0;
    p.o_rowptr = take(cur, 8 * (size_t)(g->n + 1)); p.o_col = take(cur, 4 * (size_t)g->nnz);
    p.o_inside = take(cur, (size_t)g->n); p.o_core = take(cur, 4 * (size_t)p.max_core); p.o_flag = take(cur, (size_t)p.max_core);
    p.o_B = take(cur, 4 * (size_t)p.max_core); p.o_count = take(cur, 4 * (size_t)g->n); p.o_stats = take(cur, 64);
    p.o_score = take(cur, 8 * (size_t)p.max_walks);
    // n(g_i) <= alpha (1 + d) |v_i| <= 2 alpha |v_i|
    p.max_top = leading_walks(p.max_walks, (int64_t)std::floor(cfg->alpha * 2.0 * (double)p.max_core));
    p.o_key = take(cur, 8 * (size_t)p.max_walks); p.o_hist = take(cur, 4 * (size_t)kDigits); p.o_top = take(cur, 8 * (size_t)p.max_top);
    p.bytes = cur;
    return GAD_OK;
}

thread_local std::string g_aug_error;
int aug_fail(int code, const std::string& msg) { g_aug_error = msg; return code; }

#define AUG_CK(call)                                                                      \
    do {                                                                                  \
        cudaError_t e_ = (call);                                                          \
        if (e_ != cudaSuccess) return aug_fail(GAD_ERR_CUDA, cudaGetErrorString(e_));     \
    } while (0)

}  // namespace

const char* augment_last_error() { return g_aug_error.c_str(); }

}  // namespace gad

using namespace gad;

extern "C" {

int gad_augment_workspace_bytes(const gad_csr* g, int32_t K, const int64_t* core_ptr, const int32_t* core_nodes,
                                const gad_augment_config* cfg, size_t* bytes) {
    if (!bytes) return GAD_ERR_ARG;
    AugPlan p;
    std::string err;
    int rc = plan_augment(g, K, core_ptr, core_nodes, cfg, p, err);
    if (rc != GAD_OK) return aug_fail(rc, err);
    *bytes = p.bytes;
    return GAD_OK;
}

int gad_augment(const gad_csr* g, int32_t K, const int64_t* core_ptr, const int32_t* core_nodes, const gad_augment_config* cfg,
                void* workspace, size_t workspace_bytes, void* stream_, int64_t* halo_ptr, int32_t* halo_nodes, int64_t halo_capacity,
                int64_t* walks_out) {
    if (!workspace || !halo_ptr || (halo_capacity > 0 && !halo_nodes) || ((uintptr_t)workspace & 255) != 0) return aug_fail(GAD_ERR_ARG, "bad arguments");
    AugPlan p;
    std::string err;
    int rc = plan_augment(g, K, core_ptr, core_nodes, cfg, p, err);
    if (rc != GAD_OK) return aug_fail(rc, err);
    if (workspace_bytes < p.bytes) return aug_fail(GAD_ERR_OOM, "workspace smaller than gad_augment_workspace_bytes");
    cudaStream_t s = (cudaStream_t)stream_;
    char* ws = (char*)workspace;
    int64_t* d_rowptr = (int64_t*)(ws + p.o_rowptr);
    int32_t* d_col = (int32_t*)(ws + p.o_col);
    uint8_t* d_inside = (uint8_t*)(ws + p.o_inside);
    int32_t* d_core = (int32_t*)(ws + p.o_core);
    uint8_t* d_flag = (uint8_t*)(ws + p.o_flag);
    int32_t* d_B = (int32_t*)(ws + p.o_B);
    int32_t* d_count = (int32_t*)(ws + p.o_count);
    unsigned long long* d_stats = (unsigned long long*)(ws + p.o_stats);
    int64_t* d_score = (int64_t*)(ws + p.o_score);
    unsigned long long* d_key = (unsigned long long*)(ws + p.o_key);
    unsigned* d_hist = (unsigned*)(ws + p.o_hist);
    unsigned long long* d_top = (unsigned long long*)(ws + p.o_top);
    const int64_t n = g->n;
    const int steps = cfg->steps;
    if (!cfg->graph_resident) {   // else: an earlier call left this very graph at the start of this workspace
        AUG_CK(cudaMemcpyAsync(d_rowptr, g->rowptr, 8 * (size_t)(n + 1), cudaMemcpyHostToDevice, s));
        if (g->nnz > 0) AUG_CK(cudaMemcpyAsync(d_col, g->col, 4 * (size_t)g->nnz, cudaMemcpyHostToDevice, s));
    }
    AUG_CK(cudaMemsetAsync(d_inside, 0, (size_t)n, s));
    std::vector<uint8_t> inside((size_t)n, 0), flag;
    std::vector<int32_t> B, seq((size_t)steps + 1);
    std::vector<int64_t> score, order;
    std::vector<unsigned long long> top;
    std::vector<uint8_t> taken((size_t)n, 0);
    auto grid = [](int64_t work) { return (unsigned)((work + 255) / 256); };
    int64_t out = 0;
    halo_ptr[0] = 0;
    for (int32_t k = 0; k < K; ++k) {
        const int32_t* core = core_nodes + core_ptr[k];
        const int64_t ncore = core_ptr[k + 1] - core_ptr[k];
        int64_t nwalks = 0;
        if (ncore > 0) {
            AUG_CK(cudaMemcpyAsync(d_core, core, 4 * (size_t)ncore, cudaMemcpyHostToDevice, s));
            mark_kernel<<<grid(ncore), 256, 0, s>>>(d_core, ncore, d_inside, 1); ++g_kernel_launches;
            AUG_CK(cudaMemsetAsync(d_stats + 3, 0, 16, s));
            boundary_kernel<<<grid(ncore), 256, 0, s>>>(d_rowptr, d_col, d_core, ncore, d_inside, d_flag, d_stats + 3); ++g_kernel_launches;
            flag.resize((size_t)ncore);
            unsigned long long inner_dev = 0;
            AUG_CK(cudaMemcpyAsync(flag.data(), d_flag, (size_t)ncore, cudaMemcpyDeviceToHost, s));
            AUG_CK(cudaMemcpyAsync(&inner_dev, d_stats + 3, 8, cudaMemcpyDeviceToHost, s));
            AUG_CK(cudaStreamSynchronize(s));
            B.clear();
            const int64_t inner_directed = (int64_t)inner_dev;
            // boundary nodes in ascending node id: sorted, or, when the core set is a fair share of the graph, read off a
            // byte map over the node ids (one pass over n bytes instead of a sort)
            if (n <= 16 * ncore) {
                for (int64_t t = 0; t < ncore; ++t) {
                    inside[(size_t)core[t]] = 1;
                    if (flag[(size_t)t]) taken[(size_t)core[t]] = 1;
                }
                for (int64_t v = 0; v < n; ++v)
                    if (taken[(size_t)v]) { B.push_back((int32_t)v); taken[(size_t)v] = 0; }
            } else {
                for (int64_t t = 0; t < ncore; ++t) {
                    inside[(size_t)core[t]] = 1;
                    if (flag[(size_t)t]) B.push_back(core[t]);
                }
                std::sort(B.begin(), B.end());
            }
            const int64_t nB = (int64_t)B.size();
            if (nB > 0) {
                int64_t n0 = 0;
                for (int32_t b : B) n0 += g->rowptr[b + 1] - g->rowptr[b];
                AUG_CK(cudaMemcpyAsync(d_B, B.data(), 4 * (size_t)nB, cudaMemcpyHostToDevice, s));
                AUG_CK(cudaMemsetAsync(d_count, 0, 4 * (size_t)n, s));
                AUG_CK(cudaMemsetAsync(d_stats, 0, 24, s));
                if (n0 > 0) {
                    walk_count_kernel<<<grid(n0), 256, 0, s>>>(d_rowptr, d_col, d_B, nB, d_inside, cfg->seed, k, 0, n0, steps, d_count);
                    ++g_kernel_launches;
                }
                count_stats_kernel<<<148 * 4, 256, 0, s>>>(d_count, n, d_stats); ++g_kernel_launches;
                unsigned long long st[3];
                AUG_CK(cudaMemcpyAsync(st, d_stats, 24, cudaMemcpyDeviceToHost, s));
                AUG_CK(cudaStreamSynchronize(s));
                // Monte-Carlo error equation with sigma / mean of the visit frequencies from the integer sums
                nwalks = n0;
                if (st[0] > 0) {
                    const double ratio = ((double)st[0] * (double)st[2]) / ((double)st[1] * (double)st[1]) - 1.0;
                    const int64_t want = ratio > 0.0 ? (int64_t)std::ceil((cfg->zc / cfg->E) * (cfg->zc / cfg->E) * ratio) : 0;
                    nwalks = std::max(n0, std::min(want, (int64_t)cfg->cap * n0));
                }
                if (nwalks > p.max_walks) return aug_fail(GAD_ERR_OOM, "more walks than planned");
                if (nwalks > n0) {
                    walk_count_kernel<<<grid(nwalks - n0), 256, 0, s>>>(d_rowptr, d_col, d_B, nB, d_inside, cfg->seed, k, n0, nwalks, steps, d_count);
                    ++g_kernel_launches;
                    AUG_CK(cudaMemsetAsync(d_stats, 0, 24, s));
                    count_stats_kernel<<<148 * 4, 256, 0, s>>>(d_count, n, d_stats); ++g_kernel_launches;
                    AUG_CK(cudaMemcpyAsync(st, d_stats, 24, cudaMemcpyDeviceToHost, s));
                }
                // a walk's score is at most (steps + 1) nwalks (a node counts once per walk): when score and walk index fit
                // 32 bits each, the walks get unique 64-bit ranking keys and the leading ones are selected on the device
                const bool keyed = nwalks > 0 && nwalks < ((int64_t)1 << 32) && (int64_t)(steps + 1) * nwalks < ((int64_t)1 << 31);
                if (nwalks > 0) {
                    walk_score_kernel<<<grid(nwalks), 256, 0, s>>>(d_rowptr, d_col, d_B, nB, d_inside, cfg->seed, k, nwalks, steps, d_count, d_score,
                                                                   keyed ? d_key : nullptr);
                    ++g_kernel_launches;
                }
                AUG_CK(cudaStreamSynchronize(s));   // st (the statistics of the final counts) has arrived
                // n(g_i) = alpha (1 + d(g_i)) |v_i|, at most the visited candidates
                int64_t n_rep = 0;
                if (ncore >= 2) {
                    const double dens = (double)inner_directed / ((double)ncore * (double)(ncore - 1));
                    n_rep = (int64_t)std::floor(cfg->alpha * (1.0 + dens) * (double)ncore);
                }
                n_rep = std::min<int64_t>(n_rep, (int64_t)st[0]);
                // walks in descending order of their summed importance (equal scores: ascending index).  Only the best
                // walks are ever looked at, so the order is established for a leading stretch first and for all
                // walks only if that stretch does not yield n(g_i) nodes.
                auto better = [&](int64_t a, int64_t b) {
                    return score[(size_t)a] != score[(size_t)b] ? score[(size_t)a] > score[(size_t)b] : a < b;
                };
                auto order_all = [&]() -> int {   // every score to the host, every walk ranked there
                    score.resize((size_t)nwalks);
                    AUG_CK(cudaMemcpyAsync(score.data(), d_score, 8 * (size_t)nwalks, cudaMemcpyDeviceToHost, s));
                    AUG_CK(cudaStreamSynchronize(s));
                    order.resize((size_t)nwalks);
                    std::iota(order.begin(), order.end(), (int64_t)0);
                    std::sort(order.begin(), order.end(), better);
                    return GAD_OK;
                };
                int64_t sorted = std::min(leading_walks(nwalks, n_rep), p.max_top);
                if (n_rep > 0 && keyed && sorted < nwalks) {
                    // the `sorted`-th largest key, digit by digit from the top; then the keys at least that large
                    int top_bit = 32;
                    while (top_bit < 63 && (((int64_t)(steps + 1) * nwalks) >> (top_bit - 32)) > 0) ++top_bit;
                    KeySelect* d_sel = reinterpret_cast<KeySelect*>(d_stats + 5);
                    const KeySelect sel0{0ull, 0ull, (long long)sorted};
                    AUG_CK(cudaMemcpyAsync(d_sel, &sel0, sizeof sel0, cudaMemcpyHostToDevice, s));
                    AUG_CK(cudaMemsetAsync(d_hist, 0, 4 * (size_t)kDigits, s));
                    for (int d = (top_bit + kDigitBits - 1) / kDigitBits - 1; d >= 0; --d) {
                        const int shift = d * kDigitBits;
                        key_hist_kernel<<<148 * 2, 256, 0, s>>>(d_key, nwalks, d_sel, shift, d_hist); ++g_kernel_launches;
                        key_digit_kernel<<<1, 1024, 0, s>>>(d_hist, d_sel, shift); ++g_kernel_launches;
                    }
                    AUG_CK(cudaMemsetAsync(d_stats + 4, 0, 8, s));
                    key_gather_kernel<<<grid(nwalks), 256, 0, s>>>(d_key, nwalks, d_sel, d_top, d_stats + 4, p.max_top); ++g_kernel_launches;
                    unsigned long long got = 0;
                    top.resize((size_t)sorted);
                    AUG_CK(cudaMemcpyAsync(&got, d_stats + 4, 8, cudaMemcpyDeviceToHost, s));
                    AUG_CK(cudaMemcpyAsync(top.data(), d_top, 8 * (size_t)sorted, cudaMemcpyDeviceToHost, s));
                    AUG_CK(cudaStreamSynchronize(s));
                    if ((int64_t)got != sorted) return aug_fail(GAD_ERR_CUDA, "selection of the leading walks came out with the wrong count");
                    std::sort(top.begin(), top.end(), std::greater<unsigned long long>());
                    order.resize((size_t)sorted);
                    for (int64_t a = 0; a < sorted; ++a) order[(size_t)a] = (int64_t)(0xFFFFFFFFu - (uint32_t)(top[(size_t)a] & 0xFFFFFFFFull));
                } else if (n_rep > 0) {
                    int rc2 = order_all();
                    if (rc2 != GAD_OK) return rc2;
                    sorted = nwalks;
                }
                const int64_t first = out;
                for (int64_t a = 0; a < nwalks && out - first < n_rep; ++a) {
                    if (a == sorted) {   // the leading stretch is used up: order all walks (the leading ones come out the same)
                        int rc2 = order_all();
                        if (rc2 != GAD_OK) return rc2;
                        sorted = nwalks;
                    }
                    make_walk(g->rowptr, g->col, B.data(), nB, cfg->seed, k, order[(size_t)a], steps, seq.data());
                    for (int t = 0; t <= steps && out - first < n_rep; ++t) {
                        const int32_t v = seq[(size_t)t];
                        if (inside[(size_t)v] || taken[(size_t)v]) continue;
                        if (out >= halo_capacity) return aug_fail(GAD_ERR_OOM, "halo_nodes too small");
                        taken[(size_t)v] = 1;
                        halo_nodes[out++] = v;
                    }
                }
                for (int64_t t = first; t < out; ++t) taken[(size_t)halo_nodes[t]] = 0;
            }
            for (int64_t t = 0; t < ncore; ++t) inside[(size_t)core[t]] = 0;
            mark_kernel<<<grid(ncore), 256, 0, s>>>(d_core, ncore, d_inside, 0); ++g_kernel_launches;
        }
        if (walks_out) walks_out[k] = nwalks;
        halo_ptr[k + 1] = out;
    }
    AUG_CK(cudaStreamSynchronize(s));
    AUG_CK(cudaGetLastError());
    return GAD_OK;
}

const char* gad_augment_last_error(void) { return augment_last_error(); }

}  // extern "C"
