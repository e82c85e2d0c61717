// SpMM over the block-diagonal store: out = A~ * Z (+ bias, ReLU, dropout on the forward pass), i.e. the
// aggregation half of the layer H^(l+1) = sigma(A~ (H^(l) W^(l)) + b) (Section 3.3, forward equation); run on
// the transposed store it is the backward aggregation dZ = A~^T dPre.
//
// Work list: every row, or every part of a row too long for one item, is an item {row, position of its first
// entry, entries, scratch slot}; items are grouped by subgraph and sorted longest first inside one.  Operands wider
// than 64 columns take a warp per item, narrower ones a group of 4, 8 or 16 lanes per item; every lane owns 16
// bytes of each operand row it gathers.  The parts of a cut row go to scratch slots and a second kernel adds them
// in part order, so results never depend on scheduling.
#include "epilogue.cuh"
#include "gad_internal.h"

namespace gad {

__device__ __forceinline__ int find_sub(const int32_t* __restrict__ sub_off, int K, int row) {
    int lo = 0, hi = K;  // largest k with sub_off[k] <= row (empty subgraphs are skipped by the <=)
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (sub_off[mid] <= row) lo = mid; else hi = mid;
    }
    return lo;
}

// Four consecutive operand values at p: fp32 (16 bytes), or with BF bfloat16 (8 bytes, value i in bits 16 i .. 16 i + 15),
// widened to fp32.  The bfloat16 copy of the operand is what the reduced-precision mode gathers: half the bytes per entry.
template <bool BF>
__device__ __forceinline__ float4 load_row4(const char* p) {
    if constexpr (BF) {
        const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
        return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                           __uint_as_float(u.y & 0xffff0000u));
    } else {
        return __ldg(reinterpret_cast<const float4*>(p));
    }
}
template <bool BF> struct OpBytes { static constexpr uint32_t elem = BF ? 2u : 4u, quad = BF ? 8u : 16u; };

struct EpiDev {
    ActEpi act;
    const int32_t* sub_off;
    int K;
};

// Which four columns (in units of four) accumulator j of lane gl holds: gl + group * j, or with PAIR (a lane owns eight
// consecutive columns per 16-byte bfloat16 load) the halves of the eight columns 2 (gl + group * (j / 2)).
template <bool PAIR>
__device__ __forceinline__ int col4_of(int gl, int group, int j) {
    if constexpr (PAIR) return 2 * (gl + group * (j >> 1)) + (j & 1);
    else return gl + group * j;
}

template <int NV, bool EPI, bool PAIR = false>
__device__ __forceinline__ void finish_row(float4 (&acc)[NV], int row, int gl, int group, int F4, float* __restrict__ out,
                                           int ldo, const EpiDev& ep, int known_k = -1) {
    if (EPI) {
        const int k = known_k >= 0 ? known_k : find_sub(ep.sub_off, ep.K, row);   // the list of cut rows carries the subgraph
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int v = col4_of<PAIR>(gl, group, j);
            if (v < F4) acc[j] = apply_act(acc[j], ep.act, k, row, 4 * v);
        }
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        int v = col4_of<PAIR>(gl, group, j);
        if (v < F4) reinterpret_cast<float4*>(out + (long long)row * ldo)[v] = acc[j];
    }
}

// Decoded item of the unified list.
struct Item {
    int row, len, slot;
    const uint2* ent;
};
__device__ __forceinline__ Item load_item(const int4* __restrict__ items, int idx, const uint2* __restrict__ ecv) {
    const int4 it = __ldg(items + idx);   // {row, entry position low, (position high << 16) | entries, scratch slot or -1}
    Item r;
    r.row = it.x; r.len = (int)((uint32_t)it.z & 0xFFFFu); r.slot = it.w;
    r.ent = ecv + (((long long)((uint32_t)it.z >> 16) << 32) | (long long)(uint32_t)it.y);
    return r;
}

// ---- operands of at most 64 columns: GROUP lanes per item, 32 / GROUP items per warp ----
//
// A group fetches a batch of entries at a time (the next batch is requested before this one is used), hands them
// round with shuffles and has all their operand rows in flight before the multiply-adds; a slot past the end of the
// item re-reads the item's own operand row with weight 0.  A last batch at most half full takes a half batch.
constexpr int kNarrowBatch = 8;      // entries a lane group has in flight
constexpr int kNarrowMinBlocks = 3;  // resident CTAs of 256 threads asked of the compiler
template <int GROUP> struct NarrowCfg { static constexpr int EPL = kNarrowBatch / GROUP > 0 ? kNarrowBatch / GROUP : 1; };

template <int GROUP, int NB, bool BF>
__device__ __forceinline__ void narrow_batch(float4& acc, const uint2 (&mine)[NarrowCfg<GROUP>::EPL], unsigned gmask,
                                             const char* zl, uint32_t ldzb) {
    float4 z[NB];
    float a[NB];
#pragma unroll
    for (int t = 0; t < NB; ++t) {
        const uint32_t c = __shfl_sync(gmask, mine[t / GROUP].x, t % GROUP, GROUP);
        a[t] = __uint_as_float(__shfl_sync(gmask, mine[t / GROUP].y, t % GROUP, GROUP));
        z[t] = load_row4<BF>(zl + (unsigned long long)c * ldzb);
    }
#pragma unroll
    for (int t = 0; t < NB; ++t) {
        acc.x = fmaf(a[t], z[t].x, acc.x);
        acc.y = fmaf(a[t], z[t].y, acc.y);
        acc.z = fmaf(a[t], z[t].z, acc.z);
        acc.w = fmaf(a[t], z[t].w, acc.w);
    }
}

template <int GROUP, bool EPI, bool BF>
__global__ void __launch_bounds__(256, kNarrowMinBlocks)
spmm_items_narrow_kernel(const uint2* __restrict__ ecv, const int4* __restrict__ items, int nitems, const float* __restrict__ Z, int ldz,
                         float* __restrict__ out, int ldo, float* __restrict__ scratch, int F4, EpiDev ep) {
    constexpr int NB = kNarrowBatch, EPL = NarrowCfg<GROUP>::EPL;   // entries per batch, entries a lane fetches per batch
    const int lane = threadIdx.x & 31, gl = lane & (GROUP - 1);
    const unsigned gmask = (GROUP == 32 ? 0xffffffffu : ((1u << GROUP) - 1u)) << (lane & ~(GROUP - 1));
    const long long idx = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / GROUP;
    if (idx >= nitems) return;   // the whole group leaves together
    const Item it = load_item(items, (int)idx, ecv);
    const uint2 pad = make_uint2((uint32_t)it.row, 0u);
    const char* zl = reinterpret_cast<const char*>(Z) + (long long)OpBytes<BF>::quad * min(gl, F4 - 1);   // lanes past the last column read it again
    const uint32_t ldzb = OpBytes<BF>::elem * (uint32_t)ldz;
    float4 acc[1] = {make_float4(0.f, 0.f, 0.f, 0.f)};
    uint2 next[EPL];
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
        const int e = gl + GROUP * i;
        next[i] = (e < NB && e < it.len) ? __ldg(it.ent + e) : pad;
    }
    for (int b = 0; b < it.len; b += NB) {
        uint2 mine[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) {
            mine[i] = next[i];
            const int e = gl + GROUP * i;
            next[i] = (e < NB && b + NB + e < it.len) ? __ldg(it.ent + b + NB + e) : pad;
        }
        if (it.len - b > NB / 2) narrow_batch<GROUP, NB, BF>(acc[0], mine, gmask, zl, ldzb);
        else narrow_batch<GROUP, NB / 2, BF>(acc[0], mine, gmask, zl, ldzb);
    }
    if (it.slot >= 0) {
        if (gl < F4) reinterpret_cast<float4*>(scratch + (long long)it.slot * ldo)[gl] = acc[0];
    } else {
        finish_row<1, EPI>(acc, it.row, gl, GROUP, F4, out, ldo, ep);
    }
}

// Rows made of several parts: their scratch slots added in part order, then the epilogue.  One warp per row.
template <int NV, int GROUP, bool EPI>
__global__ void __launch_bounds__(256) spmm_finish_kernel(const int4* __restrict__ fin, int nfin, const float* __restrict__ scratch,
                                                          float* __restrict__ out, int ldo, int F4, EpiDev ep) {
    const int lane = threadIdx.x & 31;
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= nfin || lane >= GROUP) return;
    const int4 f = fin[i];  // {row, first slot, slots, subgraph of the row}
    float4 acc[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    // several slots are loaded together and added in slot order (a slot past the last one counts as zero)
    constexpr int Q = NV == 1 ? 16 : (NV == 2 ? 8 : (NV <= 4 ? 4 : 2));
    for (int p = 0; p < f.z; p += Q) {
        float4 t[Q][NV];
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const float4* src = reinterpret_cast<const float4*>(scratch + (long long)(f.y + p + q) * ldo);
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                const int v = lane + GROUP * j;
                t[q][j] = (p + q < f.z && v < F4) ? src[v] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int q = 0; q < Q; ++q)
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                acc[j].x += t[q][j].x; acc[j].y += t[q][j].y; acc[j].z += t[q][j].z; acc[j].w += t[q][j].w;
            }
    }
    finish_row<NV, EPI>(acc, f.x, lane, GROUP, F4, out, ldo, ep, f.w);
}

// ---- operands wider than 64 columns: one warp per item of the unified list (a whole row or a part of a cut row) ----
//
// The warp stages 32 packed entries in shared memory (slots past the end of the item hold the item's own row with
// weight 0, so every later read is unconditional), then every lane reads them back two at a time with one
// 16-byte shared load, turns each column into an address with one multiply-add, and keeps UU operand rows
// (16 bytes per lane each) in flight before the multiply-adds.  The last entries of a batch go through the
// next smaller power of two, so a batch costs at most one round trip more than its full groups.
// Where a lane finds its 16 bytes of operand row c: operand start + c * (row stride in bytes) + the lane's column
// offset.  With OFF32 the whole operand is smaller than 4 GiB and the offset is formed in 32 bits by one multiply-add.
template <int NV, bool OFF32, bool BF, bool PAIR = false>
struct ZLane {
    const char* base;      // OFF32: start of the operand (the same for the whole warp)
    const char* ptr[NV];   // otherwise: start of the operand plus the lane's column offset
    uint32_t off[NV];
    uint32_t ldzb;
    __device__ __forceinline__ float4 load(uint32_t c, int j) const {
        if constexpr (OFF32) return load_row4<BF>(base + (c * ldzb + off[j]));
        else return load_row4<BF>(ptr[j] + (unsigned long long)c * ldzb);
    }
    // PAIR: eight bfloat16 values (16 bytes) of operand row c at this lane's j-th position, widened to two float4
    __device__ __forceinline__ void load_pair(uint32_t c, int j, float4& lo, float4& hi) const {
        const char* p;
        if constexpr (OFF32) p = base + (c * ldzb + off[j]);
        else p = ptr[j] + (unsigned long long)c * ldzb;
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
        lo = make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                         __uint_as_float(u.y & 0xffff0000u));
        hi = make_float4(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u), __uint_as_float(u.w << 16),
                         __uint_as_float(u.w & 0xffff0000u));
    }
};

template <int NV, int UU, bool OFF32, bool BF, bool PAIR>
__device__ __forceinline__ void gather_fma(float4 (&acc)[NV], const uint2* st, const ZLane<NV, OFF32, BF, PAIR>& zl) {
    uint32_t c[UU];
    float a[UU];
    if constexpr (UU == 1) {
        const uint2 v = st[0];
        c[0] = v.x; a[0] = __uint_as_float(v.y);
    } else {
#pragma unroll
        for (int p = 0; p < UU / 2; ++p) {
            const uint4 v = reinterpret_cast<const uint4*>(st)[p];
            c[2 * p] = v.x; a[2 * p] = __uint_as_float(v.y);
            c[2 * p + 1] = v.z; a[2 * p + 1] = __uint_as_float(v.w);
        }
    }
    float4 z[UU][NV];
    if constexpr (PAIR) {
#pragma unroll
        for (int u = 0; u < UU; ++u)
#pragma unroll
            for (int j = 0; j < NV / 2; ++j) zl.load_pair(c[u], j, z[u][2 * j], z[u][2 * j + 1]);
    } else {
#pragma unroll
        for (int u = 0; u < UU; ++u)
#pragma unroll
            for (int j = 0; j < NV; ++j) z[u][j] = zl.load(c[u], j);
    }
#pragma unroll
    for (int u = 0; u < UU; ++u)
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            acc[j].x = fmaf(a[u], z[u][j].x, acc[j].x);
            acc[j].y = fmaf(a[u], z[u][j].y, acc[j].y);
            acc[j].z = fmaf(a[u], z[u][j].z, acc[j].z);
            acc[j].w = fmaf(a[u], z[u][j].w, acc[j].w);
        }
}

template <int NV, int V, bool OFF32, bool BF, bool PAIR>
__device__ __forceinline__ void gather_tail(float4 (&acc)[NV], const uint2* st, int r, const ZLane<NV, OFF32, BF, PAIR>& zl) {
    if constexpr (V >= 1) {
        if (r > V / 2) gather_fma<NV, V, OFF32, BF, PAIR>(acc, st, zl);
        else gather_tail<NV, V / 2, OFF32, BF, PAIR>(acc, st, r, zl);
    }
}

// Operand rows in flight per lane and resident warps asked of the compiler: short items make the chain
// item -> entries -> operand rows the cost, and more resident warps hide it better than more loads per warp.
constexpr int kItemWarps = 4;
template <int NV> struct ItemCfg {
    static constexpr int UU = NV <= 4 ? 2 : 1;
    static constexpr int MINB = NV == 1 ? 16 : (NV == 2 ? 10 : (NV <= 4 ? 6 : 4));   // CTAs of 4 warps per SM
};

template <int NV, bool EPI, bool OFF32, bool BF, bool PAIR>
__global__ void __launch_bounds__(32 * kItemWarps, ItemCfg<NV>::MINB)
spmm_items_kernel(const uint2* __restrict__ ecv, const int4* __restrict__ items, int nitems, const float* __restrict__ Z,
                  int ldz, float* __restrict__ out, int ldo, float* __restrict__ scratch, int F4, EpiDev ep) {
    constexpr int UU = PAIR ? 2 * ItemCfg<NV>::UU : ItemCfg<NV>::UU;   // half the bytes per operand row: twice the rows in flight
    __shared__ __align__(16) uint2 stage_all[kItemWarps][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int idx = blockIdx.x * kItemWarps + warp;
    if (idx >= nitems) return;
    uint2* stage = stage_all[warp];
    const Item item = load_item(items, idx, ecv);
    const int row = item.row, len = item.len;
    const uint2* ent = item.ent;
    const uint2 pad = make_uint2((uint32_t)row, 0u);
    // lanes past the last column read the last one (their sums are never stored)
    ZLane<NV, OFF32, BF, PAIR> zl;
    zl.base = reinterpret_cast<const char*>(Z);
    zl.ldzb = OpBytes<BF>::elem * (uint32_t)ldz;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        // PAIR (F4 even): position j < NV / 2 is the lane's j-th run of eight bfloat16 columns (16 bytes)
        zl.off[j] = PAIR ? 16u * (uint32_t)min(lane + 32 * j, F4 / 2 - 1) : OpBytes<BF>::quad * (uint32_t)min(lane + 32 * j, F4 - 1);
        zl.ptr[j] = zl.base + zl.off[j];
    }
    float4 acc[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);

    uint2 next = lane < len ? __ldg(ent + lane) : pad;
    for (int b = 0; b < len; b += 32) {
        const uint2 mine = next;
        const int cnt = min(32, len - b);
        next = b + 32 + lane < len ? __ldg(ent + b + 32 + lane) : pad;
        __syncwarp();   // the previous batch has been read by every lane
        stage[lane] = mine;
        __syncwarp();
        int t = 0;
        for (; t + UU / 2 < cnt; t += UU) gather_fma<NV, UU, OFF32, BF, PAIR>(acc, stage + t, zl);
        gather_tail<NV, UU / 2, OFF32, BF, PAIR>(acc, stage + t, cnt - t, zl);
    }
    if (item.slot >= 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int v = col4_of<PAIR>(lane, 32, j);
            if (v < F4) reinterpret_cast<float4*>(scratch + (long long)item.slot * ldo)[v] = acc[j];
        }
    } else {
        finish_row<NV, EPI, PAIR>(acc, row, lane, 32, F4, out, ldo, ep);
    }
}

template <int NV, int GROUP, bool EPI, bool BF>
static cudaError_t launch_rows(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F4, const EpiDev& ep,
                               cudaStream_t s) {
    if constexpr (GROUP == 32) {
        if (A.nitems > 0) {
            const unsigned grid = (unsigned)((A.nitems + kItemWarps - 1) / kItemWarps);
            // every byte of the operand within 4 GiB of its start: 32-bit offsets
            const bool off32 = (unsigned long long)A.nrows * (unsigned long long)OpBytes<BF>::elem * (unsigned long long)ldz < (1ull << 32);
            bool paired = false;
            if constexpr (BF && NV % 2 == 0) {
                // a bfloat16 operand of a whole number of 8-column runs: 16-byte loads, eight columns per lane and load
                if (F4 % 2 == 0 && ldz % 8 == 0) {
                    paired = true;
                    if (off32) spmm_items_kernel<NV, EPI, true, true, true><<<grid, 32 * kItemWarps, 0, s>>>(A.ecv, A.items, A.nitems, Z, ldz, out, ldo, A.scratch, F4, ep);
                    else spmm_items_kernel<NV, EPI, false, true, true><<<grid, 32 * kItemWarps, 0, s>>>(A.ecv, A.items, A.nitems, Z, ldz, out, ldo, A.scratch, F4, ep);
                }
            }
            if (!paired) {
                if (off32) spmm_items_kernel<NV, EPI, true, BF, false><<<grid, 32 * kItemWarps, 0, s>>>(A.ecv, A.items, A.nitems, Z, ldz, out, ldo, A.scratch, F4, ep);
                else spmm_items_kernel<NV, EPI, false, BF, false><<<grid, 32 * kItemWarps, 0, s>>>(A.ecv, A.items, A.nitems, Z, ldz, out, ldo, A.scratch, F4, ep);
            }
            ++g_kernel_launches;
        }
        if (A.nfin > 0) {
            spmm_finish_kernel<NV, GROUP, EPI><<<(unsigned)((A.nfin + 7) / 8), 256, 0, s>>>(A.fin, A.nfin, A.scratch, out, ldo, F4, ep);
            ++g_kernel_launches;
        }
        return cudaGetLastError();
    }
    if (A.nitems > 0) {
        const unsigned grid = (unsigned)(((long long)A.nitems * GROUP + 255) / 256);
        spmm_items_narrow_kernel<GROUP, EPI, BF><<<grid, 256, 0, s>>>(A.ecv, A.items, A.nitems, Z, ldz, out, ldo, A.scratch, F4, ep);
        ++g_kernel_launches;
    }
    if (A.nfin > 0) {
        spmm_finish_kernel<NV, GROUP, EPI><<<(unsigned)((A.nfin + 7) / 8), 256, 0, s>>>(A.fin, A.nfin, A.scratch, out, ldo, F4, ep);
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}

template <bool EPI, bool BF>
static cudaError_t dispatch(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F4, const EpiDev& ep,
                            cudaStream_t s) {
    cudaError_t e;
#define GAD_ROWS(NV, G) { e = launch_rows<NV, G, EPI, BF>(A, Z, ldz, out, ldo, F4, ep, s); if (e != cudaSuccess) return e; }
    if (F4 <= 4) GAD_ROWS(1, 4) else if (F4 <= 8) GAD_ROWS(1, 8) else if (F4 <= 16) GAD_ROWS(1, 16)
    else if (F4 <= 32) GAD_ROWS(1, 32) else if (F4 <= 64) GAD_ROWS(2, 32) else if (F4 <= 96) GAD_ROWS(3, 32)
    else if (F4 <= 128) GAD_ROWS(4, 32) else if (F4 <= 160) GAD_ROWS(5, 32) else if (F4 <= 192) GAD_ROWS(6, 32)
    else GAD_ROWS(8, 32)
#undef GAD_ROWS
    return cudaSuccess;
}

// Self-check of a device store before any kernel trusts it: every index the aggregation kernels will form is tested
// against its range - an item's row, its entry range inside the store, its scratch slot, every column inside the row's own
// subgraph (the store is block-diagonal), and the slot runs of the cut rows.  bad[0] counts violations, bad[1] keeps the
// smallest offending item / cut-row index + 1.  Stands in for a memory checker on the store and its work lists.
__global__ void __launch_bounds__(256) check_store_kernel(const uint2* __restrict__ ecv, long long nnz, const int4* __restrict__ items, int nitems,
                                                          const int4* __restrict__ fin, int nfin, long long slots, long long nrows,
                                                          const int32_t* __restrict__ sub_off, int K, unsigned long long* __restrict__ bad) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long mine = 0;
    if (t < nitems) {
        const int4 it = items[t];
        const long long pos = ((long long)((uint32_t)it.z >> 16) << 32) | (long long)(uint32_t)it.y;
        const int len = (int)((uint32_t)it.z & 0xFFFFu);
        const bool head_ok = it.x >= 0 && it.x < nrows && pos >= 0 && pos + len <= nnz && (it.w == -1 || (it.w >= 0 && it.w < slots));
        if (!head_ok) ++mine;
        else {
            const int k = find_sub(sub_off, K, it.x);
            for (int e = 0; e < len; ++e) {
                const uint32_t c = ecv[pos + e].x;
                if ((long long)c < sub_off[k] || (long long)c >= sub_off[k + 1]) ++mine;
            }
        }
    } else if (t < (long long)nitems + nfin) {
        const int4 f = fin[t - nitems];
        if (!(f.x >= 0 && f.x < nrows && f.y >= 0 && f.z >= 1 && (long long)f.y + f.z <= slots && f.w >= 0 && f.w < K &&
              f.x >= sub_off[f.w] && f.x < sub_off[f.w + 1]))
            ++mine;
    }
    if (mine) {
        atomicAdd(bad, mine);
        atomicMin(bad + 1, (unsigned long long)t + 1ull);
    }
}

cudaError_t launch_check_store(const SparseDev& A, long long nnz, long long slots, const int32_t* sub_off, int K, unsigned long long* bad,
                               cudaStream_t s) {
    const long long work = (long long)A.nitems + A.nfin;
    if (work > 0) {
        check_store_kernel<<<(unsigned)((work + 255) / 256), 256, 0, s>>>(A.ecv, nnz, A.items, A.nitems, A.fin, A.nfin, slots, A.nrows, sub_off, K, bad);
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}

// fp32 -> bfloat16 (round to nearest even; NaN stays NaN), four values per thread.
__global__ void __launch_bounds__(256) to_bf16_kernel(const float4* __restrict__ in, uint2* __restrict__ out, long long n4) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    out[i] = bf16_pack4(in[i]);
}

// F up to 1024 columns per pass (8 float4 per lane); wider operands are processed in column slabs.
// With `bf16_scratch` (room for nrows x ldz bfloat16) the operand is first copied there in bfloat16 and gathered from
// that copy: the reduced-precision mode, in which the gather moves half the bytes.  `bf16_ready`: the producing kernel has
// written that copy already (and Z itself is not read).
cudaError_t launch_spmm(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F, const Epilogue* epi,
                        void* bf16_scratch, bool bf16_ready, cudaStream_t s) {
    const int F4_all = (int)(round_up(F, 4) / 4);
    if (bf16_scratch && !bf16_ready && A.nrows > 0) {
        const long long n4 = (long long)A.nrows * (ldz / 4);
        to_bf16_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, s>>>(reinterpret_cast<const float4*>(Z), reinterpret_cast<uint2*>(bf16_scratch), n4);
        ++g_kernel_launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    for (int c0 = 0; c0 < F4_all; c0 += 256) {
        const int F4 = min(256, F4_all - c0);
        EpiDev ep{};
        if (epi) {
            ep.act = make_act(*epi, 4 * c0);
            ep.sub_off = epi->sub_off; ep.K = epi->K;
        }
        cudaError_t e;
        if (bf16_scratch) {
            // the kernels take the operand as a float pointer and read it through byte offsets: 4 c0 bfloat16 = 2 c0 floats
            const float* Zb = reinterpret_cast<const float*>(bf16_scratch) + 2 * c0;
            e = epi ? dispatch<true, true>(A, Zb, ldz, out + 4 * c0, ldo, F4, ep, s) : dispatch<false, true>(A, Zb, ldz, out + 4 * c0, ldo, F4, ep, s);
        } else {
            e = epi ? dispatch<true, false>(A, Z + 4 * c0, ldz, out + 4 * c0, ldo, F4, ep, s)
                    : dispatch<false, false>(A, Z + 4 * c0, ldz, out + 4 * c0, ldo, F4, ep, s);
        }
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace gad
