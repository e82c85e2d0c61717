// SpMM over the block-diagonal store: out = A~ * Z (+ bias, ReLU, dropout on the forward pass), i.e. the
// aggregation half of the layer H^(l+1) = sigma(A~ (H^(l) W^(l)) + b) (Section 3.3, forward equation); run on
// the transposed store it is the backward aggregation dZ = A~^T dPre.
//
// Work split: a warp owns one row and walks its entries; GROUP lanes (4..32) span the feature columns with NV
// float4 accumulators each (16-byte loads of the dense operand), and when GROUP < 32 the warp's 32/GROUP
// sub-groups take different entries of the row at the same time.  Entries are fetched 32 at a time as packed
// (column, value) pairs and handed round with shuffles.  Rows come from a list binned by length (heaviest
// first); long rows are cut into parts with a warp per part and a fixed-order sum of the parts through a scratch
// buffer, so results never depend on scheduling.
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

struct EpiDev {
    ActEpi act;
    const int32_t* sub_off;
    int K;
};

template <int NV, bool EPI>
__device__ __forceinline__ void finish_row(float4 (&acc)[NV], int row, int gl, int group, int F4, float* __restrict__ out,
                                           int ldo, const EpiDev& ep) {
    if (EPI) {
        const int k = find_sub(ep.sub_off, ep.K, row);
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int v = gl + group * j;
            if (v < F4) acc[j] = apply_act(acc[j], ep.act, k, row, 4 * v);
        }
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        int v = gl + group * j;
        if (v < F4) reinterpret_cast<float4*>(out + (long long)row * ldo)[v] = acc[j];
    }
}

// Entries [e0, e1) of one row accumulated by a whole warp.  The warp fetches 32 packed entries at a time (the
// next batch is requested before the current one is consumed); with GROUP < 32 the 32/GROUP sub-groups take
// different entries of the batch, each lane loading its own 16 bytes of the operand row, and the sub-group
// sums are combined afterwards with a fixed butterfly.
template <int NV, int GROUP>
__device__ __forceinline__ void walk_entries(float4 (&acc)[NV], const uint2* __restrict__ ecv, long long e0, long long e1,
                                             const float* __restrict__ Z, int ldz, int lane, int F4) {
    constexpr int SG = 32 / GROUP;
    const int gl = lane & (GROUP - 1), sg = lane / GROUP;
    uint2 next = make_uint2(0u, 0u);
    if (e0 + lane < e1) next = __ldg(ecv + e0 + lane);
    for (long long e = e0; e < e1; e += 32) {
        const uint2 mine = next;
        if (e + 32 + lane < e1) next = __ldg(ecv + e + 32 + lane);
        const int cnt = (int)min(32ll, e1 - e);
        // U entries per sub-group are in flight together; a slot past the end of the batch re-reads the batch's
        // first operand row with weight 0, so the loads stay unconditional and can all be issued at once
        constexpr int U = NV <= 2 ? 4 : (NV <= 4 ? 2 : 1);
        const int c_first = __shfl_sync(0xffffffffu, (int)mine.x, 0);
        for (int t = 0; t < cnt; t += U * SG) {
            int c[U];
            float a[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int src = t + u * SG + sg;   // entry of the batch this sub-group takes
                c[u] = __shfl_sync(0xffffffffu, (int)mine.x, src & 31);
                a[u] = __uint_as_float(__shfl_sync(0xffffffffu, mine.y, src & 31));
                if (src >= cnt) { a[u] = 0.f; c[u] = c_first; }
            }
            float4 z[U][NV];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float4* zr = reinterpret_cast<const float4*>(Z + (long long)c[u] * ldz);
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const int v = gl + GROUP * j;
                    z[u][j] = v < F4 ? __ldg(zr + v) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    acc[j].x = fmaf(a[u], z[u][j].x, acc[j].x);
                    acc[j].y = fmaf(a[u], z[u][j].y, acc[j].y);
                    acc[j].z = fmaf(a[u], z[u][j].z, acc[j].z);
                    acc[j].w = fmaf(a[u], z[u][j].w, acc[j].w);
                }
        }
    }
    if (SG > 1) {
#pragma unroll
        for (int j = 0; j < NV; ++j)
#pragma unroll
            for (int o = GROUP; o < 32; o <<= 1) {
                acc[j].x += __shfl_xor_sync(0xffffffffu, acc[j].x, o);
                acc[j].y += __shfl_xor_sync(0xffffffffu, acc[j].y, o);
                acc[j].z += __shfl_xor_sync(0xffffffffu, acc[j].z, o);
                acc[j].w += __shfl_xor_sync(0xffffffffu, acc[j].w, o);
            }
    }
}

// Narrow operands (at most 16 float4 per row): GROUP lanes per short row, 32/GROUP rows per warp.  A group fetches
// GROUP entries at a time and has all of their operand rows in flight together; a slot past the end of the row
// re-reads the row's own operand row (its self-loop is in the sum anyway) with weight 0.
template <int GROUP, bool EPI>
__global__ void __launch_bounds__(256) spmm_rows_narrow_kernel(const int64_t* __restrict__ rowptr, const uint2* __restrict__ ecv,
                                                               const int32_t* __restrict__ rows, int nrows,
                                                               const float* __restrict__ Z, int ldz, float* __restrict__ out,
                                                               int ldo, int F4, EpiDev ep) {
    const int lane = threadIdx.x & 31, gl = lane & (GROUP - 1);
    const unsigned gmask = ((1u << GROUP) - 1u) << (lane & ~(GROUP - 1));
    const long long slot = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / GROUP;
    if (slot >= nrows) return;
    const int row = rows[slot];
    const long long e0 = rowptr[row], e1 = rowptr[row + 1];
    float4 acc[1] = {make_float4(0.f, 0.f, 0.f, 0.f)};
    for (long long e = e0; e < e1; e += GROUP) {
        uint2 mine = make_uint2((uint32_t)row, 0u);
        if (e + gl < e1) mine = __ldg(ecv + e + gl);
        float4 z[GROUP];
        float a[GROUP];
#pragma unroll
        for (int t = 0; t < GROUP; ++t) {
            const int c = __shfl_sync(gmask, (int)mine.x, t, GROUP);
            a[t] = __uint_as_float(__shfl_sync(gmask, mine.y, t, GROUP));
            z[t] = gl < F4 ? __ldg(reinterpret_cast<const float4*>(Z + (long long)c * ldz) + gl) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int t = 0; t < GROUP; ++t) {
            acc[0].x = fmaf(a[t], z[t].x, acc[0].x);
            acc[0].y = fmaf(a[t], z[t].y, acc[0].y);
            acc[0].z = fmaf(a[t], z[t].z, acc[0].z);
            acc[0].w = fmaf(a[t], z[t].w, acc[0].w);
        }
    }
    finish_row<1, EPI>(acc, row, gl, GROUP, F4, out, ldo, ep);
}

// One warp per row of the binned list.
template <int NV, int GROUP, bool EPI>
__global__ void __launch_bounds__(256) spmm_rows_kernel(const int64_t* __restrict__ rowptr, const uint2* __restrict__ ecv,
                                                        const int32_t* __restrict__ rows, int nrows,
                                                        const float* __restrict__ Z, int ldz, float* __restrict__ out,
                                                        int ldo, int F4, EpiDev ep) {
    const int lane = threadIdx.x & 31;
    const long long slot = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (slot >= nrows) return;
    const int row = rows[slot];
    float4 acc[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    walk_entries<NV, GROUP>(acc, ecv, rowptr[row], rowptr[row + 1], Z, ldz, lane, F4);
    if (lane < GROUP) finish_row<NV, EPI>(acc, row, lane, GROUP, F4, out, ldo, ep);
}

// Long rows are cut into parts; one warp per part, its partial row goes to the part's scratch slot and
// spmm_finish_kernel adds a row's slots in part order.  No barrier, no shared memory: a warp leaves as soon as
// its own entries are done.
template <int NV, int GROUP>
__global__ void __launch_bounds__(256) spmm_parts_kernel(const int64_t* __restrict__ rowptr, const uint2* __restrict__ ecv,
                                                         const int4* __restrict__ parts, int nparts,
                                                         const float* __restrict__ Z, int ldz, int ldo, int F4,
                                                         float* __restrict__ scratch) {
    const int lane = threadIdx.x & 31;
    const long long slot = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (slot >= nparts) return;
    const int4 pt = parts[slot];   // {row, first entry (relative to the row), entries, scratch slot}
    const long long e0 = rowptr[pt.x] + pt.y;
    float4 acc[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    walk_entries<NV, GROUP>(acc, ecv, e0, e0 + pt.z, Z, ldz, lane, F4);
    if (lane < GROUP) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            int v = lane + GROUP * j;
            if (v < F4) reinterpret_cast<float4*>(scratch + (long long)pt.w * ldo)[v] = acc[j];
        }
    }
}

// Rows made of several parts: their scratch slots added in part order, then the epilogue.  One warp per row.
template <int NV, int GROUP, bool EPI>
__global__ void __launch_bounds__(256) spmm_finish_kernel(const int4* __restrict__ fin, int nfin, const float* __restrict__ scratch,
                                                          float* __restrict__ out, int ldo, int F4, EpiDev ep) {
    const int lane = threadIdx.x & 31;
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= nfin || lane >= GROUP) return;
    const int4 f = fin[i];  // {row, first slot, slots, unused}
    float4 acc[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    // four slots are loaded together and added in slot order (a slot past the last one counts as zero)
    constexpr int Q = NV <= 2 ? 4 : (NV <= 4 ? 2 : 1);
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
    finish_row<NV, EPI>(acc, f.x, lane, GROUP, F4, out, ldo, ep);
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
template <int NV, bool OFF32>
struct ZLane {
    const char* base;      // OFF32: start of the operand (the same for the whole warp)
    const char* ptr[NV];   // otherwise: start of the operand plus the lane's column offset
    uint32_t off[NV];
    uint32_t ldzb;
    __device__ __forceinline__ float4 load(uint32_t c, int j) const {
        if constexpr (OFF32) return __ldg(reinterpret_cast<const float4*>(base + (c * ldzb + off[j])));
        else return __ldg(reinterpret_cast<const float4*>(ptr[j] + (unsigned long long)c * ldzb));
    }
};

template <int NV, int UU, bool OFF32>
__device__ __forceinline__ void gather_fma(float4 (&acc)[NV], const uint2* st, const ZLane<NV, OFF32>& zl) {
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
#pragma unroll
    for (int u = 0; u < UU; ++u)
#pragma unroll
        for (int j = 0; j < NV; ++j) z[u][j] = zl.load(c[u], j);
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

template <int NV, int V, bool OFF32>
__device__ __forceinline__ void gather_tail(float4 (&acc)[NV], const uint2* st, int r, const ZLane<NV, OFF32>& zl) {
    if constexpr (V >= 1) {
        if (r > V / 2) gather_fma<NV, V, OFF32>(acc, st, zl);
        else gather_tail<NV, V / 2, OFF32>(acc, st, r, zl);
    }
}

// Operand rows in flight per lane and resident warps asked of the compiler: short items make the chain
// item -> entries -> operand rows the cost, and more resident warps hide it better than more loads per warp.
#ifndef GAD_SPMM_UU1
#define GAD_SPMM_UU1 2
#endif
#ifndef GAD_SPMM_MINB1
#define GAD_SPMM_MINB1 16
#endif
#ifndef GAD_SPMM_UU2
#define GAD_SPMM_UU2 2
#endif
#ifndef GAD_SPMM_MINB2
#define GAD_SPMM_MINB2 10
#endif
constexpr int kItemWarps = 4;
template <int NV> struct ItemCfg {
    static constexpr int UU = NV == 1 ? GAD_SPMM_UU1 : (NV == 2 ? GAD_SPMM_UU2 : (NV <= 4 ? 2 : 1));
    static constexpr int MINB = NV == 1 ? GAD_SPMM_MINB1 : (NV == 2 ? GAD_SPMM_MINB2 : (NV <= 4 ? 6 : 4));   // CTAs of 4 warps per SM
};

template <int NV, bool EPI, bool OFF32>
__global__ void __launch_bounds__(32 * kItemWarps, ItemCfg<NV>::MINB)
spmm_items_kernel(const uint2* __restrict__ ecv, const int4* __restrict__ items, int nitems, const float* __restrict__ Z,
                  int ldz, float* __restrict__ out, int ldo, float* __restrict__ scratch, int F4, EpiDev ep) {
    constexpr int UU = ItemCfg<NV>::UU;
    __shared__ __align__(16) uint2 stage_all[kItemWarps][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int idx = blockIdx.x * kItemWarps + warp;
    if (idx >= nitems) return;
    uint2* stage = stage_all[warp];
    const int4 it = __ldg(items + idx);   // {row, entry position low, (position high << 16) | entries, scratch slot or -1}
    const int row = it.x, len = (int)((uint32_t)it.z & 0xFFFFu);
    const uint2* ent = ecv + (((long long)((uint32_t)it.z >> 16) << 32) | (long long)(uint32_t)it.y);
    const uint2 pad = make_uint2((uint32_t)row, 0u);
    // lanes past the last column read the last one (their sums are never stored)
    ZLane<NV, OFF32> zl;
    zl.base = reinterpret_cast<const char*>(Z);
    zl.ldzb = 4u * (uint32_t)ldz;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        zl.off[j] = 16u * (uint32_t)min(lane + 32 * j, F4 - 1);
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
        for (; t + UU / 2 < cnt; t += UU) gather_fma<NV, UU, OFF32>(acc, stage + t, zl);
        gather_tail<NV, UU / 2, OFF32>(acc, stage + t, cnt - t, zl);
    }
    if (it.w >= 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int v = lane + 32 * j;
            if (v < F4) reinterpret_cast<float4*>(scratch + (long long)it.w * ldo)[v] = acc[j];
        }
    } else {
        finish_row<NV, EPI>(acc, row, lane, 32, F4, out, ldo, ep);
    }
}

template <int NV, int GROUP, bool EPI>
static cudaError_t launch_rows(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F4, const EpiDev& ep,
                               cudaStream_t s) {
    if constexpr (GROUP == 32) {
        if (A.nitems > 0) {
            const unsigned grid = (unsigned)((A.nitems + kItemWarps - 1) / kItemWarps);
            // every byte of the operand within 4 GiB of its start: 32-bit offsets
            if ((unsigned long long)A.nrows * 4ull * (unsigned long long)ldz < (1ull << 32))
                spmm_items_kernel<NV, EPI, true><<<grid, 32 * kItemWarps, 0, s>>>(A.ecv, A.items, A.nitems, Z, ldz, out, ldo, A.scratch, F4, ep);
            else
                spmm_items_kernel<NV, EPI, false><<<grid, 32 * kItemWarps, 0, s>>>(A.ecv, A.items, A.nitems, Z, ldz, out, ldo, A.scratch, F4, ep);
            ++g_kernel_launches;
        }
        if (A.nfin > 0) {
            spmm_finish_kernel<NV, GROUP, EPI><<<(unsigned)((A.nfin + 7) / 8), 256, 0, s>>>(A.fin, A.nfin, A.scratch, out, ldo, F4, ep);
            ++g_kernel_launches;
        }
        return cudaGetLastError();
    }
    if (A.nparts > 0) {  // long rows first: they are the longest items of work
        spmm_parts_kernel<NV, GROUP><<<(unsigned)((A.nparts + 7) / 8), 256, 0, s>>>(A.rowptr, A.ecv, A.parts, A.nparts, Z, ldz, ldo, F4,
                                                                                   A.scratch);
        ++g_kernel_launches;
    }
    if (A.nfin > 0) {
        spmm_finish_kernel<NV, GROUP, EPI><<<(unsigned)((A.nfin + 7) / 8), 256, 0, s>>>(A.fin, A.nfin, A.scratch, out, ldo, F4, ep);
        ++g_kernel_launches;
    }
    if (A.nperm > 0) {
        if constexpr (GROUP < 32) {
            const unsigned grid = (unsigned)(((long long)A.nperm * GROUP + 255) / 256);
            spmm_rows_narrow_kernel<GROUP, EPI><<<grid, 256, 0, s>>>(A.rowptr, A.ecv, A.perm, A.nperm, Z, ldz, out, ldo, F4, ep);
        } else {
            const unsigned grid = (unsigned)((A.nperm + 7) / 8);
            spmm_rows_kernel<NV, GROUP, EPI><<<grid, 256, 0, s>>>(A.rowptr, A.ecv, A.perm, A.nperm, Z, ldz, out, ldo, F4, ep);
        }
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}

template <bool EPI>
static cudaError_t dispatch(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F4, const EpiDev& ep,
                            cudaStream_t s) {
    cudaError_t e;
#define GAD_ROWS(NV, G) { e = launch_rows<NV, G, EPI>(A, Z, ldz, out, ldo, F4, ep, s); if (e != cudaSuccess) return e; }
    if (F4 <= 4) GAD_ROWS(1, 4) else if (F4 <= 8) GAD_ROWS(1, 8) else if (F4 <= 16) GAD_ROWS(1, 16)
    else if (F4 <= 32) GAD_ROWS(1, 32) else if (F4 <= 64) GAD_ROWS(2, 32) else if (F4 <= 96) GAD_ROWS(3, 32)
    else if (F4 <= 128) GAD_ROWS(4, 32) else if (F4 <= 160) GAD_ROWS(5, 32) else if (F4 <= 192) GAD_ROWS(6, 32)
    else GAD_ROWS(8, 32)
#undef GAD_ROWS
    return cudaSuccess;
}

// F up to 1024 columns per pass (8 float4 per lane); wider operands are processed in column slabs.
cudaError_t launch_spmm(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F, const Epilogue* epi,
                        cudaStream_t s) {
    const int F4_all = (int)(round_up(F, 4) / 4);
    for (int c0 = 0; c0 < F4_all; c0 += 256) {
        const int F4 = min(256, F4_all - c0);
        EpiDev ep{};
        if (epi) {
            ep.act = make_act(*epi, 4 * c0);
            ep.sub_off = epi->sub_off; ep.K = epi->K;
        }
        cudaError_t e = epi ? dispatch<true>(A, Z + 4 * c0, ldz, out + 4 * c0, ldo, F4, ep, s)
                            : dispatch<false>(A, Z + 4 * c0, ldz, out + 4 * c0, ldo, F4, ep, s);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace gad
