// SpMM over the block-diagonal store: out = A~ * Z (+ bias, ReLU, dropout on the forward pass), i.e. the
// aggregation half of the layer H^(l+1) = sigma(A~ (H^(l) W^(l)) + b) (Section 3.3, forward equation); run on
// the transposed store it is the backward aggregation dZ = A~^T dPre.
//
// Work split: a group of GROUP lanes (4..32) owns one row and walks its entries; every lane keeps NV float4
// accumulators, so a group covers 4*GROUP*NV feature columns with 16-byte loads of the dense operand.  Entries
// are fetched GROUP at a time as packed (column, value) pairs and handed round with shuffles.  Rows come from a
// list binned by length (heaviest first); rows above the hub threshold get a whole CTA each and a fixed-order
// shared-memory reduction, so results never depend on scheduling.
#include "gad_internal.h"

namespace gad {

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
    return z ^ (z >> 31);
}

// Row part of the dropout hash: (seed, epoch, layer, row) -> 64 bits; the column is mixed in per element.
__device__ __forceinline__ uint64_t dropout_row_key(uint64_t seed, int64_t epoch, int layer, int64_t row) {
    const uint64_t G = 0x9e3779b97f4a7c15ULL;
    uint64_t h = mix64(seed + G * (uint64_t)(1 + epoch));
    h = mix64(h + G * (uint64_t)(1 + layer));
    return mix64(h + G * (uint64_t)(1 + row));
}
__device__ __forceinline__ bool dropout_keep(uint64_t row_key, int col, uint32_t thr24) {
    const uint64_t G = 0x9e3779b97f4a7c15ULL;
    uint64_t h = mix64(row_key + G * (uint64_t)(1 + col));
    return (uint32_t)(h >> 40) >= thr24;
}

__device__ __forceinline__ int find_sub(const int32_t* __restrict__ sub_off, int K, int row) {
    int lo = 0, hi = K;  // largest k with sub_off[k] <= row (empty subgraphs are skipped by the <=)
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (sub_off[mid] <= row) lo = mid; else hi = mid;
    }
    return lo;
}

struct EpiDev {
    const float* params;
    long long pstride, b_int;
    const int32_t* sub_off;
    int K, relu, layer, col0;
    float dropout;
    unsigned long long seed;
    long long epoch;
};

template <int NV, bool EPI>
__device__ __forceinline__ void finish_row(float4 (&acc)[NV], int row, int gl, int group, int F4, float* __restrict__ out,
                                           int ldo, const EpiDev& ep) {
    if (EPI) {
        const int k = find_sub(ep.sub_off, ep.K, row);
        const float4* bias = reinterpret_cast<const float4*>(ep.params + (long long)k * ep.pstride + ep.b_int);
        const bool drop = ep.dropout > 0.f && ep.relu;
        const float scale = drop ? 1.f / (1.f - ep.dropout) : 1.f;
        const uint32_t thr = drop ? (uint32_t)floor((double)ep.dropout * 16777216.0) : 0u;
        const uint64_t key = drop ? dropout_row_key(ep.seed, ep.epoch, ep.layer, row) : 0ull;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            int v = gl + group * j;
            if (v >= F4) continue;
            float4 b = __ldg(bias + v);
            float x[4] = {acc[j].x + b.x, acc[j].y + b.y, acc[j].z + b.z, acc[j].w + b.w};
            if (ep.relu) {
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    x[t] = fmaxf(x[t], 0.f);
                    if (drop) x[t] = dropout_keep(key, ep.col0 + 4 * v + t, thr) ? x[t] * scale : 0.f;
                }
            }
            acc[j] = make_float4(x[0], x[1], x[2], x[3]);
        }
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        int v = gl + group * j;
        if (v < F4) reinterpret_cast<float4*>(out + (long long)row * ldo)[v] = acc[j];
    }
}

template <int NV>
__device__ __forceinline__ void fma_row(float4 (&acc)[NV], const float* __restrict__ Z, int ldz, int col, float a, int gl,
                                        int group, int F4) {
    const float4* zr = reinterpret_cast<const float4*>(Z + (long long)col * ldz);
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        int v = gl + group * j;
        if (v < F4) {
            float4 z = __ldg(zr + v);
            acc[j].x = fmaf(a, z.x, acc[j].x);
            acc[j].y = fmaf(a, z.y, acc[j].y);
            acc[j].z = fmaf(a, z.z, acc[j].z);
            acc[j].w = fmaf(a, z.w, acc[j].w);
        }
    }
}

// Entries [e0, e1) of one row accumulated by a group of lanes.
template <int NV, int GROUP>
__device__ __forceinline__ void walk_entries(float4 (&acc)[NV], const uint2* __restrict__ ecv, long long e0, long long e1,
                                             const float* __restrict__ Z, int ldz, int gl, unsigned gmask, int F4) {
    for (long long e = e0; e < e1; e += GROUP) {
        uint2 mine = make_uint2(0u, 0u);
        if (e + gl < e1) mine = __ldg(ecv + e + gl);
        int cnt = (int)min((long long)GROUP, e1 - e);
        int t = 0;
        for (; t + 4 <= cnt; t += 4) {
            int c0 = __shfl_sync(gmask, (int)mine.x, t + 0, GROUP), c1 = __shfl_sync(gmask, (int)mine.x, t + 1, GROUP);
            int c2 = __shfl_sync(gmask, (int)mine.x, t + 2, GROUP), c3 = __shfl_sync(gmask, (int)mine.x, t + 3, GROUP);
            float a0 = __uint_as_float(__shfl_sync(gmask, mine.y, t + 0, GROUP));
            float a1 = __uint_as_float(__shfl_sync(gmask, mine.y, t + 1, GROUP));
            float a2 = __uint_as_float(__shfl_sync(gmask, mine.y, t + 2, GROUP));
            float a3 = __uint_as_float(__shfl_sync(gmask, mine.y, t + 3, GROUP));
            fma_row<NV>(acc, Z, ldz, c0, a0, gl, GROUP, F4);
            fma_row<NV>(acc, Z, ldz, c1, a1, gl, GROUP, F4);
            fma_row<NV>(acc, Z, ldz, c2, a2, gl, GROUP, F4);
            fma_row<NV>(acc, Z, ldz, c3, a3, gl, GROUP, F4);
        }
        for (; t < cnt; ++t) {
            int c = __shfl_sync(gmask, (int)mine.x, t, GROUP);
            float a = __uint_as_float(__shfl_sync(gmask, mine.y, t, GROUP));
            fma_row<NV>(acc, Z, ldz, c, a, gl, GROUP, F4);
        }
    }
}

template <int NV, int GROUP, bool EPI>
__global__ void __launch_bounds__(256) spmm_rows_kernel(const int64_t* __restrict__ rowptr, const uint2* __restrict__ ecv,
                                                        const int32_t* __restrict__ rows, int nrows,
                                                        const float* __restrict__ Z, int ldz, float* __restrict__ out,
                                                        int ldo, int F4, EpiDev ep) {
    const int lane = threadIdx.x & 31;
    const int gl = lane & (GROUP - 1);
    const unsigned gmask = GROUP == 32 ? 0xffffffffu : (((1u << GROUP) - 1u) << (lane & ~(GROUP - 1)));
    const long long slot = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / GROUP;
    if (slot >= nrows) return;
    const int row = rows[slot];
    float4 acc[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    walk_entries<NV, GROUP>(acc, ecv, rowptr[row], rowptr[row + 1], Z, ldz, gl, gmask, F4);
    finish_row<NV, EPI>(acc, row, gl, GROUP, F4, out, ldo, ep);
}

// One CTA of 8 warps per hub row: warp w takes the w-th eighth of the entries; the eight partial rows are
// added in warp order.
template <int NV, bool EPI>
__global__ void __launch_bounds__(256) spmm_hub_kernel(const int64_t* __restrict__ rowptr, const uint2* __restrict__ ecv,
                                                       const int32_t* __restrict__ rows, const float* __restrict__ Z,
                                                       int ldz, float* __restrict__ out, int ldo, int F4, EpiDev ep) {
    extern __shared__ float4 part[];  // [8][F4]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = rows[blockIdx.x];
    const long long e0 = rowptr[row], e1 = rowptr[row + 1];
    const long long per = ((e1 - e0 + 7) / 8 + 31) / 32 * 32;
    const long long w0 = min(e1, e0 + per * warp), w1 = min(e1, w0 + per);
    float4 acc[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    walk_entries<NV, 32>(acc, ecv, w0, w1, Z, ldz, lane, 0xffffffffu, F4);
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        int v = lane + 32 * j;
        if (v < F4) part[warp * F4 + v] = acc[j];
    }
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            int v = lane + 32 * j;
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
            if (v < F4)
                for (int w = 0; w < 8; ++w) {
                    float4 p = part[w * F4 + v];
                    s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w;
                }
            acc[j] = s;
        }
        finish_row<NV, EPI>(acc, row, lane, 32, F4, out, ldo, ep);
    }
}

template <int NV, int GROUP, bool EPI>
static cudaError_t launch_rows(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F4, const EpiDev& ep,
                               cudaStream_t s) {
    if (A.nperm > 0) {
        const int rows_per_cta = 256 / GROUP;
        const unsigned grid = (unsigned)((A.nperm + rows_per_cta - 1) / rows_per_cta);
        spmm_rows_kernel<NV, GROUP, EPI><<<grid, 256, 0, s>>>(A.rowptr, A.ecv, A.perm, A.nperm, Z, ldz, out, ldo, F4, ep);
    }
    return cudaGetLastError();
}
template <int NV, bool EPI>
static cudaError_t launch_hub(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F4, const EpiDev& ep,
                              cudaStream_t s) {
    if (A.nhub > 0)
        spmm_hub_kernel<NV, EPI><<<(unsigned)A.nhub, 256, (size_t)8 * F4 * sizeof(float4), s>>>(A.rowptr, A.ecv, A.hub, Z, ldz,
                                                                                               out, ldo, F4, ep);
    return cudaGetLastError();
}

template <bool EPI>
static cudaError_t dispatch(const SparseDev& A, const float* Z, int ldz, float* out, int ldo, int F4, const EpiDev& ep,
                            cudaStream_t s) {
    cudaError_t e;
#define GAD_ROWS(NV, G) { e = launch_rows<NV, G, EPI>(A, Z, ldz, out, ldo, F4, ep, s); if (e != cudaSuccess) return e; }
#define GAD_HUB(NV) { e = launch_hub<NV, EPI>(A, Z, ldz, out, ldo, F4, ep, s); if (e != cudaSuccess) return e; }
    // hub rows first: they are the longest items of work
    if (F4 <= 32) GAD_HUB(1) else if (F4 <= 64) GAD_HUB(2) else if (F4 <= 96) GAD_HUB(3) else if (F4 <= 128) GAD_HUB(4)
    else if (F4 <= 160) GAD_HUB(5) else if (F4 <= 192) GAD_HUB(6) else GAD_HUB(8)
    if (F4 <= 4) GAD_ROWS(1, 4) else if (F4 <= 8) GAD_ROWS(1, 8) else if (F4 <= 16) GAD_ROWS(1, 16)
    else if (F4 <= 32) GAD_ROWS(1, 32) else if (F4 <= 64) GAD_ROWS(2, 32) else if (F4 <= 96) GAD_ROWS(3, 32)
    else if (F4 <= 128) GAD_ROWS(4, 32) else if (F4 <= 160) GAD_ROWS(5, 32) else if (F4 <= 192) GAD_ROWS(6, 32)
    else GAD_ROWS(8, 32)
#undef GAD_ROWS
#undef GAD_HUB
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
            ep.params = epi->params; ep.pstride = epi->pstride; ep.b_int = epi->b_int + 4ll * c0;
            ep.sub_off = epi->sub_off; ep.K = epi->K; ep.relu = epi->relu; ep.layer = epi->layer;
            ep.dropout = epi->dropout; ep.seed = epi->seed; ep.epoch = epi->epoch; ep.col0 = 4 * c0;
        }
        cudaError_t e = epi ? dispatch<true>(A, Z + 4 * c0, ldz, out + 4 * c0, ldo, F4, ep, s)
                            : dispatch<false>(A, Z + 4 * c0, ldz, out + 4 * c0, ldo, F4, ep, s);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace gad
