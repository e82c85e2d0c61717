// Variance-based importance in its literal pairwise form (Section 3.4.1, the printed equation read as it stands):
//   zeta_k = sum over unordered pairs i < j of subgraph k of  p_i p_j / (|x_i - x_j|_2 + beta),
// p_i = deg_i / D_k (1 / n'_k when the subgraph has no edges), x the input features.  O(n'_k^2 F_0) work, so it is
// offered for subgraphs of at most kZetaPairMaxRows rows.
//
// The pairs of a subgraph are cut into 64 x 64 tiles (i-block <= j-block); one CTA of 16 x 16 threads owns a tile
// and each thread a 4 x 4 patch of it.  Squared distances are accumulated from the differences themselves
// (x_if - x_jf)^2 in fp32 - no Gram-matrix cancellation -, the weights and the sum over the tile in fp64 in a fixed
// order, one partial per tile; the last CTA of a subgraph to arrive adds the tile partials in tile order.
#include "gad_internal.h"

namespace gad {

namespace {

constexpr int PT = 64;        // rows of a tile side
constexpr int PF = 32;        // features staged per step

__device__ __forceinline__ bool arrive_last(unsigned* counter, unsigned expected) {
    __shared__ unsigned last_flag;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last_flag = (atomicAdd(counter, 1u) + 1u) % expected == 0u ? 1u : 0u;
    __syncthreads();
    const bool last = last_flag != 0u;
    if (last) __threadfence();
    return last;
}

__global__ void __launch_bounds__(256) zeta_pair_kernel(const float* __restrict__ X, int ld, int F, const int32_t* __restrict__ deg,
                                                        const int32_t* __restrict__ sub_off, const int64_t* __restrict__ deg_sum,
                                                        const int64_t* __restrict__ pair_ptr, int K, float beta, double* partial,
                                                        unsigned* counters, double* __restrict__ zeta) {
    __shared__ __align__(16) float xi[PF][PT + 4], xj[PF][PT + 4];
    __shared__ double red[8];
    __shared__ double seg[256];
    // subgraph of this CTA: largest k with pair_ptr[k] <= blockIdx.x (subgraphs without tiles are skipped by the <=)
    int lo = 0, hi = K;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pair_ptr[mid] <= (long long)blockIdx.x) lo = mid; else hi = mid;
    }
    const int k = lo;
    const int r0 = sub_off[k], n = sub_off[k + 1] - r0;
    const int T = (n + PT - 1) / PT;
    // tile (bi, bj), bi <= bj, from the CTA's position q in the row-major list of the upper triangle
    const long long q = (long long)blockIdx.x - pair_ptr[k];
    int bi = (int)(((double)(2 * T + 1) - sqrt((double)(2 * T + 1) * (double)(2 * T + 1) - 8.0 * (double)q)) * 0.5);
    bi = max(0, min(bi, T - 1));
    while (bi > 0 && (long long)bi * T - (long long)bi * (bi - 1) / 2 > q) --bi;              // rows before bi hold bi*T - bi(bi-1)/2 tiles
    while (bi + 1 < T && (long long)(bi + 1) * T - (long long)(bi + 1) * bi / 2 <= q) ++bi;
    const int bj = bi + (int)(q - ((long long)bi * T - (long long)bi * (bi - 1) / 2));

    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    const int i0 = bi * PT, j0 = bj * PT;
    const int ld4 = ld >> 2;
    for (int f0 = 0; f0 < F; f0 += PF) {
        // 64 rows x 32 features of each side, 16-byte loads, stored feature-major; pad columns of X are zero
        for (int t = threadIdx.x; t < PT * (PF / 4); t += 256) {
            const int r = t / (PF / 4), c4 = t % (PF / 4);
            float4 vi = make_float4(0.f, 0.f, 0.f, 0.f), vj = vi;
            if (f0 / 4 + c4 < ld4) {
                if (i0 + r < n) vi = __ldg(reinterpret_cast<const float4*>(X + (long long)(r0 + i0 + r) * ld) + f0 / 4 + c4);
                if (j0 + r < n) vj = __ldg(reinterpret_cast<const float4*>(X + (long long)(r0 + j0 + r) * ld) + f0 / 4 + c4);
            }
            xi[4 * c4 + 0][r] = vi.x; xi[4 * c4 + 1][r] = vi.y; xi[4 * c4 + 2][r] = vi.z; xi[4 * c4 + 3][r] = vi.w;
            xj[4 * c4 + 0][r] = vj.x; xj[4 * c4 + 1][r] = vj.y; xj[4 * c4 + 2][r] = vj.z; xj[4 * c4 + 3][r] = vj.w;
        }
        __syncthreads();
#pragma unroll 8
        for (int f = 0; f < PF; ++f) {
            const float4 av = *reinterpret_cast<const float4*>(&xi[f][4 * ty]);
            const float4 bv = *reinterpret_cast<const float4*>(&xj[f][4 * tx]);
            const float a[4] = {av.x, av.y, av.z, av.w}, b[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const float d = a[u] - b[v];
                    acc[u][v] = fmaf(d, d, acc[u][v]);
                }
        }
        __syncthreads();
    }
    // weights p_i p_j / (d + beta) of the pairs i < j inside the subgraph, summed in a fixed order
    const bool uniform = deg_sum[k] == 0;
    const double D = uniform ? (double)n : (double)deg_sum[k];
    double pi[4], pj[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int i = i0 + 4 * ty + u, j = j0 + 4 * tx + u;
        pi[u] = i < n ? (uniform ? 1.0 : (double)deg[r0 + i]) / D : 0.0;
        pj[u] = j < n ? (uniform ? 1.0 : (double)deg[r0 + j]) / D : 0.0;
    }
    double s = 0.0;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int i = i0 + 4 * ty + u, j = j0 + 4 * tx + v;
            if (i < j && j < n) s += (double)((float)(pi[u] * pj[v]) / (sqrtf(acc[u][v]) + beta));
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        partial[blockIdx.x] = t;
    }
    // the last tile of the subgraph to finish adds the tile sums: 256 segments of the tile list in parallel, then
    // the segment sums in order
    const long long np = pair_ptr[k + 1] - pair_ptr[k];
    if (!arrive_last(counters + k, (unsigned)np)) return;
    const long long len = (np + 255) / 256;
    const long long b0 = pair_ptr[k] + (long long)threadIdx.x * len, b1 = min((long long)pair_ptr[k + 1], b0 + len);
    double t = 0.0;
    for (long long c = b0; c < b1; ++c) t += __ldcg(partial + c);
    seg[threadIdx.x] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        double z = 0.0;
        for (int w = 0; w < 256; ++w) z += seg[w];
        zeta[k] = z;
    }
}

}  // namespace

// Tiles of subgraph k: T_k (T_k + 1) / 2 with T_k = ceil(n'_k / 64); pair_ptr is their prefix sum.
int64_t zeta_pair_tiles(int64_t rows) {
    const int64_t T = (rows + PT - 1) / PT;
    return T * (T + 1) / 2;
}

cudaError_t launch_zeta_pair(const float* X, int ld, int F, const int32_t* deg, const int32_t* sub_off, const int64_t* deg_sum,
                             const int64_t* pair_ptr, int64_t npairs, int K, float beta, double* partial, unsigned* counters,
                             double* zeta, cudaStream_t s) {
    if (npairs > 0) {
        zeta_pair_kernel<<<(unsigned)npairs, 256, 0, s>>>(X, ld, F, deg, sub_off, deg_sum, pair_ptr, K, beta, partial, counters, zeta);
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}

}  // namespace gad
