// gad_subgraph_weights_static: the subgraph-importance computation for callers that cannot allocate.
//
// Some users of this library run where nobody may call cudaMalloc on their behalf: a serving process that has
// handed the whole device to its own memory pool, a plug-in inside a framework whose allocator owns the GPU, or a
// latency-critical loop in which an allocation (which can synchronise the device) is not acceptable.  The regular
// path keeps its partial sums in the caller's workspace; this variant keeps them in a fixed array that is part of
// the library image, so the call needs no workspace at all: inputs and outputs only.
//
// The price: the array has a fixed, modest size (the limits below), every GPU that loads the library holds it
// until the process exits, and all calls share it.  Nothing in it has to be cleared between calls (each call
// overwrites every slot it later reads), but two calls whose kernels overlap on the GPU - different streams, or
// different host threads - would write the same slots and race.  Issue them on one stream, or serialise them.
#include <mutex>

#include "gad_internal.h"

namespace {

constexpr int kMaxK = 256;            // subgraphs
constexpr int kMaxLd = 4096;          // leading dimension of the feature matrix
constexpr long long kMaxKLd = 16384;  // K * ld
constexpr int kSlices = 16;           // row slices per subgraph

struct StaticScratch {
    double part[kMaxKLd * kSlices * 2];  // per (subgraph, slice): sum w (x - c), then sum w (x - c)^2, per feature
    long long deg_sum[kMaxK];
    long long deg_sq[kMaxK];
    double zeta[kMaxK];
};

// Device storage.  In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

constexpr int kMaxDevices = 64;
StaticScratch* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_setup_mutex;

// Sum of the local degrees and of their squares over one subgraph (exact, in 64-bit integers).
// Rows of subgraph k, cut to [0, rows): a sub_off array that does not match the matrix must not lead outside it.
__device__ __forceinline__ void sub_range(const int32_t* __restrict__ sub_off, int k, long long rows, int& r0, int& n) {
    const long long lo = min(max((long long)sub_off[k], 0ll), rows), hi = min(max((long long)sub_off[k + 1], lo), rows);
    r0 = (int)lo;
    n = (int)(hi - lo);
}

__global__ void __launch_bounds__(256) static_degree_kernel(const int32_t* __restrict__ deg, const int32_t* __restrict__ sub_off,
                                                            long long rows, StaticScratch* sc) {
    __shared__ long long s1[256], s2[256];
    const int k = blockIdx.x;
    long long a = 0, b = 0;
    int first, cnt;
    sub_range(sub_off, k, rows, first, cnt);
    for (int r = first + threadIdx.x; r < first + cnt; r += blockDim.x) {
        const long long d = deg[r];
        a += d;
        b += d * d;
    }
    s1[threadIdx.x] = a;
    s2[threadIdx.x] = b;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) { s1[threadIdx.x] += s1[threadIdx.x + o]; s2[threadIdx.x] += s2[threadIdx.x + o]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { sc->deg_sum[k] = s1[0]; sc->deg_sq[k] = s2[0]; }
}

// Weighted first and second moments of every feature over one slice of one subgraph's rows, shifted by the
// subgraph's first row.  Threads: 8 row lanes x 32 column lanes of one float4 each.
__global__ void __launch_bounds__(256) static_partial_kernel(const float* __restrict__ X, int ld, const int32_t* __restrict__ deg,
                                                             const int32_t* __restrict__ sub_off, long long rows, StaticScratch* sc) {
    __shared__ double sm[8][32][8];
    const int k = blockIdx.y, slice = blockIdx.x;
    int r0, n;
    sub_range(sub_off, k, rows, r0, n);
    const int per = (n + kSlices - 1) / kSlices;
    const int lo = min(n, slice * per), hi = min(n, lo + per);
    const bool uniform = sc->deg_sum[k] == 0;
    const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
    const int ld4 = ld >> 2;
    double* P = sc->part + ((long long)k * kSlices + slice) * 2 * ld;
    for (int v0 = 0; v0 < ld4; v0 += 32) {
        const int v = v0 + cx;
        double a[4] = {0.0, 0.0, 0.0, 0.0}, b[4] = {0.0, 0.0, 0.0, 0.0};
        if (v < ld4 && n > 0) {
            const float4 sh = reinterpret_cast<const float4*>(X + (long long)r0 * ld)[v];
            for (int r = lo + ry; r < hi; r += 8) {
                const float4 u = reinterpret_cast<const float4*>(X + (long long)(r0 + r) * ld)[v];
                const double w = uniform ? 1.0 : (double)deg[r0 + r];
                const double d[4] = {(double)(u.x - sh.x), (double)(u.y - sh.y), (double)(u.z - sh.z), (double)(u.w - sh.w)};
#pragma unroll
                for (int t = 0; t < 4; ++t) { a[t] = fma(w, d[t], a[t]); b[t] = fma(w * d[t], d[t], b[t]); }
            }
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) { sm[ry][cx][t] = a[t]; sm[ry][cx][4 + t] = b[t]; }
        __syncthreads();
        if (ry == 0 && v < ld4) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                double sa = 0.0, sb = 0.0;
                for (int w = 0; w < 8; ++w) { sa += sm[w][cx][t]; sb += sm[w][cx][4 + t]; }
                P[4 * v + t] = sa;       // every slot is rewritten on every call, empty slices included
                P[ld + 4 * v + t] = sb;
            }
        }
        __syncthreads();
    }
}

// zeta_k = S_k / (D_k + beta) from the slice sums, slices added in order.
__global__ void __launch_bounds__(256) static_final_kernel(int F, int ld, const int32_t* __restrict__ sub_off, long long rows, float beta,
                                                           StaticScratch* sc, float* __restrict__ zeta_out) {
    __shared__ double red[256];
    const int k = blockIdx.x;
    int first, cnt;
    sub_range(sub_off, k, rows, first, cnt);
    const long long n = cnt;
    const bool uniform = sc->deg_sum[k] == 0;
    const double D = uniform ? (double)n : (double)sc->deg_sum[k];
    double q = 0.0;
    if (n > 0)
        for (int f = threadIdx.x; f < F; f += blockDim.x) {
            double a = 0.0, b = 0.0;
            for (int s = 0; s < kSlices; ++s) {
                const double* P = sc->part + ((long long)k * kSlices + s) * 2 * ld;
                a += P[f];
                b += P[ld + f];
            }
            const double m1 = a / D;
            q += b / D - m1 * m1;
        }
    red[threadIdx.x] = q;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        double z = 0.0;
        if (n > 0) {
            const double sq = uniform ? 1.0 / (double)n : (double)sc->deg_sq[k] / (D * D);
            const double S = 0.5 * (1.0 - sq);
            const double Q = red[0] > 0.0 ? red[0] : 0.0;
            if (S > 0.0) z = S / (sqrt(Q / S) + (double)beta);
        }
        sc->zeta[k] = z;
        zeta_out[k] = (float)z;
    }
}

__global__ void static_weights_kernel(int K, int weighted, const StaticScratch* sc, float* __restrict__ w_out) {
    __shared__ double total;
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int k = 0; k < K; ++k) t += sc->zeta[k];
        total = t;
    }
    __syncthreads();
    for (int k = threadIdx.x; k < K; k += blockDim.x)
        w_out[k] = (weighted && total > 0.0) ? (float)(sc->zeta[k] / total) : 1.f / (float)K;
}

}  // namespace

extern "C" int gad_subgraph_weights_static(const float* X, int64_t rows, int32_t F, int32_t ld, const int32_t* deg,
                                           const int32_t* sub_off, int32_t K, float beta, int32_t weighted, float* zeta_out,
                                           float* w_out, void* stream) {
    if (!X || !deg || !sub_off || !zeta_out || !w_out) return GAD_ERR_ARG;
    if (rows < 0 || rows >= ((int64_t)1 << 31) || K < 1 || F < 1 || ld < F || (ld & 3) != 0 || !(beta > 0.f)) return GAD_ERR_ARG;
    if (((uintptr_t)X & 15) != 0) return GAD_ERR_ARG;
    // the fixed scratch array bounds the problem: refuse anything that would not fit
    if (K > kMaxK || ld > kMaxLd || (long long)K * ld > kMaxKLd) return GAD_ERR_RANGE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GAD_ERR_CUDA;
    StaticScratch* sc = nullptr;
    {
        // once per device, with that device current: turn the symbol into its device address
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_scratch_ptr[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return GAD_ERR_CUDA;
            g_scratch_ptr[dev] = static_cast<StaticScratch*>(p);
        }
        sc = g_scratch_ptr[dev];
    }
    cudaStream_t s = (cudaStream_t)stream;
    static_degree_kernel<<<(unsigned)K, 256, 0, s>>>(deg, sub_off, (long long)rows, sc);
    static_partial_kernel<<<dim3(kSlices, (unsigned)K), 256, 0, s>>>(X, ld, deg, sub_off, (long long)rows, sc);
    static_final_kernel<<<(unsigned)K, 256, 0, s>>>(F, ld, sub_off, (long long)rows, beta, sc, zeta_out);
    static_weights_kernel<<<1, 256, 0, s>>>(K, weighted, sc, w_out);
    gad::g_kernel_launches += 4;
    return cudaGetLastError() == cudaSuccess ? GAD_OK : GAD_ERR_CUDA;
}
