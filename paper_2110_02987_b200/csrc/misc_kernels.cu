// Memory-bound kernels of the epoch other than the SpMM: fused softmax cross-entropy with its gradient,
// chunked column sums, the statistics of the variance-based importance weight, the fused SGD step +
// weighted global consensus, and the create-time / accessor gathers.  Every reduction runs in a fixed order
// (rows of a chunk in order, chunks of a subgraph in order, replicas in ascending k), so a run is bitwise
// reproducible.
#include <math.h>

#include "gad_internal.h"

namespace gad {

// ---------------------------------------------------------------------------------------------
// "The last CTA finishes the reduction": every CTA writes its partial result, then counts itself in; the CTA
// whose arrival completes the group adds the partial results in their fixed order.  Which CTA that is varies
// from run to run, the order of the additions does not, so the results stay bitwise reproducible.  Counters only
// grow (a group is complete at every multiple of its size), so they never need resetting.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ bool cta_arrive_last(unsigned* counter, unsigned expected) {
    __shared__ unsigned last_flag;
    __threadfence();                  // this CTA's partial results are visible before its arrival is counted
    __syncthreads();
    if (threadIdx.x == 0) last_flag = (atomicAdd(counter, 1u) + 1u) % expected == 0u ? 1u : 0u;
    __syncthreads();
    const bool last = last_flag != 0u;
    if (last) __threadfence();        // the other CTAs published their results before they arrived
    return last;
}

// Sum over the chunks [c0, c1) of src[c * stride + j], for one column j, as the finishing CTA does it: the chunk
// range is cut into `nseg` equal segments, segment `seg` is added in chunk order by the calling thread (up to
// eight loads in flight), and the caller then adds the segment sums in segment order.  The order of the additions
// depends only on (c0, c1, nseg).
template <class T>
__device__ __forceinline__ T segment_sum(const T* src, long long stride, long long j, int c0, int c1, int seg, int nseg) {
    const int len = (c1 - c0 + nseg - 1) / nseg;
    int c = c0 + seg * len;
    const int e = min(c1, c + len);
    T s = (T)0;
    for (; c + 8 <= e; c += 8) {
        T v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = __ldcg(src + (long long)(c + u) * stride + j);
#pragma unroll
        for (int u = 0; u < 8; ++u) s += v[u];
    }
    for (; c < e; ++c) s += __ldcg(src + (long long)c * stride + j);
    return s;
}
// Columns are handled 256 / nseg at a time; nseg = 256 / (columns rounded up to a power of two), at least 1.
__device__ __forceinline__ int segments_for(int cols) {
    int p = 1;
    while (p < cols && p < 256) p <<= 1;
    return 256 / p;
}

struct LossTail {
    const int32_t* chunk_ptr;   // [K+1]
    int K;
    float inv_total;
    float* loss;                // [K+1]
    int32_t* nonfinite;
    unsigned* counter;
};

// The chunk sums are first brought into shared memory by the whole CTA (4096 at a time); one thread per subgraph
// then adds its subgraph's sums in chunk order, and thread 0 adds the K subgraph sums in ascending k for the global
// loss sum_k |T_k| L_k / sum_k |T_k|.
__device__ __forceinline__ void loss_finalize(const float* loss_partial, const float* __restrict__ inv_ntrain, const LossTail& t) {
    __shared__ float stage[4096];
    __shared__ float sums[1024];
    const int nchunks = t.chunk_ptr[t.K];
    const bool staged = nchunks <= 4096;
    if (staged)
        for (int c = threadIdx.x; c < nchunks; c += blockDim.x) stage[c] = __ldcg(loss_partial + c);
    __syncthreads();
    for (int k = threadIdx.x; k < t.K; k += blockDim.x) {
        float s = 0.f;
        for (int c = t.chunk_ptr[k]; c < t.chunk_ptr[k + 1]; ++c) s += staged ? stage[c] : __ldcg(loss_partial + c);
        if (k < 1024) sums[k] = s;
        t.loss[k] = s * inv_ntrain[k];
        if (!isfinite(s)) atomicExch(t.nonfinite, 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int k = 0; k < t.K; ++k) {
            if (k < 1024) { s += sums[k]; continue; }
            float sk = 0.f;
            for (int c = t.chunk_ptr[k]; c < t.chunk_ptr[k + 1]; ++c) sk += staged ? stage[c] : __ldcg(loss_partial + c);
            s += sk;
        }
        t.loss[t.K] = s * t.inv_total;
    }
}

// ---------------------------------------------------------------------------------------------
// Softmax cross-entropy over the core training rows and d(loss)/d(logits)  (loss equation, Section 3.3, read
// as multi-class cross-entropy averaged over the subgraph's training nodes).  One CTA per row chunk, one warp
// per row; lanes stride over the classes.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) softmax_xent_kernel(const float* __restrict__ logits, int ld, int C,
                                                           const int32_t* __restrict__ label,
                                                           const uint8_t* __restrict__ train,
                                                           const RowSpan* __restrict__ chunks,
                                                           const float* __restrict__ inv_ntrain,
                                                           float* __restrict__ dlogits, float* loss_partial, LossTail fin) {
    __shared__ float wsum[8];
    const RowSpan c = chunks[blockIdx.x];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float inv = inv_ntrain[c.k];
    float acc = 0.f;
    for (int r = warp; r < c.nrows; r += 8) {
        const long long row = c.row0 + r;
        const float* z = logits + row * ld;
        float* g = dlogits + row * ld;
        if (!train[row]) {
            for (int j = lane; j < ld; j += 32) g[j] = 0.f;
            continue;
        }
        float mx = -INFINITY;
        for (int j = lane; j < C; j += 32) mx = fmaxf(mx, z[j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float se = 0.f;
        for (int j = lane; j < C; j += 32) se += expf(z[j] - mx);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
        const float lse = mx + logf(se);
        const int y = label[row];
        acc += lse - z[y];
        for (int j = lane; j < ld; j += 32) {
            float v = 0.f;
            if (j < C) v = (expf(z[j] - lse) - (j == y ? 1.f : 0.f)) * inv;
            g[j] = v;
        }
    }
    if (lane == 0) wsum[warp] = acc;  // every lane holds the same acc
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int w = 0; w < 8; ++w) s += wsum[w];
        loss_partial[blockIdx.x] = s;
    }
    if (cta_arrive_last(fin.counter, gridDim.x)) loss_finalize(loss_partial, inv_ntrain, fin);
}

// Up to 128 classes: L lanes hold one row (a float4 each), 32/L rows per warp step, the row stays in registers.
template <int L>
__global__ void __launch_bounds__(256) softmax_xent_small_kernel(const float* __restrict__ logits, int ld, int C,
                                                                 const int32_t* __restrict__ label,
                                                                 const uint8_t* __restrict__ train,
                                                                 const RowSpan* __restrict__ chunks,
                                                                 const float* __restrict__ inv_ntrain,
                                                                 float* __restrict__ dlogits, float* loss_partial, LossTail fin) {
    constexpr int RPW = 32 / L;
    __shared__ float wsum[8];
    const RowSpan c = chunks[blockIdx.x];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane / L, gl = lane & (L - 1);
    const unsigned gmask = L == 32 ? 0xffffffffu : (((1u << L) - 1u) << (lane & ~(L - 1)));
    const int ld4 = ld >> 2;
    const float inv = inv_ntrain[c.k];
    float acc = 0.f;
    // the loads of a row (loss mask, label, logits) do not wait for one another, and the next row's are requested
    // before this row's are used
    struct RowIn { bool train; int y; float4 v; };
    auto fetch = [&](int r) {
        RowIn in{false, 0, make_float4(0.f, 0.f, 0.f, 0.f)};
        if (r < c.nrows) {
            const long long row = c.row0 + r;
            in.train = train[row] != 0;
            in.y = label[row];
            if (gl < ld4) in.v = reinterpret_cast<const float4*>(logits + row * ld)[gl];
        }
        return in;
    };
    int r = warp * RPW + g;
    RowIn cur = fetch(r);
    for (; r < c.nrows; r += 8 * RPW) {
        const RowIn nxt = fetch(r + 8 * RPW);
        const long long row = c.row0 + r;
        float4* gout = reinterpret_cast<float4*>(dlogits + row * ld);
        if (!cur.train) {
            if (gl < ld4) gout[gl] = make_float4(0.f, 0.f, 0.f, 0.f);
            cur = nxt;
            continue;
        }
        float z[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (gl < ld4) {
            const float4 v = cur.v;
            if (4 * gl + 0 < C) z[0] = v.x;
            if (4 * gl + 1 < C) z[1] = v.y;
            if (4 * gl + 2 < C) z[2] = v.z;
            if (4 * gl + 3 < C) z[3] = v.w;
        }
        float mx = fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3]));
#pragma unroll
        for (int o = L / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(gmask, mx, o, L));
        float se = 0.f;
#pragma unroll
        for (int t = 0; t < 4; ++t) se += 4 * gl + t < C ? expf(z[t] - mx) : 0.f;
#pragma unroll
        for (int o = L / 2; o > 0; o >>= 1) se += __shfl_xor_sync(gmask, se, o, L);
        const float lse = mx + logf(se);
        const int y = cur.y;
        const int yt = y & 3;
        const float mine = yt == 0 ? z[0] : (yt == 1 ? z[1] : (yt == 2 ? z[2] : z[3]));
        const float zy = __shfl_sync(gmask, mine, y >> 2, L);
        if (gl == 0) acc += lse - zy;
        if (gl < ld4) {
            float o4[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int j = 4 * gl + t;
                o4[t] = j < C ? (expf(z[t] - lse) - (j == y ? 1.f : 0.f)) * inv : 0.f;
            }
            gout[gl] = make_float4(o4[0], o4[1], o4[2], o4[3]);
        }
        cur = nxt;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) wsum[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int w = 0; w < 8; ++w) s += wsum[w];
        loss_partial[blockIdx.x] = s;
    }
    if (cta_arrive_last(fin.counter, gridDim.x)) loss_finalize(loss_partial, inv_ntrain, fin);
}

cudaError_t launch_softmax_xent(const float* logits, int ld, int C, const int32_t* label, const uint8_t* train,
                                const RowSpan* chunks, int nchunks, const float* inv_ntrain, float* dlogits,
                                float* loss_partial, const int32_t* chunk_ptr, int K, float inv_total, float* loss,
                                int32_t* nonfinite, unsigned* counter, cudaStream_t s) {
    if (nchunks > 0) {
        const int ld4 = ld >> 2;
        const LossTail fin{chunk_ptr, K, inv_total, loss, nonfinite, counter};
#define GAD_SMALL(L) softmax_xent_small_kernel<L><<<(unsigned)nchunks, 256, 0, s>>>(logits, ld, C, label, train, chunks, inv_ntrain, dlogits, loss_partial, fin)
        if (ld4 <= 1) GAD_SMALL(1);
        else if (ld4 <= 2) GAD_SMALL(2);
        else if (ld4 <= 4) GAD_SMALL(4);
        else if (ld4 <= 8) GAD_SMALL(8);
        else if (ld4 <= 16) GAD_SMALL(16);
        else if (ld4 <= 32) GAD_SMALL(32);
        else softmax_xent_kernel<<<(unsigned)nchunks, 256, 0, s>>>(logits, ld, C, label, train, chunks, inv_ntrain, dlogits, loss_partial, fin);
#undef GAD_SMALL
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Column sums of a row chunk (bias gradient db = column sums of dPre over the subgraph's rows).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) colsum_chunks_kernel(const float* __restrict__ G, int ld,
                                                            const RowSpan* __restrict__ chunks, float* partial,
                                                            long long pstride_chunk, const int32_t* __restrict__ chunk_ptr,
                                                            unsigned* counters, float* __restrict__ out, long long ostride,
                                                            long long off) {
    // threads = 8 row lanes x 32 column lanes of one float4 each; a block of 128 columns is summed over the
    // rows ry, ry+8, ... by every row lane and the 8 row lanes are then added in order
    __shared__ float4 sm[8][32];
    const RowSpan c = chunks[blockIdx.x];
    const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
    const int ld4 = ld >> 2;
    for (int v0 = 0; v0 < ld4; v0 += 32) {
        const int v = v0 + cx;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        if (v < ld4) {
            const float4* g = reinterpret_cast<const float4*>(G + (long long)c.row0 * ld) + v;
            int r = ry;
            for (; r + 24 < c.nrows; r += 32) {
                float4 a0 = g[(long long)r * ld4], a1 = g[(long long)(r + 8) * ld4];
                float4 a2 = g[(long long)(r + 16) * ld4], a3 = g[(long long)(r + 24) * ld4];
                s.x += a0.x; s.y += a0.y; s.z += a0.z; s.w += a0.w;
                s.x += a1.x; s.y += a1.y; s.z += a1.z; s.w += a1.w;
                s.x += a2.x; s.y += a2.y; s.z += a2.z; s.w += a2.w;
                s.x += a3.x; s.y += a3.y; s.z += a3.z; s.w += a3.w;
            }
            for (; r < c.nrows; r += 8) {
                float4 a0 = g[(long long)r * ld4];
                s.x += a0.x; s.y += a0.y; s.z += a0.z; s.w += a0.w;
            }
        }
        sm[ry][cx] = s;
        __syncthreads();
        if (ry == 0 && v < ld4) {
            float4 t = sm[0][cx];
            for (int w = 1; w < 8; ++w) { t.x += sm[w][cx].x; t.y += sm[w][cx].y; t.z += sm[w][cx].z; t.w += sm[w][cx].w; }
            reinterpret_cast<float4*>(partial + (long long)blockIdx.x * pstride_chunk)[v] = t;
        }
        __syncthreads();
    }
    // the last CTA of this subgraph adds the subgraph's chunk sums: segments of the chunk range in parallel, then
    // the segment sums in order
    const int c0 = chunk_ptr[c.k], c1 = chunk_ptr[c.k + 1];
    if (!cta_arrive_last(counters + c.k, (unsigned)(c1 - c0))) return;
    float* seg_sm = reinterpret_cast<float*>(sm);   // 256 floats of the 4 KiB tile above
    const int nseg = segments_for(ld), per = 256 / nseg;
    const int jl = threadIdx.x % per, seg = threadIdx.x / per;
    for (int j0 = 0; j0 < ld; j0 += per) {
        const int j = j0 + jl;
        seg_sm[threadIdx.x] = j < ld ? segment_sum(partial, pstride_chunk, j, c0, c1, seg, nseg) : 0.f;
        __syncthreads();
        if (seg == 0 && j < ld) {
            float t = seg_sm[jl];
            for (int q = 1; q < nseg; ++q) t += seg_sm[q * per + jl];
            out[(long long)c.k * ostride + off + j] = t;
        }
        __syncthreads();
    }
}
// Column sums of G over every subgraph's rows: out[k][off + j] = sum over the rows of subgraph k of G[row][j], j < ld.
cudaError_t launch_colsum_chunks(const float* G, int ld, const RowSpan* chunks, int nchunks, float* partial,
                                 int64_t pstride_chunk, const int32_t* chunk_ptr, unsigned* counters, float* out,
                                 int64_t ostride, int64_t off, cudaStream_t s) {
    if (nchunks > 0) {
        colsum_chunks_kernel<<<(unsigned)nchunks, 256, 0, s>>>(G, ld, chunks, partial, pstride_chunk, chunk_ptr, counters, out, ostride, off);
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}

__global__ void reduce_chunks_kernel(const float* __restrict__ partial, long long pstride_chunk,
                                     const int32_t* __restrict__ chunk_ptr, float* __restrict__ out, long long ostride,
                                     long long off, long long len) {
    const int k = blockIdx.y;
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= len) return;
    float s = 0.f;
    const int c1 = chunk_ptr[k + 1];
    int c = chunk_ptr[k];
    for (; c + 8 <= c1; c += 8) {   // eight chunks' values requested together, added in chunk order
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = partial[(long long)(c + u) * pstride_chunk + i];
#pragma unroll
        for (int u = 0; u < 8; ++u) s += v[u];
    }
    for (; c < c1; ++c) s += partial[(long long)c * pstride_chunk + i];
    out[(long long)k * ostride + off + i] = s;
}
cudaError_t launch_reduce_chunks(const float* partial, int64_t pstride_chunk, const int32_t* chunk_ptr, int K, float* out,
                                 int64_t ostride, int64_t off, int64_t len, cudaStream_t s) {
    if (len > 0 && K > 0) {
        reduce_chunks_kernel<<<dim3((unsigned)((len + 255) / 256), (unsigned)K), 256, 0, s>>>(partial, pstride_chunk, chunk_ptr, out,
                                                                                               ostride, off, len); ++g_kernel_launches; }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Variance-based importance (Section 3.4.1).  With p_i = deg_i / D (D = sum of local degrees; weight 1 and
// D = n' when the subgraph has no edges) the distance statistic splits by feature dimension:
//   sum_{i<j} p_i p_j |x_i - x_j|^2 = sum_f ( sum_i p_i (x_if - c_f)^2 - (sum_i p_i (x_if - c_f))^2 )
// for any shift c_f; c_f = the subgraph's first row keeps the two sums small.  This kernel accumulates the
// two weighted sums per chunk and per feature in double precision.
// ---------------------------------------------------------------------------------------------
// zeta_k = S_k / (D_k + beta) from the chunk sums of subgraph k, chunks added in order; run by one whole CTA.
// `phase` spreads one zeta over several matrices (the layers' inputs, zeta_mode 2): 0 = this matrix alone; 1 = the first
// of several (its distance sum goes to q_acc[k]); 2 = a further one (added to q_acc[k]); 3 = the last one (added, then zeta).
__device__ __forceinline__ void zeta_finalize(int k, const double* partial, int F, int ld, const int32_t* __restrict__ chunk_ptr,
                                              const int32_t* __restrict__ sub_off, const int64_t* __restrict__ deg_sum,
                                              const int64_t* __restrict__ deg_sq, float beta, double* __restrict__ zeta,
                                              double* __restrict__ q_acc, int phase) {
    __shared__ double red[256];
    __shared__ double seg_a[256], seg_b[256];
    const long long n = sub_off[k + 1] - sub_off[k];
    const bool uniform = deg_sum[k] == 0;
    const double D = uniform ? (double)n : (double)deg_sum[k];
    double q = 0.0;
    if (n > 0) {
        // segments of the chunk range in parallel, the segment sums then added in order, per feature
        const int c0 = chunk_ptr[k], c1 = chunk_ptr[k + 1];
        const int nseg = segments_for(F), per = 256 / nseg;
        const int fl = threadIdx.x % per, seg = threadIdx.x / per;
        for (int f0 = 0; f0 < F; f0 += per) {
            const int f = f0 + fl;
            seg_a[threadIdx.x] = f < F ? segment_sum(partial, 2ll * ld, f, c0, c1, seg, nseg) : 0.0;
            seg_b[threadIdx.x] = f < F ? segment_sum(partial, 2ll * ld, (long long)ld + f, c0, c1, seg, nseg) : 0.0;
            __syncthreads();
            if (seg == 0 && f < F) {
                double a = seg_a[fl], b = seg_b[fl];
                for (int t = 1; t < nseg; ++t) { a += seg_a[t * per + fl]; b += seg_b[t * per + fl]; }
                const double m1 = a / D;
                q += b / D - m1 * m1;
            }
            __syncthreads();
        }
    }
    red[threadIdx.x] = q;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        double Q = red[0] > 0.0 ? red[0] : 0.0;
        if (phase == 2 || phase == 3) Q += q_acc[k];
        if (phase == 1 || phase == 2) {
            q_acc[k] = Q;
        } else {
            double z = 0.0;
            if (n > 0) {
                const double sq = uniform ? 1.0 / (double)n : (double)deg_sq[k] / (D * D);
                const double S = 0.5 * (1.0 - sq);
                if (S > 0.0) z = S / (sqrt(Q / S) + (double)beta);
            }
            zeta[k] = z;
        }
    }
}

__global__ void __launch_bounds__(256) zeta_partial_kernel(const float* __restrict__ X, int ld, int F,
                                                           const int32_t* __restrict__ deg,
                                                           const RowSpan* __restrict__ chunks,
                                                           const int32_t* __restrict__ sub_off,
                                                           const int64_t* __restrict__ deg_sum, double* partial,
                                                           const int32_t* __restrict__ chunk_ptr,
                                                           const int64_t* __restrict__ deg_sq, float beta,
                                                           unsigned* counters, double* __restrict__ zeta,
                                                           double* __restrict__ q_acc, int phase) {
    // threads = 8 row lanes x 32 column lanes of one float4 each (as in the column sums above)
    __shared__ double sm[8][32][8];
    const RowSpan c = chunks[blockIdx.x];
    const bool uniform = deg_sum[c.k] == 0;
    const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
    const int ld4 = ld >> 2;
    const float4* x0 = reinterpret_cast<const float4*>(X + (long long)sub_off[c.k] * ld);
    double* P = partial + (long long)blockIdx.x * 2 * ld;
    for (int v0 = 0; v0 < ld4; v0 += 32) {
        const int v = v0 + cx;
        double a[4] = {0.0, 0.0, 0.0, 0.0}, b[4] = {0.0, 0.0, 0.0, 0.0};
        if (v < ld4) {
            const float4 sh = x0[v];
            const float4* g = reinterpret_cast<const float4*>(X + (long long)c.row0 * ld) + v;
            const int32_t* dg = deg + c.row0;
            int r = ry;
            for (; r + 8 < c.nrows; r += 16) {
                const float4 u0 = g[(long long)r * ld4], u1 = g[(long long)(r + 8) * ld4];
                const double w0 = uniform ? 1.0 : (double)dg[r], w1 = uniform ? 1.0 : (double)dg[r + 8];
                const double d0[4] = {(double)(u0.x - sh.x), (double)(u0.y - sh.y), (double)(u0.z - sh.z), (double)(u0.w - sh.w)};
                const double d1[4] = {(double)(u1.x - sh.x), (double)(u1.y - sh.y), (double)(u1.z - sh.z), (double)(u1.w - sh.w)};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    a[t] = fma(w0, d0[t], a[t]); b[t] = fma(w0 * d0[t], d0[t], b[t]);
                    a[t] = fma(w1, d1[t], a[t]); b[t] = fma(w1 * d1[t], d1[t], b[t]);
                }
            }
            for (; r < c.nrows; r += 8) {
                const float4 u0 = g[(long long)r * ld4];
                const double w0 = uniform ? 1.0 : (double)dg[r];
                const double d0[4] = {(double)(u0.x - sh.x), (double)(u0.y - sh.y), (double)(u0.z - sh.z), (double)(u0.w - sh.w)};
#pragma unroll
                for (int t = 0; t < 4; ++t) { a[t] = fma(w0, d0[t], a[t]); b[t] = fma(w0 * d0[t], d0[t], b[t]); }
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
                P[4 * v + t] = sa;
                P[ld + 4 * v + t] = sb;
            }
        }
        __syncthreads();
    }
    // the last CTA of this subgraph turns the chunk sums into zeta_k
    if (cta_arrive_last(counters + c.k, (unsigned)(chunk_ptr[c.k + 1] - chunk_ptr[c.k])))
        zeta_finalize(c.k, partial, F, ld, chunk_ptr, sub_off, deg_sum, deg_sq, beta, zeta, q_acc, phase);
}

// zeta[k] for every subgraph that has rows (the entry of an empty subgraph is left as it is: zero since creation).
cudaError_t launch_zeta(const float* X, int ld, int F, const int32_t* deg, const RowSpan* chunks, int nchunks,
                        const int32_t* chunk_ptr, const int32_t* sub_off, const int64_t* deg_sum, const int64_t* deg_sq,
                        float beta, double* partial, unsigned* counters, double* zeta, double* q_acc, int phase, cudaStream_t s) {
    if (nchunks > 0) {
        zeta_partial_kernel<<<(unsigned)nchunks, 256, 0, s>>>(X, ld, F, deg, chunks, sub_off, deg_sum, partial, chunk_ptr, deg_sq, beta,
                                                              counters, zeta, q_acc, phase);
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Consensus weights w_k = zeta_k / sum_j zeta_j (Section 3.4.2); 1/K for the plain average of Definition 3
// or when every zeta is zero.  Computed by each CTA for itself (K is small).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void consensus_weights(const double* __restrict__ zeta, int K, int weighted, float* w_sm) {
    __shared__ double total;
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int k = 0; k < K; ++k) t += zeta[k];
        total = t;
    }
    __syncthreads();
    for (int k = threadIdx.x; k < K; k += blockDim.x)
        w_sm[k] = (weighted && total > 0.0) ? (float)(zeta[k] / total) : 1.f / (float)K;
    __syncthreads();
}

// sum_k w_k (theta_k - lr grad_k) for the four parameters at float4 index i, k ascending.  The copies are read eight at a time,
// all sixteen loads of a batch issued before the first is used: with many copies of a small model (K = 64 copies of a
// 256-256 layer are 50 MB spread over 65 CTAs) the kernel is a chain of dependent loads otherwise.
__device__ __forceinline__ float4 weighted_sum(const float* __restrict__ params, const float* __restrict__ grads, long long pstride,
                                               long long i, int K, float lr, int with_sgd, const float* w_sm) {
    constexpr int B = 8;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k0 = 0; k0 < K; k0 += B) {
        float4 p[B], g[B];
#pragma unroll
        for (int t = 0; t < B; ++t) {
            const int k = min(k0 + t, K - 1);   // past the end: the last copy again, with weight 0 below
            p[t] = reinterpret_cast<const float4*>(params + (long long)k * pstride)[i];
            g[t] = with_sgd ? reinterpret_cast<const float4*>(grads + (long long)k * pstride)[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int t = 0; t < B; ++t) {
            if (k0 + t < K) {
                const float w = w_sm[k0 + t];
                float4 q = p[t];
                if (with_sgd) { q.x = fmaf(-lr, g[t].x, q.x); q.y = fmaf(-lr, g[t].y, q.y); q.z = fmaf(-lr, g[t].z, q.z); q.w = fmaf(-lr, g[t].w, q.w); }
                acc.x = fmaf(w, q.x, acc.x); acc.y = fmaf(w, q.y, acc.y); acc.z = fmaf(w, q.z, acc.z); acc.w = fmaf(w, q.w, acc.w);
            }
        }
    }
    return acc;
}

// theta_k <- theta_k - lr * grad_k (each replica's own step, update equation of Section 3.3), then
// theta_k <- sum_j w_j theta_j for every k (weighted global consensus, Section 3.4.2).  One float4 per thread.
__global__ void __launch_bounds__(256) sgd_consensus_kernel(float* __restrict__ params, const float* __restrict__ grads,
                                                            long long pstride, long long len4, int K, float lr,
                                                            const double* __restrict__ zeta, int weighted, int with_sgd,
                                                            const int32_t* __restrict__ err_word) {
    extern __shared__ float w_sm[];
    if (err_word && *err_word) return;   // a bounded wait ran out earlier in this epoch: keep the parameters as they are
    consensus_weights(zeta, K, weighted, w_sm);
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= len4) return;
    const float4 acc = weighted_sum(params, grads, pstride, i, K, lr, with_sgd, w_sm);
    for (int k = 0; k < K; ++k) reinterpret_cast<float4*>(params + (long long)k * pstride)[i] = acc;
}
cudaError_t launch_sgd_consensus(float* params, const float* grads, int64_t pstride, int64_t len, int K, float lr,
                                 const double* zeta, int weighted, int with_sgd, const int32_t* err_word, cudaStream_t s) {
    const long long len4 = len / 4;
    if (len4 > 0) {
        const int threads = len4 >= 148 * 256 * 4 ? 256 : 64;   // a small model is spread over more CTAs
        sgd_consensus_kernel<<<(unsigned)((len4 + threads - 1) / threads), threads, (size_t)K * sizeof(float), s>>>(params, grads, pstride, len4, K, lr,
                                                                                                   zeta, weighted, with_sgd, err_word); ++g_kernel_launches; }
    return cudaGetLastError();
}

// The same sum over the replicas of one context when the subgraphs are spread over several contexts:
//   out = sum_k w_k (theta_k - lr * grad_k),  w_k = zeta_k / total (weighted) or 1 / total,
// with `total` the sum over ALL contexts, so that the contexts' results add up to the consensus.  The parameters
// themselves are left alone; consensus_apply_kernel writes the finished sum to every replica.
__global__ void __launch_bounds__(256) consensus_partial_kernel(const float* __restrict__ params, const float* __restrict__ grads,
                                                                long long pstride, long long len4, int K, float lr,
                                                                const double* __restrict__ zeta, int weighted, int with_sgd,
                                                                double total, float* __restrict__ out, const int32_t* __restrict__ err_word) {
    extern __shared__ float w_sm[];
    if (err_word && *err_word) return;
    for (int k = threadIdx.x; k < K; k += blockDim.x) w_sm[k] = (float)((weighted ? zeta[k] : 1.0) / total);
    __syncthreads();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= len4) return;
    const float4 acc = weighted_sum(params, grads, pstride, i, K, lr, with_sgd, w_sm);
    reinterpret_cast<float4*>(out)[i] = acc;
}
__global__ void __launch_bounds__(256) consensus_apply_kernel(float* __restrict__ params, long long pstride, long long len4, int K,
                                                              const float* __restrict__ in, const int32_t* __restrict__ err_word) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= len4 || (err_word && *err_word)) return;
    const float4 v = reinterpret_cast<const float4*>(in)[i];
    for (int k = 0; k < K; ++k) reinterpret_cast<float4*>(params + (long long)k * pstride)[i] = v;
}
cudaError_t launch_consensus_partial(const float* params, const float* grads, int64_t pstride, int64_t len, int K, float lr,
                                     const double* zeta, int weighted, int with_sgd, double total, float* out, const int32_t* err_word, cudaStream_t s) {
    const long long len4 = len / 4;
    if (len4 > 0) {
        const int threads = len4 >= 148 * 256 * 4 ? 256 : 64;
        consensus_partial_kernel<<<(unsigned)((len4 + threads - 1) / threads), threads, (size_t)K * sizeof(float), s>>>(params, grads, pstride, len4, K, lr,
                                                                                                       zeta, weighted, with_sgd, total, out, err_word);
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}
cudaError_t launch_consensus_apply(float* params, int64_t pstride, int64_t len, int K, const float* in, const int32_t* err_word, cudaStream_t s) {
    const long long len4 = len / 4;
    if (len4 > 0) { consensus_apply_kernel<<<(unsigned)((len4 + 255) / 256), 256, 0, s>>>(params, pstride, len4, K, in, err_word); ++g_kernel_launches; }
    return cudaGetLastError();
}

__global__ void weights_kernel(const double* __restrict__ zeta, int K, int weighted, float* __restrict__ zeta_f,
                               float* __restrict__ w_f) {
    extern __shared__ float w_sm[];
    consensus_weights(zeta, K, weighted, w_sm);
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        zeta_f[k] = (float)zeta[k];
        w_f[k] = w_sm[k];
    }
}
cudaError_t launch_weights(const double* zeta, int K, int weighted, float* zeta_f, float* w_f, cudaStream_t s) {
    weights_kernel<<<1, 256, (size_t)K * sizeof(float), s>>>(zeta, K, weighted, zeta_f, w_f); ++g_kernel_launches;
    return cudaGetLastError();
}

__global__ void __launch_bounds__(256) relu_mask_kernel(float4* __restrict__ G, const float4* __restrict__ H, long long n4, float scale) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    float4 g = G[i];
    const float4 h = H[i];
    g.x = h.x > 0.f ? g.x * scale : 0.f; g.y = h.y > 0.f ? g.y * scale : 0.f;
    g.z = h.z > 0.f ? g.z * scale : 0.f; g.w = h.w > 0.f ? g.w * scale : 0.f;
    G[i] = g;
}
cudaError_t launch_relu_mask(float* G, const float* H, int ld, int64_t rows, float scale, cudaStream_t s) {
    const long long n4 = (long long)rows * (ld / 4);
    if (n4 > 0) {
        relu_mask_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, s>>>(reinterpret_cast<float4*>(G), reinterpret_cast<const float4*>(H), n4, scale);
        ++g_kernel_launches;
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Gathers between graph-node order and store-row order.
// ---------------------------------------------------------------------------------------------
__global__ void gather_rows_kernel(const float* __restrict__ Xg, int F, const int32_t* __restrict__ gid, long long Np,
                                   float* __restrict__ H0, int ld) {
    const long long row = blockIdx.x;
    const float* src = Xg + (long long)gid[row] * F;
    float* dst = H0 + row * ld;
    for (int j = threadIdx.x; j < ld; j += blockDim.x) dst[j] = j < F ? src[j] : 0.f;
}
cudaError_t launch_gather_rows(const float* Xg, int F, const int32_t* gid, int64_t Np, float* H0, int ld, cudaStream_t s) {
    if (Np > 0) { gather_rows_kernel<<<(unsigned)Np, 128, 0, s>>>(Xg, F, gid, Np, H0, ld); ++g_kernel_launches; }
    return cudaGetLastError();
}
__global__ void gather_labels_kernel(const int32_t* __restrict__ yg, const int32_t* __restrict__ gid, long long Np,
                                     int32_t* __restrict__ label) {
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < Np) label[r] = yg[gid[r]];
}
cudaError_t launch_gather_labels(const int32_t* yg, const int32_t* gid, int64_t Np, int32_t* label, cudaStream_t s) {
    if (Np > 0) { gather_labels_kernel<<<(unsigned)((Np + 255) / 256), 256, 0, s>>>(yg, gid, Np, label); ++g_kernel_launches; }
    return cudaGetLastError();
}
// Logits of the core rows back to graph-node order; one CTA per span of core rows.
__global__ void scatter_core_kernel(const float* __restrict__ logits, int ld, int C, const int32_t* __restrict__ gid,
                                    const RowSpan* __restrict__ spans, float* __restrict__ out) {
    const RowSpan sp = spans[blockIdx.x];
    for (long long i = threadIdx.x; i < (long long)sp.nrows * C; i += blockDim.x) {
        const long long r = sp.row0 + i / C;
        const int j = (int)(i % C);
        out[(long long)gid[r] * C + j] = logits[r * ld + j];
    }
}
cudaError_t launch_scatter_core(const float* logits, int ld, int C, const int32_t* gid, const RowSpan* core_spans, int nspans,
                                float* out, cudaStream_t s) {
    if (nspans > 0) { scatter_core_kernel<<<(unsigned)nspans, 256, 0, s>>>(logits, ld, C, gid, core_spans, out); ++g_kernel_launches; }
    return cudaGetLastError();
}

}  // namespace gad
