// Grouped dense transforms on the FP32 ALUs: the always-correct fp32 path of
//   Z_l   = H^(l) W_k^(l)                       (the H.W of the forward equation, Section 3.3)
//   dPre  = (dZ_l W_k^(l)^T) masked by H^(l)>0  (chain rule through the forward equation)
//   dW_k  = H^(l)_k^T dZ_l,k                    (weight gradient, Section 3.3)
// "Grouped": every row tile / row chunk belongs to exactly one subgraph k and uses that replica's W_k.
// All matrices keep zero-filled pad columns up to their leading dimension, so 16-byte loads never need a
// column guard beyond "below the leading dimension".
#include "epilogue.cuh"
#include "gad_internal.h"

namespace gad {

// ---------------------------------------------------------------------------------------------
// C[rows x N] = A[rows x Kd] * B, rows tiled by RowSpan.  MODE 0: B[kd][n] = W[kd*ldw + n];
// MODE 1: B[kd][n] = W[n*ldw + kd] and the result is masked / scaled.  MODE 2: as MODE 0, followed by bias, ReLU and
// dropout (a layer that aggregates first finishes in its transform).
// ---------------------------------------------------------------------------------------------
template <int BM, int BN, int BK, int TM, int TN, int MODE>
__global__ void __launch_bounds__((BM / TM) * (BN / TN))
gemm_rows_kernel(const float* __restrict__ A, int lda, int Kd, const float* __restrict__ params, long long pstride,
                 long long w_int, int ldw, int N, float* __restrict__ C, int ldc, const RowSpan* __restrict__ tiles,
                 const float* __restrict__ Hmask, int ldh, float scale, ActEpi act) {
    constexpr int NT = (BM / TM) * (BN / TN);
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const RowSpan t = tiles[blockIdx.x];
    const int n0 = blockIdx.y * BN;
    const float* W = params + (long long)t.k * pstride + w_int;
    const int tid = threadIdx.x;
    const int tx = tid % (BN / TN), ty = tid / (BN / TN);
    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    const int Kpad = (Kd + 3) & ~3;
    for (int k0 = 0; k0 < Kpad; k0 += BK) {
        // A tile: BM rows x BK columns, read as float4 along k, stored transposed
        for (int i = tid; i < BM * (BK / 4); i += NT) {
            int r = i / (BK / 4), kq = (i % (BK / 4)) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < t.nrows && k0 + kq < lda) v = *reinterpret_cast<const float4*>(A + (long long)(t.row0 + r) * lda + k0 + kq);
            As[kq + 0][r] = v.x; As[kq + 1][r] = v.y; As[kq + 2][r] = v.z; As[kq + 3][r] = v.w;
        }
        if (MODE != 1) {
            for (int i = tid; i < BK * (BN / 4); i += NT) {
                int kk = i / (BN / 4), nq = (i % (BN / 4)) * 4;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (k0 + kk < Kd && n0 + nq < ldw) v = *reinterpret_cast<const float4*>(W + (long long)(k0 + kk) * ldw + n0 + nq);
                *reinterpret_cast<float4*>(&Bs[kk][nq]) = v;
            }
        } else {
            for (int i = tid; i < BN * (BK / 4); i += NT) {
                int n = i / (BK / 4), kq = (i % (BK / 4)) * 4;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (n0 + n < N && k0 + kq < ldw) v = *reinterpret_cast<const float4*>(W + (long long)(n0 + n) * ldw + k0 + kq);
                Bs[kq + 0][n] = v.x; Bs[kq + 1][n] = v.y; Bs[kq + 2][n] = v.z; Bs[kq + 3][n] = v.w;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
#pragma unroll
            for (int i = 0; i < TM; i += 4) *reinterpret_cast<float4*>(&a[i]) = *reinterpret_cast<const float4*>(&As[kk][ty * TM + i]);
#pragma unroll
            for (int j = 0; j < TN; j += 4) *reinterpret_cast<float4*>(&b[j]) = *reinterpret_cast<const float4*>(&Bs[kk][tx * TN + j]);
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        int r = ty * TM + i;
        if (r >= t.nrows) continue;
        long long row = t.row0 + r;
#pragma unroll
        for (int j = 0; j < TN; j += 4) {
            int n = n0 + tx * TN + j;
            if (n >= ldc) continue;
            float4 v = make_float4(acc[i][j], acc[i][j + 1], acc[i][j + 2], acc[i][j + 3]);
            if (MODE == 1 && Hmask) {   // without a mask: plain A W^T
                float4 h = *reinterpret_cast<const float4*>(Hmask + row * ldh + n);
                v.x = h.x > 0.f ? v.x * scale : 0.f;
                v.y = h.y > 0.f ? v.y * scale : 0.f;
                v.z = h.z > 0.f ? v.z * scale : 0.f;
                v.w = h.w > 0.f ? v.w * scale : 0.f;
            }
            if (MODE == 2) v = apply_act(v, act, t.k, row, n);
            *reinterpret_cast<float4*>(C + row * ldc + n) = v;
        }
    }
}

template <int BM, int BN, int BK, int TM, int TN>
static cudaError_t launch_rows_cfg(int mode, const float* A, int lda, int Kd, const float* params, int64_t pstride,
                                   int64_t w_int, int ldw, int N, float* C, int ldc, const RowSpan* tiles, int ntiles,
                                   const float* Hmask, int ldh, float scale, const ActEpi* act, cudaStream_t s) {
    dim3 grid((unsigned)ntiles, (unsigned)((ldc + BN - 1) / BN));
    constexpr int NT = (BM / TM) * (BN / TN);
    const ActEpi none{};
    if (mode == 0)
        gemm_rows_kernel<BM, BN, BK, TM, TN, 0><<<grid, NT, 0, s>>>(A, lda, Kd, params, pstride, w_int, ldw, N, C, ldc, tiles,
                                                                    Hmask, ldh, scale, none);
    else if (mode == 1)
        gemm_rows_kernel<BM, BN, BK, TM, TN, 1><<<grid, NT, 0, s>>>(A, lda, Kd, params, pstride, w_int, ldw, N, C, ldc, tiles,
                                                                    Hmask, ldh, scale, none);
    else
        gemm_rows_kernel<BM, BN, BK, TM, TN, 2><<<grid, NT, 0, s>>>(A, lda, Kd, params, pstride, w_int, ldw, N, C, ldc, tiles,
                                                                    Hmask, ldh, scale, *act);
    ++g_kernel_launches;
    return cudaGetLastError();
}

// Row tiles hold at most 128 rows (the tile table is built with that height).
cudaError_t launch_gemm_rows_simt(int mode, const float* A, int lda, int Kd, const float* params, int64_t pstride,
                                  int64_t w_int, int ldw, int N, float* C, int ldc, const RowSpan* tiles, int ntiles,
                                  const float* Hmask, int ldh, float scale, const ActEpi* act, cudaStream_t s) {
    if (ntiles <= 0) return cudaSuccess;
    if (mode == 2 && !act) return cudaErrorInvalidValue;
    if (ldc > 64)
        return launch_rows_cfg<128, 128, 16, 8, 8>(mode, A, lda, Kd, params, pstride, w_int, ldw, N, C, ldc, tiles, ntiles, Hmask, ldh, scale, act, s);
    if (ldc > 32)
        return launch_rows_cfg<128, 64, 16, 8, 4>(mode, A, lda, Kd, params, pstride, w_int, ldw, N, C, ldc, tiles, ntiles, Hmask, ldh, scale, act, s);
    return launch_rows_cfg<128, 32, 16, 4, 4>(mode, A, lda, Kd, params, pstride, w_int, ldw, N, C, ldc, tiles, ntiles, Hmask, ldh, scale, act, s);
}

// ---------------------------------------------------------------------------------------------
// partial[chunk][m*ldw + n] = sum over the chunk's rows r of H[r][m] * dZ[r][n]
// ---------------------------------------------------------------------------------------------
template <int BM, int BN, int BK, int TM, int TN>
__global__ void __launch_bounds__((BM / TM) * (BN / TN))
gemm_tn_kernel(const float* __restrict__ H, int ldh, int M, const float* __restrict__ dZ, int ldz, int N,
               const RowSpan* __restrict__ chunks, float* __restrict__ partial, long long pstride_chunk, int ldw, int ntn) {
    constexpr int NT = (BM / TM) * (BN / TN);
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const RowSpan c = chunks[blockIdx.y];
    const int m0 = (blockIdx.x / ntn) * BM, n0 = (blockIdx.x % ntn) * BN;
    const int tid = threadIdx.x;
    const int tx = tid % (BN / TN), ty = tid / (BN / TN);
    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < c.nrows; k0 += BK) {
        for (int i = tid; i < BK * (BM / 4); i += NT) {
            int kk = i / (BM / 4), mq = (i % (BM / 4)) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + kk < c.nrows && m0 + mq < ldh) v = *reinterpret_cast<const float4*>(H + (long long)(c.row0 + k0 + kk) * ldh + m0 + mq);
            *reinterpret_cast<float4*>(&As[kk][mq]) = v;
        }
        for (int i = tid; i < BK * (BN / 4); i += NT) {
            int kk = i / (BN / 4), nq = (i % (BN / 4)) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + kk < c.nrows && n0 + nq < ldz) v = *reinterpret_cast<const float4*>(dZ + (long long)(c.row0 + k0 + kk) * ldz + n0 + nq);
            *reinterpret_cast<float4*>(&Bs[kk][nq]) = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
#pragma unroll
            for (int i = 0; i < TM; i += 4) *reinterpret_cast<float4*>(&a[i]) = *reinterpret_cast<const float4*>(&As[kk][ty * TM + i]);
#pragma unroll
            for (int j = 0; j < TN; j += 4) *reinterpret_cast<float4*>(&b[j]) = *reinterpret_cast<const float4*>(&Bs[kk][tx * TN + j]);
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* P = partial + (long long)blockIdx.y * pstride_chunk;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        int m = m0 + ty * TM + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < TN; j += 4) {
            int n = n0 + tx * TN + j;
            if (n >= ldw) continue;
            *reinterpret_cast<float4*>(P + (long long)m * ldw + n) = make_float4(acc[i][j], acc[i][j + 1], acc[i][j + 2], acc[i][j + 3]);
        }
    }
}

cudaError_t launch_gemm_tn_simt(const float* H, int ldh, int M, const float* dZ, int ldz, int N, const RowSpan* chunks,
                                int nchunks, float* partial, int ldw, cudaStream_t s) {
    if (nchunks <= 0) return cudaSuccess;
    const long long pstride_chunk = (long long)M * ldw;
    if (ldw > 32) {
        constexpr int BM = 128, BN = 64;
        int ntm = (M + BM - 1) / BM, ntn = (ldw + BN - 1) / BN;
        gemm_tn_kernel<BM, BN, 16, 8, 4><<<dim3((unsigned)(ntm * ntn), (unsigned)nchunks), 256, 0, s>>>(H, ldh, M, dZ, ldz, N, chunks, partial,
                                                                                                     pstride_chunk, ldw, ntn); ++g_kernel_launches;
    } else {
        constexpr int BM = 128, BN = 32;
        int ntm = (M + BM - 1) / BM, ntn = (ldw + BN - 1) / BN;
        gemm_tn_kernel<BM, BN, 16, 4, 4><<<dim3((unsigned)(ntm * ntn), (unsigned)nchunks), 256, 0, s>>>(H, ldh, M, dZ, ldz, N, chunks, partial,
                                                                                                     pstride_chunk, ldw, ntn); ++g_kernel_launches;
    }
    return cudaGetLastError();
}

}  // namespace gad
