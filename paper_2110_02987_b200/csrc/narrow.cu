// Backward transforms of a layer with at most 16 output columns (a classifier layer: the paper's datasets have
// 3 .. 41 classes), on the FP32 ALUs:
//
//   dW_k^(l) = H^(l)^T dZ_l   and   dPre_(l-1) = (dZ_l W_k^(l)^T) masked by H^(l) > 0
//   (and db_k^(l-1), the column sums of the dPre_(l-1) rows it writes)
//
// in ONE pass over H^(l) and dZ_l (chain rule through the forward equation, Section 3.3).  With so few columns
// both products cost 2 * 16 flops per loaded value of H^(l), and the tensor-core kernels, whose M = 128 tile costs
// the same for any N, would read H^(l) twice for them.
//
// A CTA of four warps owns a run of rows of one subgraph (a chunk) and streams it through a three-stage ring in
// shared memory: one thread issues bulk asynchronous copies (cp.async.bulk, completion on an mbarrier) of the next
// row blocks of H^(l) and dZ_l while the warps work on the current one.  A lane owns four columns of H^(l) (a warp a
// slab of 128 columns, wider layers spread their slabs over the warps) and keeps its 4 x 16 blocks of W_k^(l) and of
// dW in registers for the whole chunk.  Chunk results of dW are added per subgraph in chunk
// order by reduce_chunks, so nothing depends on scheduling.  Every mbarrier wait is bounded: on a time-out the CTA
// raises the error word and returns.
#include <algorithm>

#include "gad_internal.h"

namespace gad {

namespace {

constexpr int kWarps = 4, kStages = 3;
constexpr uint32_t kWaitLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.b32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i)
        if (bar_try(bar, parity)) return true;
    return false;
}
// Contiguous global -> shared copy of `bytes` (a multiple of 16, both addresses 16-byte aligned).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// Rows per ring stage: a stage holds 4096 floats of H^(l) per 128-column slab set.
__host__ __device__ inline int block_rows(int nslab) { return 32 / nslab; }

struct Ring {
    uint32_t bar0;       // shared address of the first stage's mbarrier (8 bytes each)
    const float* A;      // H^(l) rows of the chunk
    const float* B;      // dZ_l rows of the chunk, or null
    int lda, ldb, nrows, BR;
    uint32_t a_addr, b_addr, stage_a_bytes, stage_b_bytes;
    __device__ __forceinline__ void issue(int b) const {
        const int s = b % kStages, nb = min(BR, nrows - b * BR);
        const uint32_t ab = (uint32_t)nb * (uint32_t)lda * 4u, bb = B ? (uint32_t)nb * (uint32_t)ldb * 4u : 0u;
        const uint32_t bar = bar0 + 8u * (uint32_t)s;
        bar_expect(bar, ab + bb);
        bulk_load(a_addr + s * stage_a_bytes, A + (long long)b * BR * lda, ab, bar);
        if (B) bulk_load(b_addr + s * stage_b_bytes, B + (long long)b * BR * ldb, bb, bar);
    }
};

// ---------------------------------------------------------------------------------------------
// backward: dW partial of the chunk, and dPre_(l-1) rows
// ---------------------------------------------------------------------------------------------
template <int NQ>
__global__ void __launch_bounds__(32 * kWarps, 3)
narrow_bwd_kernel(const float* __restrict__ H, int ldh, int fi, const float* __restrict__ dZ, int ldz, const float* __restrict__ params,
                  long long pstride, long long w_int, int ldw, const RowSpan* __restrict__ chunks, float scale, float* __restrict__ dPre,
                  float* __restrict__ partial, long long partial_stride, int nslab, int32_t* __restrict__ err) {
    constexpr int NP = 4 * NQ;
    extern __shared__ __align__(128) unsigned char narrow_smem[];
    __shared__ __align__(8) unsigned long long bars[kStages];
    const RowSpan ch = chunks[blockIdx.x];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int slab = warp % nslab, rg = warp / nslab, nrg = kWarps / nslab;
    const int ldh4 = ldh >> 2, col4 = 32 * slab + lane, col = 4 * col4;
    const bool live = col4 < ldh4;
    const int BR = block_rows(nslab);
    const int nblk = (ch.nrows + BR - 1) / BR;
    Ring ring;
    ring.A = H + (long long)ch.row0 * ldh; ring.B = dZ + (long long)ch.row0 * ldz;
    ring.lda = ldh; ring.ldb = ldz; ring.nrows = ch.nrows; ring.BR = BR;
    ring.stage_a_bytes = (uint32_t)BR * ldh * 4u; ring.stage_b_bytes = (uint32_t)BR * ldz * 4u;
    ring.a_addr = smem_addr(narrow_smem);
    ring.b_addr = ring.a_addr + kStages * ring.stage_a_bytes;
    ring.bar0 = smem_addr(&bars[0]);
    if (threadIdx.x == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) bar_init(ring.bar0 + 8u * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0)
        for (int b = 0; b < min(kStages, nblk); ++b) ring.issue(b);

    // this lane's block of W_k: rows col .. col+3, all NP columns, kept as pairs of neighbouring columns for the
    // two-wide FP32 multiply-add (one instruction, two IEEE fused multiply-adds)
    float2 Wp[4][NP / 2], accp[4][NP / 2];
    {
        const float* W = params + (long long)ch.k * pstride + w_int;
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const float4 t = (live && col + j < fi) ? __ldg(reinterpret_cast<const float4*>(W + (long long)(col + j) * ldw) + q)
                                                        : make_float4(0.f, 0.f, 0.f, 0.f);
                Wp[j][2 * q] = make_float2(t.x, t.y); Wp[j][2 * q + 1] = make_float2(t.z, t.w);
            }
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int m = 0; m < NP / 2; ++m) accp[j][m] = make_float2(0.f, 0.f);
    }
    float bsum[4] = {0.f, 0.f, 0.f, 0.f};   // column sums of the dPre rows this lane writes (the bias gradient of the layer below)
    const float4* As = reinterpret_cast<const float4*>(narrow_smem);
    const float4* Bs = reinterpret_cast<const float4*>(narrow_smem + kStages * ring.stage_a_bytes);
    const int a_stage4 = (int)(ring.stage_a_bytes >> 4), b_stage4 = (int)(ring.stage_b_bytes >> 4);
    for (int b = 0; b < nblk; ++b) {
        const int s = b % kStages;
        const bool ok = bar_wait(ring.bar0 + 8u * (uint32_t)s, (uint32_t)(b / kStages) & 1u);
        if (__syncthreads_or(!ok)) {   // a copy never arrived: report it and stop
            if (threadIdx.x == 0) {
                atomicExch(err, 90);
                // copies of later stages may still be on their way into this CTA's shared memory: give each a short,
                // bounded chance to land before the memory is released
                for (int s2 = 0; s2 < kStages; ++s2)
                    for (uint32_t i = 0; i < 4096u; ++i)
                        if (bar_try(ring.bar0 + 8u * (uint32_t)s2, 0u) || bar_try(ring.bar0 + 8u * (uint32_t)s2, 1u)) break;
            }
            return;
        }
        const int nb = min(BR, ch.nrows - b * BR);
        const float4* Ab = As + s * a_stage4;
        const float4* Bb = Bs + s * b_stage4;
#pragma unroll 2
        for (int r = rg; r < nb; r += nrg) {
            const float4 h4 = live ? Ab[r * ldh4 + col4] : make_float4(0.f, 0.f, 0.f, 0.f);
            float2 dzp[NP / 2];
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const float4 t = Bb[r * NQ + q];
                dzp[2 * q] = make_float2(t.x, t.y); dzp[2 * q + 1] = make_float2(t.z, t.w);
            }
            const float h[4] = {h4.x, h4.y, h4.z, h4.w};
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 hh = make_float2(h[j], h[j]);
                float2 v2 = make_float2(0.f, 0.f);   // even and odd columns of the dot product, added at the end
#pragma unroll
                for (int m = 0; m < NP / 2; ++m) {
                    v2 = __ffma2_rn(dzp[m], Wp[j][m], v2);
                    accp[j][m] = __ffma2_rn(hh, dzp[m], accp[j][m]);
                }
                v[j] = v2.x + v2.y;
            }
            if (live) {
                float4 o;
                o.x = h[0] > 0.f ? v[0] * scale : 0.f; o.y = h[1] > 0.f ? v[1] * scale : 0.f;
                o.z = h[2] > 0.f ? v[2] * scale : 0.f; o.w = h[3] > 0.f ? v[3] * scale : 0.f;
                reinterpret_cast<float4*>(dPre + (long long)(ch.row0 + b * BR + r) * ldh)[col4] = o;
                bsum[0] += o.x; bsum[1] += o.y; bsum[2] += o.z; bsum[3] += o.w;
            }
        }
        __syncthreads();   // the stage has been read by every warp
        if (threadIdx.x == 0 && b + kStages < nblk) ring.issue(b + kStages);
    }
    // dW of the chunk: the row groups of a slab added in order (through the ring's memory, now idle)
    float* red = reinterpret_cast<float*>(narrow_smem);   // [warp][4 * NP][32 lanes]
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int n = 0; n < NP; ++n) red[(warp * 4 * NP + j * NP + n) * 32 + lane] = (n & 1) ? accp[j][n / 2].y : accp[j][n / 2].x;
    float* redb = red + kWarps * 4 * NP * 32;             // [warp][4][32 lanes]
#pragma unroll
    for (int j = 0; j < 4; ++j) redb[(warp * 4 + j) * 32 + lane] = bsum[j];
    __syncthreads();
    // the chunk's result: [column sums of dPre (ldh)] [dW (fi x ldw)]
    float* outb = partial + (long long)blockIdx.x * partial_stride;
    float* out = outb + ldh;
    for (int e = threadIdx.x; e < nslab * 4 * NP * 32; e += 32 * kWarps) {
        const int sl = e / (4 * NP * 32), jn = (e / 32) % (4 * NP), ln = e & 31;
        float sum = 0.f;
        for (int g = 0; g < nrg; ++g) sum += red[((g * nslab + sl) * 4 * NP + jn) * 32 + ln];
        const int c = 128 * sl + 4 * ln + jn / NP, n = jn % NP;
        if (c < fi) out[(long long)c * ldw + n] = sum;
    }
    for (int e = threadIdx.x; e < nslab * 4 * 32; e += 32 * kWarps) {
        const int sl = e / 128, j = (e / 32) & 3, ln = e & 31;
        float sum = 0.f;
        for (int g = 0; g < nrg; ++g) sum += redb[((g * nslab + sl) * 4 + j) * 32 + ln];
        const int c = 128 * sl + 4 * ln + j;
        if (c < ldh) outb[c] = sum;
    }
}

}  // namespace

// At least three quarters of a warp's lanes must own columns (a lane owns four): narrower inputs stay on the tensor cores.
bool narrow_supported(int ldi, int ldo) { return ldo >= 4 && ldo <= 16 && ldi >= 96 && ldi <= 128 * kWarps; }

// Room for the ring beyond the default 48 KB, and the shared-memory share of the SM set for three resident CTAs; once
// per kernel (the instantiations share one function-pointer type, so they are told apart by address).
template <class Kernel>
static cudaError_t prepare(Kernel kernel) {
    return configure_kernel_once(reinterpret_cast<const void*>(kernel), 100 * 1024, true);
}

static int slabs_for(int ldi) { const int s = (ldi + 127) / 128; return s <= 1 ? 1 : (s <= 2 ? 2 : 4); }

cudaError_t launch_narrow_bwd(const float* H, int ldh, int fi, const float* dZ, int ldz, const float* params, int64_t pstride,
                              int64_t w_int, int ldw, const RowSpan* chunks, int nchunks, float scale, float* dPre, float* partial,
                              int64_t partial_stride, int32_t* err, cudaStream_t s) {
    if (nchunks <= 0) return cudaSuccess;
    const int nslab = slabs_for(ldh), BR = block_rows(nslab), nq = ldz / 4;
    size_t smem = (size_t)kStages * BR * (ldh + ldz) * 4;
    smem = std::max(smem, (size_t)kWarps * 4 * (ldz + 1) * 32 * 4);   // the exchange of the dW blocks and column sums at the end
    auto go = [&](auto kernel) -> cudaError_t {
        cudaError_t e = prepare(kernel);
        if (e != cudaSuccess) return e;
        kernel<<<(unsigned)nchunks, 32 * kWarps, smem, s>>>(H, ldh, fi, dZ, ldz, params, pstride, w_int, ldw, chunks, scale, dPre, partial,
                                                            partial_stride, nslab, err);
        ++g_kernel_launches;
        return cudaGetLastError();
    };
    switch (nq) {
        case 1: return go(narrow_bwd_kernel<1>);
        case 2: return go(narrow_bwd_kernel<2>);
        case 3: return go(narrow_bwd_kernel<3>);
        default: return go(narrow_bwd_kernel<4>);
    }
}

}  // namespace gad
