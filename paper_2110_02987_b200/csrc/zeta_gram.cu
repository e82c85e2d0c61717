// Variance-based importance in its literal pairwise form (Section 3.4.1, the printed equation read as it stands),
//   zeta_k = sum over unordered pairs i < j of subgraph k of  p_i p_j / (|x_i - x_j|_2 + beta),
// with the squared distances taken from a Gram matrix on the tensor cores:
//   |x_i - x_j|^2 = |x_i|^2 + |x_j|^2 - 2 x_i . x_j .
// The pairs of a subgraph are cut into tiles of 128 x 128 (i-block <= j-block).  A tile's inner products are one
// tcgen05 accumulator: both operand tiles are rows of the feature matrix (K-major, loaded by TMA with the 128-byte
// swizzle).  The features are split once per call into TF32-exact hi and lo = x - hi copies (a streaming kernel that
// also takes the squared norms), and the product is accumulated as hi.hi + hi.lo + lo.hi in fp32 in tensor memory -
// the error-compensated product of the layer transforms, here with both operands split ahead of time because the
// drain below needs the SM's issue slots.  While the MMA warp fills the second accumulator, sixteen warps read the
// first one back (tcgen05.ld), turn every inner product into a distance and add p_j / (d + beta) over the pairs
// i < j inside the subgraph (approximate square root and reciprocal, relative error 2^-23 each: far inside the
// 2e-6 the result is held to, and the errors of different pairs do not add up coherently).
//
// Cancellation: for two rows that are close compared with their norms the Gram form loses digits, so a pair whose
// squared distance comes out below 5 % of |x_i|^2 + |x_j|^2 is recomputed from the differences x_if - x_jf
// themselves (plain loads, FP32 ALU).  On generic features that never happens; on features that are all alike it is
// every pair, which then costs what the FP32 tile kernel of zeta_pair.cu costs.
//
// Order of the sum: persistent CTAs take the tiles t = blockIdx.x, blockIdx.x + gridDim.x, ... (ascending, subgraph
// by subgraph); every draining warp keeps one fp64 running sum per subgraph and writes it to its own slot; a second
// kernel adds the slots in slot order.  For a given number of CTAs the result does not depend on scheduling.
#include "gad_internal.h"
#include "tc_common.cuh"

namespace gad {

namespace {

constexpr int GT = 128;                                   // rows of a tile side (M and N of the MMA)
constexpr int GBK = 32;                                   // features per ring stage
constexpr int G_TILE_BYTES = GT * GBK * 4;                // 16 KiB
constexpr int G_STAGE_BYTES = 4 * G_TILE_BYTES;           // A_hi | A_lo | B_hi | B_lo
constexpr int G_STAGES = 3;
constexpr int G_RING_BYTES = G_STAGES * G_STAGE_BYTES;
constexpr int G_EPI_WARPS = 16;                           // four per quarter of the tensor-memory lanes, one block of 32 columns each
constexpr int G_EPI_WARP0 = 2;
constexpr int G_THREADS = 32 * (G_EPI_WARP0 + G_EPI_WARPS);
constexpr int G_COL_BYTES = G_EPI_WARPS * 32 * 8;         // per draining warp: (p_j, |x_j|^2) of its 32 columns
constexpr int G_SMEM_BYTES = G_RING_BYTES + 1024 + 256 + G_COL_BYTES;
constexpr int G_TMEM_COLS = 2 * GT;                       // two accumulators of 128 columns

struct GramArgs {
    const float* X;            // [rows x ld] features in store-row order
    int ld, F;
    const float* norm2;        // [rows] squared norms of the rows
    const int32_t* deg;
    const int32_t* sub_off;
    const int64_t* deg_sum;
    const int64_t* tile_ptr;   // [K+1] first tile of every subgraph
    int K;
    long long ntiles;
    float beta;
    double* partial;           // [gridDim.x][G_EPI_WARPS][K]
    int32_t* err;
};

struct TilePos { int k, r0, n, i0, j0; };

// Tile t of the list: subgraph k (largest k with tile_ptr[k] <= t), then (bi, bj), bi <= bj, from the position inside
// the row-major list of the upper triangle of T x T blocks.
__device__ __forceinline__ TilePos tile_pos(const GramArgs& a, long long t) {
    int lo = 0, hi = a.K;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (a.tile_ptr[mid] <= t) lo = mid; else hi = mid;
    }
    TilePos p;
    p.k = lo;
    p.r0 = a.sub_off[lo];
    p.n = a.sub_off[lo + 1] - p.r0;
    const long long T = (p.n + GT - 1) / GT;
    const long long q = t - a.tile_ptr[lo];
    long long bi = (long long)(((double)(2 * T + 1) - sqrt((double)(2 * T + 1) * (double)(2 * T + 1) - 8.0 * (double)q)) * 0.5);
    bi = max(0ll, min(bi, T - 1));
    while (bi > 0 && bi * T - bi * (bi - 1) / 2 > q) --bi;                      // rows before bi hold bi T - bi (bi - 1) / 2 tiles
    while (bi + 1 < T && (bi + 1) * T - (bi + 1) * bi / 2 <= q) ++bi;
    const long long bj = bi + (q - (bi * T - bi * (bi - 1) / 2));
    p.i0 = (int)bi * GT;
    p.j0 = (int)bj * GT;
    return p;
}

__device__ __forceinline__ float sqrt_approx(float x) {
    float y;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(G_THREADS, 1)
zeta_gram_kernel(const __grid_constant__ CUtensorMap tmHi, const __grid_constant__ CUtensorMap tmLo, const GramArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* sm = smem_raw + pad;                 // 1024-byte aligned: the 128B swizzle pattern repeats every 1024 bytes
    const uint32_t sm_addr = raw_addr + pad;
    const uint32_t bars = sm_addr + G_RING_BYTES;
    auto full = [&](int s) { return bars + 8u * s; };
    auto empty = [&](int s) { return bars + 8u * (G_STAGES + s); };
    auto tfull = [&](int i) { return bars + 8u * (2 * G_STAGES + i); };
    auto tempty = [&](int i) { return bars + 8u * (2 * G_STAGES + 2 + i); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + G_RING_BYTES + 8 * (2 * G_STAGES + 4));
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float2* col_sm = reinterpret_cast<float2*>(sm + G_RING_BYTES + 256);   // [G_EPI_WARPS][32]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < G_STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(tfull(i), 1); mbar_init(tempty(i), G_EPI_WARPS); }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(G_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    const int nkb = (a.F + GBK - 1) / GBK;

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer: hi and lo of the two row blocks of the tile, 32 features at a time ----------------
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (long long t = blockIdx.x; t < a.ntiles && ok; t += gridDim.x) {
            const TilePos p = tile_pos(a, t);
            for (int kb = 0; kb < nkb; ++kb) {
                if (!(ok = mbar_wait(empty(stage), phase ^ 1u, abort_flag, a.err, 21))) break;
                mbar_expect_tx(full(stage), 4u * G_TILE_BYTES);
                const uint32_t base = sm_addr + stage * G_STAGE_BYTES;
                tma_load_2d(base, &tmHi, kb * GBK, p.r0 + p.i0, full(stage));
                tma_load_2d(base + G_TILE_BYTES, &tmLo, kb * GBK, p.r0 + p.i0, full(stage));
                tma_load_2d(base + 2 * G_TILE_BYTES, &tmHi, kb * GBK, p.r0 + p.j0, full(stage));
                tma_load_2d(base + 3 * G_TILE_BYTES, &tmLo, kb * GBK, p.r0 + p.j0, full(stage));
                if (++stage == G_STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer ----------------
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        const uint32_t idesc = instr_desc(GT);
        bool ok = true;
        for (long long t = blockIdx.x; t < a.ntiles && ok; t += gridDim.x) {
            if (!(ok = mbar_wait(tempty(acc), acc_phase ^ 1u, abort_flag, a.err, 22))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t d = tmem_base + (uint32_t)(acc * GT);
            for (int kb = 0; kb < nkb; ++kb) {
                if (!(ok = mbar_wait(full(stage), phase, abort_flag, a.err, 23))) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t base = sm_addr + stage * G_STAGE_BYTES;
                const uint64_t a_hi = smem_desc(base), a_lo = smem_desc(base + G_TILE_BYTES);
                const uint64_t b_hi = smem_desc(base + 2 * G_TILE_BYTES), b_lo = smem_desc(base + 3 * G_TILE_BYTES);
                const int nks = min(GBK / 8, (a.F - kb * GBK + 7) / 8);
                if (nks == GBK / 8) {
#pragma unroll
                    for (int ks = 0; ks < GBK / 8; ++ks) {           // 8 TF32 values = 32 bytes = 2 descriptor units along K
                        mma_tf32(d, a_hi + 2 * ks, b_hi + 2 * ks, idesc, ks == 0 ? (kb != 0 ? 1u : 0u) : 1u);
                        mma_tf32(d, a_hi + 2 * ks, b_lo + 2 * ks, idesc, 1u);
                        mma_tf32(d, a_lo + 2 * ks, b_hi + 2 * ks, idesc, 1u);
                    }
                } else {
                    for (int ks = 0; ks < nks; ++ks) {
                        const uint64_t adv = (uint64_t)(2 * ks);
                        mma_tf32(d, a_hi + adv, b_hi + adv, idesc, (kb | ks) != 0 ? 1u : 0u);
                        mma_tf32(d, a_hi + adv, b_lo + adv, idesc, 1u);
                        mma_tf32(d, a_lo + adv, b_hi + adv, idesc, 1u);
                    }
                }
                mma_commit(empty(stage));
                if (++stage == G_STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            mma_commit(tfull(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    } else if (warp >= G_EPI_WARP0) {
        // ---------------- drain: inner products -> distances -> weighted sum over the pairs i < j ----------------
        // this warp may read tensor-memory lanes 32q .. 32q+31 (tile rows i); of the four warps of a quarter each takes
        // one block of 32 columns (tile columns j)
        const int ew = warp - G_EPI_WARP0, q = warp & 3, c0 = 32 * (ew >> 2);
        float2* cols = col_sm + ew * 32;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        double sum = 0.0;
        int cur_k = -1;
        double* slot = a.partial + ((long long)blockIdx.x * G_EPI_WARPS + ew) * a.K;
        auto flush = [&]() {
            if (cur_k < 0) return;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) slot[cur_k] = sum;
            sum = 0.0;
        };
        for (long long t = blockIdx.x; t < a.ntiles && ok; t += gridDim.x) {
            const TilePos p = tile_pos(a, t);
            if (p.k != cur_k) { flush(); cur_k = p.k; }
            const bool uniform = a.deg_sum[p.k] == 0;
            const float invD = (float)(1.0 / (uniform ? (double)p.n : (double)a.deg_sum[p.k]));
            const int i = p.i0 + q * 32 + lane;                       // this thread's row of the tile, inside the subgraph
            const bool iv = i < p.n;
            const float pi = iv ? (uniform ? 1.f : (float)a.deg[p.r0 + i]) * invD : 0.f;
            const float ni = iv ? a.norm2[p.r0 + i] : 0.f;
            {
                const int jl = p.j0 + c0 + lane;                      // the column this lane looks up for the warp
                const bool jlv = jl < p.n;
                __syncwarp();                                         // the previous tile's columns have been read
                cols[lane] = make_float2(jlv ? (uniform ? 1.f : (float)a.deg[p.r0 + jl]) * invD : 0.f, jlv ? a.norm2[p.r0 + jl] : 0.f);
                __syncwarp();
            }
            if (!(ok = __all_sync(0xffffffffu, mbar_wait(tfull(acc), acc_phase, abort_flag, a.err, 26)))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t v[32];
            tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * GT + c0), v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            // the accumulator block is in registers: hand the accumulator back before the arithmetic
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }

            // every pair of the block counts (a tile off the diagonal and wholly inside the subgraph), or each is tested
            const bool whole = p.i0 != p.j0 && p.i0 + GT <= p.n && p.j0 + GT <= p.n;
            float part = 0.f;
            bool close = false;
            if (whole) {
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) {
                    const float2 c = cols[jj];                         // (p_j, |x_j|^2), one broadcast load
                    const float s2 = ni + c.y;
                    const float d2 = fmaf(-2.f, __uint_as_float(v[jj]), s2);
                    close |= d2 < 0.05f * s2;
                    part = fmaf(c.x, rcp_approx(sqrt_approx(fmaxf(d2, 0.f)) + a.beta), part);
                }
            } else {
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) {
                    const float2 c = cols[jj];
                    const int j = p.j0 + c0 + jj;
                    const bool valid = iv && j < p.n && i < j;
                    const float s2 = ni + c.y;
                    const float d2 = fmaf(-2.f, __uint_as_float(v[jj]), s2);
                    close |= valid && d2 < 0.05f * s2;
                    const float term = c.x * rcp_approx(sqrt_approx(fmaxf(d2, 0.f)) + a.beta);
                    part += valid ? term : 0.f;
                }
            }
            if (__any_sync(0xffffffffu, close)) {
                // rows close to each other compared with their norms: those pairs again, from the differences themselves
                const float4* xi = reinterpret_cast<const float4*>(a.X + (long long)(p.r0 + min(i, p.n - 1)) * a.ld);
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) {                      // (unrolled: the accumulator block stays in registers)
                    const float2 c = cols[jj];
                    const int j = p.j0 + c0 + jj;
                    const bool valid = iv && j < p.n && i < j;
                    const float s2 = ni + c.y;
                    const float d2 = fmaf(-2.f, __uint_as_float(v[jj]), s2);
                    if (valid && d2 < 0.05f * s2) {
                        const float4* xj = reinterpret_cast<const float4*>(a.X + (long long)(p.r0 + j) * a.ld);
                        float s = 0.f;
                        for (int f4 = 0; f4 < (a.ld >> 2); ++f4) {       // pad columns are zero
                            const float4 u = __ldg(xi + f4), w = __ldg(xj + f4);
                            const float dx = u.x - w.x, dy = u.y - w.y, dz = u.z - w.z, dw = u.w - w.w;
                            s = fmaf(dx, dx, s); s = fmaf(dy, dy, s); s = fmaf(dz, dz, s); s = fmaf(dw, dw, s);
                        }
                        part += c.x / (sqrtf(s) + a.beta) - c.x * rcp_approx(sqrt_approx(fmaxf(d2, 0.f)) + a.beta);
                    }
                }
            }
            sum += (double)(pi * part);
        }
        if (ok) flush();
    }

    // Tear-down.  After a time-out, give loads that may still be in flight a bounded chance to land before the
    // shared memory is released.
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0)
        for (int s = 0; s < G_STAGES; ++s)
            for (uint32_t i = 0; i < 4096u; ++i)
                if (mbar_try_wait(full(s), 0) || mbar_try_wait(full(s), 1)) break;
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(G_TMEM_COLS) : "memory");
    }
}

// One pass over the features: hi = x rounded to TF32, lo = x - hi (rounded the same way), and |x_r|^2 in fp32.  One warp
// per row (pad columns are zero and stay zero).
__global__ void __launch_bounds__(256) split_rows_kernel(const float* __restrict__ X, int ld, long long rows, float* __restrict__ Xhi,
                                                         float* __restrict__ Xlo, float* __restrict__ norm2) {
    const long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    const float4* x = reinterpret_cast<const float4*>(X + r * ld);
    float4* xh = reinterpret_cast<float4*>(Xhi + r * ld);
    float4* xl = reinterpret_cast<float4*>(Xlo + r * ld);
    float s = 0.f;
    for (int f4 = lane; f4 < (ld >> 2); f4 += 32) {
        const float4 v = __ldg(x + f4);
        s = fmaf(v.x, v.x, s); s = fmaf(v.y, v.y, s); s = fmaf(v.z, v.z, s); s = fmaf(v.w, v.w, s);
        float4 h, l;
        h.x = tf32_hi(v.x); l.x = tf32_round(v.x - h.x);
        h.y = tf32_hi(v.y); l.y = tf32_round(v.y - h.y);
        h.z = tf32_hi(v.z); l.z = tf32_round(v.z - h.z);
        h.w = tf32_hi(v.w); l.w = tf32_round(v.w - h.w);
        xh[f4] = h;
        xl[f4] = l;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) norm2[r] = s;
}

// zeta_k = the slots of subgraph k added in slot order (one warp per subgraph).
__global__ void zeta_gram_finish_kernel(const double* __restrict__ partial, int nslots, int K, double* __restrict__ zeta) {
    const int k = blockIdx.x, lane = threadIdx.x;
    double s = 0.0;
    for (int i = lane; i < nslots; i += 32) s += partial[(long long)i * K + k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) zeta[k] = s;
}

}  // namespace

// Tiles of a subgraph of `rows` rows: T (T + 1) / 2 with T = ceil(rows / 128).
int64_t zeta_gram_tiles(int64_t rows) {
    const int64_t T = (rows + GT - 1) / GT;
    return T * (T + 1) / 2;
}
int64_t zeta_gram_partials(int num_sms, int K) { return (int64_t)num_sms * G_EPI_WARPS * K; }

cudaError_t launch_zeta_gram(const void* mapHi, const void* mapLo, const float* X, int ld, int F, long long rows, const int32_t* deg,
                             const int32_t* sub_off, const int64_t* deg_sum, const int64_t* tile_ptr, int64_t ntiles, int K, float beta,
                             float* Xhi, float* Xlo, float* norm2, double* partial, double* zeta, int32_t* err, int num_sms, cudaStream_t s) {
    if (rows <= 0 || K <= 0) return cudaSuccess;
    cudaError_t e = configure_kernel_once(reinterpret_cast<const void*>(zeta_gram_kernel), G_SMEM_BYTES, false);
    if (e != cudaSuccess) return e;
    split_rows_kernel<<<(unsigned)((rows * 32 + 255) / 256), 256, 0, s>>>(X, ld, rows, Xhi, Xlo, norm2);
    ++g_kernel_launches;
    e = cudaMemsetAsync(partial, 0, sizeof(double) * (size_t)zeta_gram_partials(num_sms, K), s);
    if (e != cudaSuccess) return e;
    if (ntiles > 0) {
        GramArgs a;
        a.X = X; a.ld = ld; a.F = F; a.norm2 = norm2; a.deg = deg; a.sub_off = sub_off; a.deg_sum = deg_sum; a.tile_ptr = tile_ptr;
        a.K = K; a.ntiles = ntiles; a.beta = beta; a.partial = partial; a.err = err;
        const unsigned grid = (unsigned)(ntiles < num_sms ? ntiles : num_sms);
        zeta_gram_kernel<<<grid, G_THREADS, G_SMEM_BYTES, s>>>(*reinterpret_cast<const CUtensorMap*>(mapHi),
                                                               *reinterpret_cast<const CUtensorMap*>(mapLo), a);
        ++g_kernel_launches;
    }
    zeta_gram_finish_kernel<<<(unsigned)K, 32, 0, s>>>(partial, num_sms * G_EPI_WARPS, K, zeta);
    ++g_kernel_launches;
    return cudaGetLastError();
}

}  // namespace gad
