// Grouped dense transforms on the 5th-generation tensor cores (tcgen05, accumulators in tensor memory):
//   mode 0   Z_l  = H^(l) W_k^(l)                        (the H.W of the forward equation, Section 3.3)
//   mode 1   dPre = (dZ_l W_k^(l)^T) masked by H^(l) > 0  (chain rule through the forward equation)
//   mode 2   H^(l+1) = sigma((A~ H^(l)) W_k^(l) + b_k^(l)) with dropout: mode 0 finished in the epilogue, for a layer
//            that aggregates before it transforms
// Both are C[rows x N] = A[rows x Kd] * B_k^T with A row-major (Kd contiguous) and B_k stored as N rows of Kd
// contiguous values, i.e. both operands K-major.  Row tiles never cross a subgraph, so a tile uses one replica's B.
//
// fp32 accuracy from TF32 tensor cores: every operand value x is split into hi, a value with a 10-bit mantissa
// (exactly representable in TF32), and lo = x - hi rounded to TF32, and the product is accumulated as
// A_hi B_hi + A_hi B_lo + A_lo B_hi in fp32 (the dropped A_lo B_lo term and the rounding of lo are ~2^-20 relative).  B is split once per
// epoch by a small kernel (hi = x rounded).  For A the tile as loaded is its own hi part, because the tensor core
// ignores the low 13 mantissa bits of an fp32 operand (hi = x truncated); eight warps of the GEMM kernel write only
// the lo tile beside it.  With passes = 1 only A B is issued on the unsplit operands (TF32 operand precision).
//
// One persistent CTA per SM, 18 warps: warp 0 issues TMA loads (128B-swizzled tiles) through a 3-stage ring,
// warps 2-9 split the A tile, warp 1 issues tcgen05.mma, warps 10-17 drain the accumulator (tcgen05.ld, two warps
// per quarter of the tensor-memory lanes) while the MMA warp already fills the second accumulator.  Every mbarrier wait is bounded: on a time-out the CTA
// raises an error word, stops, frees its tensor memory and returns.
#include <cuda.h>

#include "epilogue.cuh"
#include "gad_internal.h"
#include "tc_common.cuh"

namespace gad {

namespace {

constexpr int BK = 32, STAGES = 3, BN_MAX = 128;
constexpr int A_BYTES = BM * BK * 4;                      // 16 KiB
constexpr int B_BYTES = BN_MAX * BK * 4;                  // 16 KiB
constexpr int STAGE_BYTES = 2 * A_BYTES + 2 * B_BYTES;    // A_hi | A_lo | B_hi | B_lo
constexpr int RING_BYTES = STAGES * STAGE_BYTES;           // the rows kernel cuts this into 3 .. 6 stages
constexpr int MAX_STAGES = 6;
constexpr int SMEM_BYTES = RING_BYTES + 1024 + 256;
constexpr int EPI_WARPS = 8;                              // two per quarter of the tensor-memory lanes
constexpr int EPI_BYTES = EPI_WARPS * 32 * 33 * 4;        // per-warp transpose tiles of the epilogue
constexpr int SPLIT_WARPS = 8;                            // warps that split the A tile
constexpr int EPI_WARP0 = 2 + SPLIT_WARPS;                // first epilogue warp (a multiple of 2, see the lane quarters)
constexpr int ROWS_THREADS = 32 * (EPI_WARP0 + EPI_WARPS);
constexpr int SMEM_BYTES_ROWS = SMEM_BYTES + EPI_BYTES;
constexpr int ACC_COLS = 256;                             // widest output tile of the rows kernel (one MMA: N <= 256)
constexpr int TMEM_COLS = 2 * ACC_COLS;                   // two accumulators: all 512 columns of the SM's tensor memory

struct TcArgs {
    const RowSpan* tiles;
    int ntiles_rows, ntn, BN, Kd;
    float* C;
    uint2* Cbf;   // mode 0: the result as bfloat16 (four values per uint2) instead of C, or null
    int ldc;
    const float* Hmask;
    int ldh;
    float scale;
    int mode, passes;
    int32_t* err;
    ActEpi act;   // mode 2
};

__global__ void __launch_bounds__(ROWS_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmBlo, const TcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* sm = smem_raw + pad;                 // 1024-byte aligned: the 128B swizzle pattern repeats every 1024 bytes
    const uint32_t sm_addr = raw_addr + pad;
    // The ring holds as many stages as fit: a stage is A (and its low half when splitting) plus the B tile(s) of
    // BN rows, so narrow outputs and the single-pass mode get a deeper ring.
    const uint32_t b_bytes = (uint32_t)a.BN * BK * 4;
    const uint32_t off_b = a.passes > 1 ? 2u * A_BYTES : (uint32_t)A_BYTES;
    const uint32_t stage_bytes = off_b + (a.passes > 1 ? 2u : 1u) * b_bytes;
    const int nst = min(MAX_STAGES, (int)(RING_BYTES / stage_bytes));
    const uint32_t bars = sm_addr + RING_BYTES;
    auto full = [&](int s) { return bars + 8u * s; };
    auto xfull = [&](int s) { return bars + 8u * (MAX_STAGES + s); };
    auto empty = [&](int s) { return bars + 8u * (2 * MAX_STAGES + s); };
    auto tfull = [&](int i) { return bars + 8u * (3 * MAX_STAGES + i); };
    auto tempty = [&](int i) { return bars + 8u * (3 * MAX_STAGES + 2 + i); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + RING_BYTES + 8 * (3 * MAX_STAGES + 4));
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* epi_sm = reinterpret_cast<float*>(sm + RING_BYTES + 256);   // EPI_WARPS x 32 x 33 floats

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        // one arrival per splitting / draining warp
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(full(s), 1); mbar_init(xfull(s), SPLIT_WARPS); mbar_init(empty(s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(tfull(i), 1); mbar_init(tempty(i), EPI_WARPS); }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    const int ntiles = a.ntiles_rows * a.ntn;
    const int nkb = (a.Kd + BK - 1) / BK;
    const uint32_t tx_bytes = A_BYTES + (a.passes > 1 ? 2u : 1u) * b_bytes;

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer ----------------
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
            const RowSpan sp = a.tiles[t / a.ntn];
            const int n0 = (t % a.ntn) * a.BN;
            for (int kb = 0; kb < nkb; ++kb) {
                if (!(ok = mbar_wait(empty(stage), phase ^ 1u, abort_flag, a.err, 1))) break;
                mbar_expect_tx(full(stage), tx_bytes);
                const uint32_t base = sm_addr + stage * stage_bytes;
                tma_load_2d(base, &tmA, kb * BK, sp.row0, full(stage));
                tma_load_3d(base + off_b, &tmB, kb * BK, n0, sp.k, full(stage));
                if (a.passes > 1) tma_load_3d(base + off_b + b_bytes, &tmBlo, kb * BK, n0, sp.k, full(stage));
                if (++stage == nst) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer ----------------
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        const uint32_t idesc = instr_desc(a.BN);
        bool ok = true;
        for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
            if (!(ok = mbar_wait(tempty(acc), acc_phase ^ 1u, abort_flag, a.err, 2))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t d = tmem_base + (uint32_t)(acc * ACC_COLS);
            for (int kb = 0; kb < nkb; ++kb) {
                if (!(ok = mbar_wait(full(stage), phase, abort_flag, a.err, 3))) break;
                if (!(ok = mbar_wait(xfull(stage), phase, abort_flag, a.err, 4))) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t base = sm_addr + stage * stage_bytes;
                const uint64_t a_hi = smem_desc(base), a_lo = smem_desc(base + A_BYTES);
                const uint64_t b_hi = smem_desc(base + off_b), b_lo = smem_desc(base + off_b + b_bytes);
                // One thread issues every MMA, so the instructions between two MMAs are the cost: the common case of a
                // full block of four K steps is unrolled with constant descriptor offsets (8 TF32 values = 32 bytes = 2
                // descriptor units along K).
                const int nks = min(BK / 8, (a.Kd - kb * BK + 7) / 8);
                if (nks == BK / 8) {
                    if (a.passes > 1) {
#pragma unroll
                        for (int ks = 0; ks < BK / 8; ++ks) {
                            mma_tf32(d, a_hi + 2 * ks, b_hi + 2 * ks, idesc, ks == 0 ? (kb != 0 ? 1u : 0u) : 1u);
                            mma_tf32(d, a_hi + 2 * ks, b_lo + 2 * ks, idesc, 1u);
                            mma_tf32(d, a_lo + 2 * ks, b_hi + 2 * ks, idesc, 1u);
                        }
                    } else {
#pragma unroll
                        for (int ks = 0; ks < BK / 8; ++ks)
                            mma_tf32(d, a_hi + 2 * ks, b_hi + 2 * ks, idesc, ks == 0 ? (kb != 0 ? 1u : 0u) : 1u);
                    }
                } else {
                    for (int ks = 0; ks < nks; ++ks) {
                        const uint64_t adv = (uint64_t)(2 * ks);
                        mma_tf32(d, a_hi + adv, b_hi + adv, idesc, (kb | ks) != 0 ? 1u : 0u);
                        if (a.passes > 1) {
                            mma_tf32(d, a_hi + adv, b_lo + adv, idesc, 1u);
                            mma_tf32(d, a_lo + adv, b_hi + adv, idesc, 1u);
                        }
                    }
                }
                mma_commit(empty(stage));     // the stage may be refilled once these MMAs have read it
                if (++stage == nst) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            mma_commit(tfull(acc));           // accumulator complete
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    } else if (warp >= 2 && warp < EPI_WARP0) {
        // ---------------- A split: lo = x - (x as the tensor core reads it) ----------------
        const int tt = threadIdx.x - 64;
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
            for (int kb = 0; kb < nkb; ++kb) {
                // (the vote keeps the warp together: lanes may see a time-out or an abort at different polls)
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(full(stage), phase, abort_flag, a.err, 5)))) break;
                if (a.passes > 1) {
                    float4* hi = reinterpret_cast<float4*>(sm + stage * stage_bytes);
                    float4* lo = reinterpret_cast<float4*>(sm + stage * stage_bytes + A_BYTES);
#pragma unroll 4
                    for (int j = 0; j < A_BYTES / 16 / (32 * SPLIT_WARPS); ++j) {
                        const int i = tt + 32 * SPLIT_WARPS * j;
                        const float4 v = hi[i];   // stays where it is: the MMA reads it as the hi part
                        lo[i] = make_float4(tf32_rest(v.x), tf32_rest(v.y), tf32_rest(v.z), tf32_rest(v.w));
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> tensor-core reads
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(xfull(stage));
                if (++stage == nst) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp >= EPI_WARP0) {
        // ---------------- epilogue: tensor memory -> registers -> global ----------------
        // this warp may read tensor-memory lanes 32q .. 32q+31; the two warps of a quarter take alternate
        // blocks of 32 columns
        const int q = warp & 3, half = (warp - EPI_WARP0) >> 2;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
            const RowSpan sp = a.tiles[t / a.ntn];
            const int n0 = (t % a.ntn) * a.BN;
            if (!(ok = __all_sync(0xffffffffu, mbar_wait(tfull(acc), acc_phase, abort_flag, a.err, 6)))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // A thread receives one accumulator row (32 columns at a time); the warp turns its 32 x 32 block through
            // shared memory so that 8 lanes write 128 contiguous bytes of one output row.
            float* tr = epi_sm + (warp - EPI_WARP0) * (32 * 33);
            const int sub_r = lane >> 3, sub_c = (lane & 7) * 4;
            for (int c0 = 32 * half; c0 < a.BN && n0 + c0 < a.ldc; c0 += 64) {
                const int n = n0 + c0 + sub_c;
                // the eight mask loads of this lane go out together, ahead of the accumulator read and of any store
                float4 hm[8];
                const bool masked = a.mode == 1 && a.Hmask != nullptr;   // mode 1 without a mask: plain A W^T
                if (masked) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int r = q * 32 + 4 * i + sub_r;
                        hm[i] = (r < sp.nrows && n < a.ldc)
                                    ? __ldg(reinterpret_cast<const float4*>(a.Hmask + ((long long)sp.row0 + r) * a.ldh + n))
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                float4 bias4 = make_float4(0.f, 0.f, 0.f, 0.f);
                if (a.mode == 2 && n < a.ldc) bias4 = load_bias(a.act, sp.k, n);
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * ACC_COLS + c0), v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int j = 0; j < 32; ++j) tr[lane * 33 + j] = __uint_as_float(v[j]);
                __syncwarp();
                float4 o[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float* src = tr + (4 * i + sub_r) * 33 + sub_c;
                    o[i] = make_float4(src[0], src[1], src[2], src[3]);
                    if (masked) {
                        o[i].x = hm[i].x > 0.f ? o[i].x * a.scale : 0.f;
                        o[i].y = hm[i].y > 0.f ? o[i].y * a.scale : 0.f;
                        o[i].z = hm[i].z > 0.f ? o[i].z * a.scale : 0.f;
                        o[i].w = hm[i].w > 0.f ? o[i].w * a.scale : 0.f;
                    }
                    if (a.mode == 2) o[i] = apply_act(o[i], bias4, a.act, (long long)sp.row0 + q * 32 + 4 * i + sub_r, n);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = q * 32 + 4 * i + sub_r;
                    if (r < sp.nrows && n < a.ldc) {
                        if (a.Cbf) a.Cbf[(((long long)sp.row0 + r) * a.ldc + n) >> 2] = bf16_pack4(o[i]);
                        else *reinterpret_cast<float4*>(a.C + ((long long)sp.row0 + r) * a.ldc + n) = o[i];
                    }
                }
                __syncwarp();
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }

    // Tear-down.  After a time-out, give loads that may still be in flight a bounded chance to land before the
    // shared memory is released.
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0)
        for (int s = 0; s < nst; ++s)
            for (uint32_t i = 0; i < 4096u; ++i)
                if (mbar_try_wait(full(s), 0) || mbar_try_wait(full(s), 1)) break;
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// W_k^(l) [fi x ldw] -> the four K-major operand copies the tensor-core kernels read:
//   w_hi / w_lo   [K][fi][ldw]    (B of mode 1: rows n = input feature, Kd = output feature)
//   wt_hi / wt_lo [K][fo][ldkt]   (B of mode 0: rows n = output feature, Kd = input feature)
__global__ void split_weights_kernel(const float* __restrict__ params, long long pstride, long long w_int, int fi, int fo, int ldw,
                                     int ldkt, float* __restrict__ w_hi, float* __restrict__ w_lo, float* __restrict__ wt_hi,
                                     float* __restrict__ wt_lo) {
    const int k = blockIdx.y;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)fi * ldw) return;
    const int i = (int)(idx / ldw), j = (int)(idx % ldw);
    const float w = params[(long long)k * pstride + w_int + idx];
    const float h = tf32_hi(w), l = tf32_round(w - h);
    w_hi[(long long)k * fi * ldw + idx] = h;
    w_lo[(long long)k * fi * ldw + idx] = l;
    if (j < fo) {
        wt_hi[((long long)k * fo + j) * ldkt + i] = h;
        wt_lo[((long long)k * fo + j) * ldkt + i] = l;
    }
}

// ---------------------------------------------------------------------------------------------
// Weight gradient dW_k = H_k^T dZ_k on the tensor cores: partial[chunk][m][n] = sum over the chunk's rows r of
// H[r][m] dZ[r][n].  The reduction index is the row, so both operands are "MN-major": a tile of 32 rows x 32
// values (128 bytes per row, swizzled in 32-byte units) is one block of the canonical layout, blocks of 32 values
// are 4096 bytes apart (leading byte offset), groups of 4 rows 512 bytes apart (stride byte offset), and one MMA
// (K = 8) consumes 8 rows.  Both operands are activations, so both get a lo tile written beside them in shared memory;
// rows past the end of the chunk are zeroed there.  One CTA per (chunk, 128 x BN output tile).
// ---------------------------------------------------------------------------------------------
struct TnArgs {
    const RowSpan* chunks;
    int ntm, ntn, BN, M, ldw;   // output tiles per chunk, MMA N, valid output rows, leading dimension of the output
    float* partial;
    long long pstride_chunk;
    int passes;
    int32_t* err;
};

// Rows of the reduction per ring stage of the weight-gradient kernel (a multiple of 8, the K of one MMA).  With 32 rows the
// ring holds two stages at 256 output columns; 16 rows (four stages) measured the same on the 2.5 M-row workload (2.37 vs
// 2.49 ms at 256 x 256, but 1.41 vs 1.26 ms at 256 x 47) and slower on the small one: the stage count is not what limits it.
constexpr int TBK = 32;
constexpr int TN_BLOCK_BYTES = TBK * 128;                 // one block: TBK rows x 32 values
constexpr int TN_A_BYTES = 4 * TN_BLOCK_BYTES;            // 128 output rows = 4 blocks
// MN-major TF32 tile: layout type 1 (128-byte swizzle of 32-byte units, repeating every 4 rows = 512 bytes), blocks of
// 32 values TN_BLOCK_BYTES apart (leading byte offset), groups of 4 rows 512 bytes apart (stride byte offset).
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(TN_BLOCK_BYTES >> 4) << 16) | ((uint64_t)(512 >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)1 << 61);
}

constexpr int TN_THREADS = 512;   // warp 0: TMA, warp 1: MMA, warps 2..15: operand split, warps 8..15 also drain the accumulator
__global__ void __launch_bounds__(TN_THREADS, 1)
gemm_tn_tc_kernel(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmZ, const TnArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
    uint8_t* sm = smem_raw + pad;
    const uint32_t sm_addr = raw_addr + pad;
    // a stage holds the H tile and its low half and the dZ tile of BN columns with its low half, TBK rows each
    const int nb_blocks = (a.BN + 31) / 32;                    // 32-value blocks of the B tile
    const uint32_t b_bytes = (uint32_t)nb_blocks * TN_BLOCK_BYTES;
    const uint32_t stage_bytes = 2u * TN_A_BYTES + 2u * b_bytes;
    const int nst = min(MAX_STAGES, (int)(RING_BYTES / stage_bytes));
    const uint32_t bars = sm_addr + RING_BYTES;
    auto full = [&](int s) { return bars + 8u * s; };
    auto xfull = [&](int s) { return bars + 8u * (MAX_STAGES + s); };
    auto empty = [&](int s) { return bars + 8u * (2 * MAX_STAGES + s); };
    const uint32_t tfull = bars + 8u * (3 * MAX_STAGES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + RING_BYTES + 8 * (3 * MAX_STAGES + 4));
    volatile uint32_t* abort_flag = tmem_slot + 1;
    constexpr int NSPLIT = TN_THREADS - 64;   // threads of warps 2..15

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(full(s), 1); mbar_init(xfull(s), NSPLIT / 32); mbar_init(empty(s), 1); }   // one arrival per splitting warp
        mbar_init(tfull, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(ACC_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    const int tiles_per_chunk = a.ntm * a.ntn;
    const RowSpan c = a.chunks[blockIdx.x / tiles_per_chunk];
    const int tile = blockIdx.x % tiles_per_chunk;
    const int m0 = (tile / a.ntn) * BM, n0 = (tile % a.ntn) * a.BN;
    const int nkb = (c.nrows + TBK - 1) / TBK;
    const uint32_t tx_bytes = (uint32_t)(4 + nb_blocks) * TN_BLOCK_BYTES;
    bool ok = true;

    if (warp == 0 && lane == 0) {
        int stage = 0;
        uint32_t phase = 0;
        for (int kb = 0; kb < nkb; ++kb) {
            if (!(ok = mbar_wait(empty(stage), phase ^ 1u, abort_flag, a.err, 11))) break;
            mbar_expect_tx(full(stage), tx_bytes);
            const uint32_t base = sm_addr + stage * stage_bytes;
            const int r = c.row0 + kb * TBK;
            for (int j = 0; j < 4; ++j) tma_load_2d(base + j * TN_BLOCK_BYTES, &tmH, m0 + 32 * j, r, full(stage));
            for (int j = 0; j < nb_blocks; ++j) tma_load_2d(base + 2 * TN_A_BYTES + j * TN_BLOCK_BYTES, &tmZ, n0 + 32 * j, r, full(stage));
            if (++stage == nst) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == 1 && lane == 0) {
        int stage = 0;
        uint32_t phase = 0;
        const uint32_t idesc = instr_desc(a.BN) | (1u << 15) | (1u << 16);   // A and B MN-major
        for (int kb = 0; kb < nkb; ++kb) {
            if (!(ok = mbar_wait(full(stage), phase, abort_flag, a.err, 13))) break;
            if (!(ok = mbar_wait(xfull(stage), phase, abort_flag, a.err, 14))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t base = sm_addr + stage * stage_bytes;
            const int nks = min(TBK / 8, (c.nrows - kb * TBK + 7) / 8);
            const uint64_t a_hi = smem_desc_mn(base), a_lo = smem_desc_mn(base + TN_A_BYTES);
            const uint64_t b_hi = smem_desc_mn(base + 2 * TN_A_BYTES), b_lo = smem_desc_mn(base + 2 * TN_A_BYTES + b_bytes);
            // the next group of 8 rows is 1024 bytes = 64 descriptor units further on; a full block is unrolled so that
            // the issuing thread spends few instructions between two MMAs
            if (nks == TBK / 8 && a.passes > 1) {
#pragma unroll
                for (int ks = 0; ks < TBK / 8; ++ks) {
                    mma_tf32(tmem_base, a_hi + 64 * ks, b_hi + 64 * ks, idesc, ks == 0 ? (kb != 0 ? 1u : 0u) : 1u);
                    mma_tf32(tmem_base, a_hi + 64 * ks, b_lo + 64 * ks, idesc, 1u);
                    mma_tf32(tmem_base, a_lo + 64 * ks, b_hi + 64 * ks, idesc, 1u);
                }
            } else {
                for (int ks = 0; ks < nks; ++ks) {
                    const uint64_t adv = (uint64_t)(64 * ks);
                    mma_tf32(tmem_base, a_hi + adv, b_hi + adv, idesc, (kb | ks) != 0 ? 1u : 0u);
                    if (a.passes > 1) {
                        mma_tf32(tmem_base, a_hi + adv, b_lo + adv, idesc, 1u);
                        mma_tf32(tmem_base, a_lo + adv, b_hi + adv, idesc, 1u);
                    }
                }
            }
            mma_commit(empty(stage));
            if (++stage == nst) { stage = 0; phase ^= 1u; }
        }
        if (ok) mma_commit(tfull);
    } else if (warp >= 2) {
        // write the lo tile of both operands and zero the rows past the end of the chunk
        const int tt = threadIdx.x - 64;
        int stage = 0;
        uint32_t phase = 0;
        constexpr int BF4 = TN_BLOCK_BYTES / 16;              // float4 values of one block
        const int nf4 = (4 + nb_blocks) * BF4;                // float4 values of the stage's A and B tiles
        for (int kb = 0; kb < nkb; ++kb) {
            // (the vote keeps the warp together: lanes may see a time-out or an abort at different polls)
            if (!(ok = __all_sync(0xffffffffu, mbar_wait(full(stage), phase, abort_flag, a.err, 15)))) break;
            const int rows_valid = min(TBK, c.nrows - kb * TBK);
            if (a.passes > 1 || rows_valid < TBK) {
                uint8_t* sb = sm + stage * stage_bytes;
                for (int i = tt; i < nf4; i += NSPLIT) {
                    const int blk = i / BF4, in = i % BF4;                        // block of 32 values, float4 inside it
                    const int row = in >> 3;                                      // 8 float4 per 128-byte row
                    const int byte_off = (blk < 4 ? blk * TN_BLOCK_BYTES : 2 * TN_A_BYTES + (blk - 4) * TN_BLOCK_BYTES) + in * 16;
                    float4* hi = reinterpret_cast<float4*>(sb + byte_off);
                    float4* lo = reinterpret_cast<float4*>(sb + byte_off + (blk < 4 ? (uint32_t)TN_A_BYTES : b_bytes));
                    float4 v = *hi;   // a valid row stays where it is: the MMA reads it as the hi part
                    if (row >= rows_valid) {
                        v = make_float4(0.f, 0.f, 0.f, 0.f);
                        *hi = v;
                    }
                    if (a.passes > 1) *lo = make_float4(tf32_rest(v.x), tf32_rest(v.y), tf32_rest(v.z), tf32_rest(v.w));
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(xfull(stage));
            if (++stage == nst) { stage = 0; phase ^= 1u; }
        }
    }
    // epilogue by warps 8..15 (two per quarter of the tensor-memory lanes, alternate blocks of 32 columns) once
    // every MMA has completed
    if (warp >= 8) {
        const int q = warp & 3, half = (warp - 8) >> 2;
        const bool done = mbar_wait(tfull, 0, abort_flag, a.err, 16);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int m = m0 + q * 32 + lane;
        float* P = a.partial + (long long)(blockIdx.x / tiles_per_chunk) * a.pstride_chunk;
        for (int c0 = 32 * half; c0 < a.BN && n0 + c0 < a.ldw; c0 += 64) {
            uint32_t v[32];
            tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (done && m < a.M) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int n = n0 + c0 + 4 * j;
                    if (n >= a.ldw) break;
                    *reinterpret_cast<float4*>(P + (long long)m * a.ldw + n) =
                        make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                    __uint_as_float(v[4 * j + 3]));
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(ACC_COLS) : "memory");
    }
}

// The bounded wait of the kernels above, made to run out: one thread polls a barrier that nothing ever arrives at.
__global__ void expire_wait_kernel(int32_t* err, uint32_t polls) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(smem_u32(&bar), 0u, &abort_flag, err, 99, polls);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

}  // namespace

// Output columns per tile: one MMA covers up to 256, and an M = 128, K = 8 TF32 MMA costs about the same for any N, so
// the widest tile that the ring still holds twice is the cheapest.  (Measured again on 2.5 M rows x 256 x 256: two tiles of
// 128 columns with a three-stage ring take 2.07 ms where one tile of 256 columns with two stages takes 1.72 ms.)
int tc_tn_rows() { return TBK; }
int tc_bn_for(int n_cols) { return n_cols <= 16 ? 16 : n_cols <= 32 ? 32 : n_cols <= 64 ? 64 : n_cols <= 128 ? 128 : 256; }

// fp32 tensor [outer (z)] x [rows (y)] x [inner (x)], box = 32 floats x box_rows x 1, zero fill outside.  K-major
// operand tiles use the 128-byte swizzle of 16-byte units; MN-major TF32 tiles need the 128-byte swizzle of
// 32-byte units (the only MN-major layout the tensor cores accept for 32-bit operands).
bool tc_make_map(void* out_map, const void* base, uint64_t inner, uint64_t rows, uint64_t outer, uint64_t row_stride_bytes,
                 uint64_t outer_stride_bytes, uint32_t box_rows, bool mn_major) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const bool three = outer > 0;
    cuuint64_t dims[3] = {inner, rows, three ? outer : 1};
    cuuint64_t strides[2] = {row_stride_bytes, outer_stride_bytes};
    cuuint32_t box[3] = {(cuuint32_t)BK, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(reinterpret_cast<CUtensorMap*>(out_map), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, three ? 3 : 2, const_cast<void*>(base), dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    mn_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

cudaError_t launch_expire_wait(int32_t* err, uint32_t polls, cudaStream_t s) {
    expire_wait_kernel<<<1, 32, 0, s>>>(err, polls);
    ++g_kernel_launches;
    return cudaGetLastError();
}

cudaError_t launch_split_weights(const float* params, int64_t pstride, int64_t w_int, int fi, int fo, int ldw, int ldkt, int K,
                                 float* w_hi, float* w_lo, float* wt_hi, float* wt_lo, cudaStream_t s) {
    const long long n = (long long)fi * ldw;
    split_weights_kernel<<<dim3((unsigned)((n + 255) / 256), (unsigned)K), 256, 0, s>>>(params, pstride, w_int, fi, fo, ldw, ldkt, w_hi, w_lo,
                                                                                        wt_hi, wt_lo);
    ++g_kernel_launches;
    return cudaGetLastError();
}

cudaError_t launch_gemm_rows_tc(const void* mapA, const void* mapB, const void* mapBlo, int mode, int passes, int Kd, int n_cols,
                                float* C, int ldc, const RowSpan* tiles, int ntiles, const float* Hmask, int ldh, float scale,
                                const ActEpi* act, int32_t* err, int num_sms, cudaStream_t s, void* Cbf16) {
    if (ntiles <= 0) return cudaSuccess;
    if ((mode == 2 && !act) || (Cbf16 && mode != 0)) return cudaErrorInvalidValue;
    {
        cudaError_t e = configure_kernel_once(reinterpret_cast<const void*>(gemm_tc_kernel), SMEM_BYTES_ROWS, false);
        if (e != cudaSuccess) return e;
    }
    TcArgs a;
    a.tiles = tiles; a.ntiles_rows = ntiles; a.BN = tc_bn_for(n_cols); a.ntn = (ldc + a.BN - 1) / a.BN; a.Kd = Kd;
    a.C = C; a.Cbf = reinterpret_cast<uint2*>(Cbf16); a.ldc = ldc; a.Hmask = Hmask; a.ldh = ldh; a.scale = scale; a.mode = mode; a.passes = passes; a.err = err;
    a.act = act ? *act : ActEpi{};
    const long long total = (long long)ntiles * a.ntn;
    const unsigned grid = (unsigned)(total < num_sms ? total : num_sms);
    gemm_tc_kernel<<<grid, ROWS_THREADS, SMEM_BYTES_ROWS, s>>>(*reinterpret_cast<const CUtensorMap*>(mapA), *reinterpret_cast<const CUtensorMap*>(mapB),
                                                 *reinterpret_cast<const CUtensorMap*>(mapBlo), a);
    ++g_kernel_launches;
    return cudaGetLastError();
}

cudaError_t launch_gemm_tn_tc(const void* mapH, const void* mapZ, int passes, int M, int n_cols, int ldw, const RowSpan* chunks,
                              int nchunks, float* partial, int32_t* err, cudaStream_t s) {
    if (nchunks <= 0) return cudaSuccess;
    {
        cudaError_t e = configure_kernel_once(reinterpret_cast<const void*>(gemm_tn_tc_kernel), SMEM_BYTES, false);
        if (e != cudaSuccess) return e;
    }
    TnArgs a;
    a.chunks = chunks; a.BN = tc_bn_for(n_cols); a.ntm = (M + BM - 1) / BM; a.ntn = (ldw + a.BN - 1) / a.BN; a.M = M; a.ldw = ldw;
    a.partial = partial; a.pstride_chunk = (long long)M * ldw; a.passes = passes; a.err = err;
    const unsigned grid = (unsigned)((long long)nchunks * a.ntm * a.ntn);
    gemm_tn_tc_kernel<<<grid, TN_THREADS, SMEM_BYTES, s>>>(*reinterpret_cast<const CUtensorMap*>(mapH), *reinterpret_cast<const CUtensorMap*>(mapZ), a);
    ++g_kernel_launches;
    return cudaGetLastError();
}

}  // namespace gad
