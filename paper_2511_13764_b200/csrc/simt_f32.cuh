// FP32 GEMM on the FMA pipe (B200 has no exact-FP32 tensor-core MMA).
//
// This is the FP32 body of the paper's Algorithm 1 ("broadcast the A sub-column,
// load a B chunk, FMA into the resident accumulators") in its outer-product form:
// each thread keeps a TM x TN block of C in registers for the whole K loop and,
// per k, reads TM values of A and TN values of B from shared memory with 128-bit
// loads.  Tiles are double-buffered through registers so the global loads of
// k-tile t+1 are in flight while k-tile t is multiplied.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace nk {

constexpr int SIMT_BK = 16;

struct SimtParams {
    int M, N, K;
    int splits;        // gridDim.z; > 1 writes partials
    int kt_per_split;  // k-tiles (of 16) per split
    int batch;         // batch-reduce: number of (A_b, B_b) pairs summed into C (>= 1)
    int kt_per_item;   // ceil(K / 16): k-tiles of one pair
    long long stride_a, stride_b;  // elements between consecutive A_b / B_b
    int beta;          // 1: the old C is added before the epilogue
    int gemms;         // independent GEMMs in one launch (batched matmul), else 1; gridDim.z = splits * gemms
    long long stride_c;  // elements from C_g to C_g+1
    int epilogue;      // 0 none, 1 bias + ReLU
    const float* A;    // [M][K]
    const float* B;    // [K][N]
    const float* bias; // [N] or null
    float* C;          // [M][N]
    float* partial;    // [splits][M][N]
};

template <int BM, int BN, int TM, int TN>
__global__ void __launch_bounds__((BM / TM) * (BN / TN), (BM >= 128 ? 2 : 1))
simt_f32_kernel(const SimtParams p) {
    constexpr int THREADS = (BM / TM) * (BN / TN);
    constexpr int TX = BN / TN;          // threads across N
    constexpr int GM = TM / 4, GN = TN / 4;  // 4-wide groups per thread
    constexpr int SM_STRIDE = BM / GM;   // row distance between a thread's groups
    constexpr int SN_STRIDE = BN / GN;
    constexpr int AP = BM + 4;           // padded row length of the transposed A tile
    constexpr int A_V4 = BM * SIMT_BK / 4 / THREADS;  // float4 loads per thread per tile
    constexpr int B_V4 = BN * SIMT_BK / 4 / THREADS;
    static_assert(TM % 4 == 0 && TN % 4 == 0, "thread tile is built from 4-wide groups");
    static_assert(A_V4 >= 1 && B_V4 >= 1, "tile too small for the thread count");

    __shared__ __align__(16) float As[2][SIMT_BK][AP];  // As[k][m]
    __shared__ __align__(16) float Bs[2][SIMT_BK][BN];  // Bs[k][n]

    const int t = threadIdx.x;
    const int ty = t / TX, tx = t % TX;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int ktiles = p.batch * p.kt_per_item;   // k-tiles of the whole batch-reduce
    const int gemm = blockIdx.z / p.splits, split = blockIdx.z - gemm * p.splits;
    const int kt0 = split * p.kt_per_split;
    const int kt1 = min(ktiles, kt0 + p.kt_per_split);

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.0f;

    float4 ra[A_V4], rb[B_V4];

    // Where this thread's share of the next k-tile lives in global memory.  The position is
    // kept as two running pointers that step by one k-tile per load (and by the item stride at
    // the end of a batch-reduce item), so the K loop carries no divisions or 64-bit multiplies.
    const int item0 = kt0 / p.kt_per_item;
    int kin = kt0 - item0 * p.kt_per_item;                 // k-tile inside the current (A_b, B_b) pair
    const int a_row = t >> 2, a_kq = (t & 3) * 4;          // A: rows a_row + i * THREADS / 4, 4 k per load
    const int b_kr = t / (BN / 4), b_nq = (t % (BN / 4)) * 4;   // B: k rows b_kr + i * THREADS / (BN / 4)
    const float* pa = p.A + (gemm + item0) * p.stride_a + static_cast<size_t>(m0 + a_row) * p.K + kin * SIMT_BK + a_kq;
    const float* pb = p.B + (gemm + item0) * p.stride_b + static_cast<size_t>(kin * SIMT_BK + b_kr) * p.N + n0 + b_nq;
    const int a_step_i = (THREADS / 4) * p.K, b_step_i = (THREADS / (BN / 4)) * p.N;   // K, N < 2^24: these fit 32 bits
    const int b_step_kt = SIMT_BK * p.N;
    const bool b_col_ok = n0 + b_nq < p.N;

    auto load_global = [&]() {
        const int k0 = kin * SIMT_BK;
#pragma unroll
        for (int i = 0; i < A_V4; ++i)
            ra[i] = (m0 + a_row + i * (THREADS / 4) < p.M && k0 + a_kq < p.K)
                        ? __ldg(reinterpret_cast<const float4*>(pa + i * a_step_i))
                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < B_V4; ++i)
            rb[i] = (b_col_ok && k0 + b_kr + i * (THREADS / (BN / 4)) < p.K)
                        ? __ldg(reinterpret_cast<const float4*>(pb + i * b_step_i))
                        : make_float4(0.f, 0.f, 0.f, 0.f);
        pa += SIMT_BK;
        pb += b_step_kt;
        if (++kin == p.kt_per_item) {   // next item of the batch-reduce
            kin = 0;
            pa += p.stride_a - static_cast<long long>(p.kt_per_item) * SIMT_BK;
            pb += p.stride_b - static_cast<long long>(p.kt_per_item) * SIMT_BK * p.N;
        }
    };
    auto store_shared = [&](int buf) {
#pragma unroll
        for (int i = 0; i < A_V4; ++i) {
            const int idx = t + i * THREADS;
            const int row = idx >> 2, kq = (idx & 3) * 4;
            As[buf][kq + 0][row] = ra[i].x;
            As[buf][kq + 1][row] = ra[i].y;
            As[buf][kq + 2][row] = ra[i].z;
            As[buf][kq + 3][row] = ra[i].w;
        }
#pragma unroll
        for (int i = 0; i < B_V4; ++i) {
            const int idx = t + i * THREADS;
            const int kr = idx / (BN / 4), nq = (idx % (BN / 4)) * 4;
            *reinterpret_cast<float4*>(&Bs[buf][kr][nq]) = rb[i];
        }
    };

    int buf = 0;
    if (kt0 < kt1) {
        load_global();
        store_shared(0);
    }
    __syncthreads();

    for (int kt = kt0; kt < kt1; ++kt) {
        const bool more = kt + 1 < kt1;
        if (more) load_global();
#pragma unroll
        for (int k = 0; k < SIMT_BK; ++k) {
            float a[TM], b[TN];
#pragma unroll
            for (int g = 0; g < GM; ++g) {
                const float4 v = *reinterpret_cast<const float4*>(&As[buf][k][g * SM_STRIDE + ty * 4]);
                a[4 * g] = v.x; a[4 * g + 1] = v.y; a[4 * g + 2] = v.z; a[4 * g + 3] = v.w;
            }
#pragma unroll
            for (int g = 0; g < GN; ++g) {
                const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][k][g * SN_STRIDE + tx * 4]);
                b[4 * g] = v.x; b[4 * g + 1] = v.y; b[4 * g + 2] = v.z; b[4 * g + 3] = v.w;
            }
            // serpentine order over the thread tile: consecutive FMAs share an operand register
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int jj = 0; jj < TN; ++jj) {
                    const int j = (i & 1) ? TN - 1 - jj : jj;
                    acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
                }
        }
        if (more) {
            store_shared(buf ^ 1);
            __syncthreads();
            buf ^= 1;
        }
    }

    // Epilogue: bias + ReLU on the accumulator, then the single store of C.
    const bool to_partial = p.splits > 1;
    float* out = to_partial ? p.partial + (static_cast<size_t>(split) * p.gemms + gemm) * p.M * p.N
                            : p.C + gemm * p.stride_c;
#pragma unroll
    for (int gi = 0; gi < GM; ++gi)
#pragma unroll
        for (int ii = 0; ii < 4; ++ii) {
            const int gm = m0 + gi * SM_STRIDE + ty * 4 + ii;
            if (gm >= p.M) continue;
#pragma unroll
            for (int gj = 0; gj < GN; ++gj) {
                const int gn = n0 + gj * SN_STRIDE + tx * 4;
                if (gn >= p.N) continue;
                float4 v = make_float4(acc[4 * gi + ii][4 * gj], acc[4 * gi + ii][4 * gj + 1],
                                       acc[4 * gi + ii][4 * gj + 2], acc[4 * gi + ii][4 * gj + 3]);
                if (!to_partial && p.beta) {       // beta = 1: the accumulation tile starts from the stored C
                    const float4 cv = *reinterpret_cast<const float4*>(out + static_cast<size_t>(gm) * p.N + gn);
                    v.x += cv.x; v.y += cv.y; v.z += cv.z; v.w += cv.w;
                }
                if (!to_partial && p.epilogue) {
                    const float4 bv = __ldg(reinterpret_cast<const float4*>(p.bias + gn));
                    v.x = fmaxf(v.x + bv.x, 0.f);
                    v.y = fmaxf(v.y + bv.y, 0.f);
                    v.z = fmaxf(v.z + bv.z, 0.f);
                    v.w = fmaxf(v.w + bv.w, 0.f);
                }
                *reinterpret_cast<float4*>(out + static_cast<size_t>(gm) * p.N + gn) = v;
            }
        }
}

}  // namespace nk

namespace nk {

// Skinny FP32 GEMM (M <= MR rows): bound by the one pass over B, not by the FMA pipe.
// A CTA of 128 threads owns 512 consecutive columns and a chunk of K: it parks its slice of A
// in shared memory once (transposed, so the MR values of one k are read with broadcast
// 128-bit loads), then streams B with no barrier in the loop: every thread keeps 8 independent
// 16-byte loads in flight (row segments of 512 B per warp; a rolling window) and holds an MR x 4 block of C in
// registers (Algorithm 1's resident accumulator), as MR / 2 x 4 register pairs along M that are
// updated with packed FMAs (fma.rn.f32x2: the pair of A values comes straight from shared
// memory, the B value is copied into both halves), which halves the issue slots the 16 FMAs
// per loaded element need.  K chunks are combined by the split-K reduce.
constexpr int SKINNY_COLS = 512;
constexpr int SKINNY_THREADS = 128;
constexpr int SKINNY_A_FLOATS = 8192;   // MR * k-chunk <= this (32 KB of shared memory)

struct SkinnyParams {
    int M, N, K;
    int kc;            // k per CTA (multiple of 8)
    int splits;        // gridDim.y
    int epilogue;
    const float* A;
    const float* B;
    const float* bias;
    float* C;
    float* partial;
};

template <int MR>
__global__ void __launch_bounds__(SKINNY_THREADS, MR == 16 ? 4 : 2) simt_f32_skinny_kernel(const SkinnyParams p) {
    __shared__ __align__(16) float As[SKINNY_A_FLOATS];   // As[kk][MR]
    const int t = threadIdx.x;
    const int n = blockIdx.x * SKINNY_COLS + t * 4;
    const int k0 = blockIdx.y * p.kc;
    const int k1 = min(p.K, k0 + p.kc);
    const int klen = k1 - k0;

    // A slice: rows 0..MR-1 (zero beyond M), k0..k1, four k per load
    for (int idx = t; idx < MR * (p.kc / 4); idx += SKINNY_THREADS) {
        const int m = idx % MR, kq = (idx / MR) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (m < p.M && k0 + kq < k1)
            v = __ldg(reinterpret_cast<const float4*>(p.A + static_cast<size_t>(m) * p.K + k0 + kq));
        As[(kq + 0) * MR + m] = v.x;
        As[(kq + 1) * MR + m] = v.y;
        As[(kq + 2) * MR + m] = v.z;
        As[(kq + 3) * MR + m] = v.w;
    }
    __syncthreads();

    float2 acc[MR / 2][4];   // acc[mp][c] = rows 2 mp, 2 mp + 1 of column n + c
#pragma unroll
    for (int m = 0; m < MR / 2; ++m) acc[m][0] = acc[m][1] = acc[m][2] = acc[m][3] = make_float2(0.f, 0.f);

    const bool col_ok = n < p.N;
    const float* bptr = p.B + static_cast<size_t>(k0) * p.N + (col_ok ? n : 0);
    // a rolling window of 8 rows of B per thread: row kk + 8 + i is requested as soon as row kk + i has
    // been taken out of its register, so eight 16-byte loads stay in flight with one set of registers
    // (a second, "next group" set cost 32 registers and a CTA per SM)
    float4 b[8];
    auto load_row = [&](int k) {
        return (col_ok && k < klen) ? __ldcs(reinterpret_cast<const float4*>(bptr + static_cast<size_t>(k) * p.N))
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
    };
#pragma unroll
    for (int i = 0; i < 8; ++i) b[i] = load_row(i);
    for (int kk = 0; kk < klen; kk += 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 cur = b[i];
            b[i] = load_row(kk + 8 + i);
            const float* arow = &As[(kk + i) * MR];
            const float2 bx = make_float2(cur.x, cur.x), by = make_float2(cur.y, cur.y);
            const float2 bz = make_float2(cur.z, cur.z), bw = make_float2(cur.w, cur.w);
#pragma unroll
            for (int mq = 0; mq < MR; mq += 4) {
                const float4 a = *reinterpret_cast<const float4*>(arow + mq);
                const float2 alo = make_float2(a.x, a.y), ahi = make_float2(a.z, a.w);
                float2* c0 = acc[mq / 2];
                float2* c1 = acc[mq / 2 + 1];
                c0[0] = __ffma2_rn(alo, bx, c0[0]); c0[1] = __ffma2_rn(alo, by, c0[1]);
                c0[2] = __ffma2_rn(alo, bz, c0[2]); c0[3] = __ffma2_rn(alo, bw, c0[3]);
                c1[0] = __ffma2_rn(ahi, bx, c1[0]); c1[1] = __ffma2_rn(ahi, by, c1[1]);
                c1[2] = __ffma2_rn(ahi, bz, c1[2]); c1[3] = __ffma2_rn(ahi, bw, c1[3]);
            }
        }
    }

    if (!col_ok) return;
    const bool to_partial = p.splits > 1;
    float* out = to_partial ? p.partial + static_cast<size_t>(blockIdx.y) * p.M * p.N : p.C;
    float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
    if (!to_partial && p.epilogue) bv = __ldg(reinterpret_cast<const float4*>(p.bias + n));
#pragma unroll
    for (int m = 0; m < MR; ++m) {
        if (m >= p.M) break;
        const float2* r = acc[m / 2];
        float4 v = (m & 1) ? make_float4(r[0].y, r[1].y, r[2].y, r[3].y) : make_float4(r[0].x, r[1].x, r[2].x, r[3].x);
        if (!to_partial && p.epilogue) {
            v.x = fmaxf(v.x + bv.x, 0.f);
            v.y = fmaxf(v.y + bv.y, 0.f);
            v.z = fmaxf(v.z + bv.z, 0.f);
            v.w = fmaxf(v.w + bv.w, 0.f);
        }
        *reinterpret_cast<float4*>(out + static_cast<size_t>(m) * p.N + n) = v;
    }
}

}  // namespace nk

#include "ptx.cuh"

namespace nk {

// The same FP32 GEMM with the operand staging done by cp.async instead of registers: tiles of
// k-block t+2 and t+1 are in flight while k-block t is multiplied (three shared-memory stages),
// nothing is held in registers for staging, and the transpose of A into As[k][m] happens in
// the copy itself (4-byte copies, one element each; B rows go as 16-byte copies).
constexpr int SIMT_STAGES = 3;

template <int BM, int BN>
__host__ __device__ constexpr int simt_async_smem_bytes() {
    return SIMT_STAGES * SIMT_BK * ((BM + 4) + BN) * 4;
}

//
// X2 selects packed FMAs (fma.rn.f32x2, new with sm_100: two IEEE FP32 FMAs per instruction on an
// aligned register pair).  The FMA pipe's peak is the same, but a k-step needs half the issue
// slots, which is what makes an 8 x 16 thread tile pay: a thread then reads (8 + 16) operands
// from shared memory per 128 FMAs instead of 16 per 64, and shared-memory bandwidth (128 B per
// clock per SM against 128 FMA lanes) is the other limit of this kernel.  Accumulators are
// paired along N, the way a 128-bit load of B delivers them; the A value of a row is copied
// into both halves of a register pair.
template <int BM, int BN, int TM, int TN, bool X2>
__global__ void __launch_bounds__((BM / TM) * (BN / TN), (BM >= 128 ? 2 : 1))
simt_f32_async_kernel(const SimtParams p) {
    constexpr int THREADS = (BM / TM) * (BN / TN);
    constexpr int TX = BN / TN;
    constexpr int GM = TM / 4, GN = TN / 4;
    constexpr int SM_STRIDE = BM / GM;
    constexpr int SN_STRIDE = BN / GN;
    constexpr int AP = BM + 4;
    constexpr int A_ELEMS = BM * SIMT_BK / THREADS;        // 4-byte copies per thread per tile
    constexpr int B_V4 = BN * SIMT_BK / 4 / THREADS;       // 16-byte copies per thread per tile
    constexpr int A_STAGE = SIMT_BK * AP, B_STAGE = SIMT_BK * BN;   // floats
    static_assert(A_ELEMS >= 1 && B_V4 >= 1, "tile too small for the thread count");

    extern __shared__ __align__(16) float simt_smem[];
    float* As = simt_smem;                                  // [stage][k][AP]
    float* Bs = simt_smem + SIMT_STAGES * A_STAGE;          // [stage][k][BN]
    const uint32_t as_u32 = smem_u32(As), bs_u32 = smem_u32(Bs);

    const int t = threadIdx.x;
    const int ty = t / TX, tx = t % TX;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int ktiles = p.batch * p.kt_per_item;   // k-tiles of the whole batch-reduce
    const int gemm = blockIdx.z / p.splits, split = blockIdx.z - gemm * p.splits;
    const int kt0 = split * p.kt_per_split;
    const int kt1 = min(ktiles, kt0 + p.kt_per_split);

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.0f;

    // running global positions of this thread's copies (see simt_f32_kernel)
    const int item0 = kt0 / p.kt_per_item;
    int kin = kt0 - item0 * p.kt_per_item;
    const int a_k = t & (SIMT_BK - 1), a_row = t / SIMT_BK;     // A: rows a_row + i * THREADS / 16
    const int b_kr = t / (BN / 4), b_nq = (t % (BN / 4)) * 4;   // B: k rows b_kr + i * THREADS / (BN / 4)
    const float* pa = p.A + (gemm + item0) * p.stride_a + static_cast<size_t>(m0 + a_row) * p.K + kin * SIMT_BK + a_k;
    const float* pb = p.B + (gemm + item0) * p.stride_b + static_cast<size_t>(kin * SIMT_BK + b_kr) * p.N + n0 + b_nq;
    const int a_step_i = (THREADS / SIMT_BK) * p.K, b_step_i = (THREADS / (BN / 4)) * p.N;   // fit 32 bits
    const int b_step_kt = SIMT_BK * p.N;
    const bool b_col_ok = n0 + b_nq < p.N;

    auto issue_tile = [&](int kt, int stage) {
        if (kt < kt1) {
            const int k0 = kin * SIMT_BK;
#pragma unroll
            for (int i = 0; i < A_ELEMS; ++i) {
                const int row = a_row + i * (THREADS / SIMT_BK);   // 16 consecutive lanes = one row's 16 k
                const bool ok = m0 + row < p.M && k0 + a_k < p.K;
                cp_async_4(as_u32 + (stage * A_STAGE + a_k * AP + row) * 4, ok ? pa + i * a_step_i : p.A, ok ? 4u : 0u);
            }
#pragma unroll
            for (int i = 0; i < B_V4; ++i) {
                const int kr = b_kr + i * (THREADS / (BN / 4));
                const bool ok = b_col_ok && k0 + kr < p.K;
                cp_async_16(bs_u32 + (stage * B_STAGE + kr * BN + b_nq) * 4, ok ? pb + i * b_step_i : p.B, ok ? 16u : 0u);
            }
            pa += SIMT_BK;
            pb += b_step_kt;
            if (++kin == p.kt_per_item) {   // next item of the batch-reduce
            kin = 0;
            pa += p.stride_a - static_cast<long long>(p.kt_per_item) * SIMT_BK;
            pb += p.stride_b - static_cast<long long>(p.kt_per_item) * SIMT_BK * p.N;
        }
        }
        cp_async_commit();                                  // an empty group keeps the counts aligned
    };

#pragma unroll
    for (int s = 0; s < SIMT_STAGES - 1; ++s) issue_tile(kt0 + s, s);

    int stage = 0;
    for (int kt = kt0; kt < kt1; ++kt) {
        cp_async_wait_group<SIMT_STAGES - 2>();             // tile kt has landed (this thread's copies)
        __syncthreads();                                    // ... everyone's; and tile kt-1 is consumed
        int nstage = stage + SIMT_STAGES - 1;
        if (nstage >= SIMT_STAGES) nstage -= SIMT_STAGES;
        issue_tile(kt + SIMT_STAGES - 1, nstage);
        const float* as = As + stage * A_STAGE;
        const float* bs = Bs + stage * B_STAGE;
#pragma unroll
        for (int k = 0; k < SIMT_BK; ++k) {
            float a[TM], b[TN];
#pragma unroll
            for (int g = 0; g < GM; ++g) {
                const float4 v = *reinterpret_cast<const float4*>(as + k * AP + g * SM_STRIDE + ty * 4);
                a[4 * g] = v.x; a[4 * g + 1] = v.y; a[4 * g + 2] = v.z; a[4 * g + 3] = v.w;
            }
#pragma unroll
            for (int g = 0; g < GN; ++g) {
                const float4 v = *reinterpret_cast<const float4*>(bs + k * BN + g * SN_STRIDE + tx * 4);
                b[4 * g] = v.x; b[4 * g + 1] = v.y; b[4 * g + 2] = v.z; b[4 * g + 3] = v.w;
            }
            if (X2) {
#pragma unroll
                for (int i = 0; i < TM; ++i) {
                    const float2 a2 = make_float2(a[i], a[i]);
#pragma unroll
                    for (int j = 0; j < TN; j += 2) {
                        float2* c = reinterpret_cast<float2*>(&acc[i][j]);
                        *c = __ffma2_rn(a2, make_float2(b[j], b[j + 1]), *c);
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < TM; ++i)
#pragma unroll
                    for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
        }
        if (++stage == SIMT_STAGES) stage = 0;
    }
    cp_async_wait_group<0>();

    const bool to_partial = p.splits > 1;
    float* out = to_partial ? p.partial + (static_cast<size_t>(split) * p.gemms + gemm) * p.M * p.N
                            : p.C + gemm * p.stride_c;
#pragma unroll
    for (int gi = 0; gi < GM; ++gi)
#pragma unroll
        for (int ii = 0; ii < 4; ++ii) {
            const int gm = m0 + gi * SM_STRIDE + ty * 4 + ii;
            if (gm >= p.M) continue;
#pragma unroll
            for (int gj = 0; gj < GN; ++gj) {
                const int gn = n0 + gj * SN_STRIDE + tx * 4;
                if (gn >= p.N) continue;
                float4 v = make_float4(acc[4 * gi + ii][4 * gj], acc[4 * gi + ii][4 * gj + 1],
                                       acc[4 * gi + ii][4 * gj + 2], acc[4 * gi + ii][4 * gj + 3]);
                if (!to_partial && p.beta) {       // beta = 1: the accumulation tile starts from the stored C
                    const float4 cv = *reinterpret_cast<const float4*>(out + static_cast<size_t>(gm) * p.N + gn);
                    v.x += cv.x; v.y += cv.y; v.z += cv.z; v.w += cv.w;
                }
                if (!to_partial && p.epilogue) {
                    const float4 bv = __ldg(reinterpret_cast<const float4*>(p.bias + gn));
                    v.x = fmaxf(v.x + bv.x, 0.f);
                    v.y = fmaxf(v.y + bv.y, 0.f);
                    v.z = fmaxf(v.z + bv.z, 0.f);
                    v.w = fmaxf(v.w + bv.w, 0.f);
                }
                *reinterpret_cast<float4*>(out + static_cast<size_t>(gm) * p.N + gn) = v;
            }
        }
}

}  // namespace nk

namespace nk {

// Small FP32 GEMM: a problem whose whole K fits shared memory next to a 32 x 32 tile of C and
// whose tiles number a CTA or two per SM.  Such a problem is all latency: a pipelined K loop
// would pay a global-load round trip per k-tile, and K splits a second kernel.  Here a CTA issues
// every copy of its A and B slabs at once (one round trip), then its 256 threads multiply: four
// groups of 64 threads take a quarter of K each, a thread keeps 4 x 4 of C in registers
// (Algorithm 1's resident accumulator), and the four partial tiles meet in shared memory and are
// added in group order (k order: deterministic) by the first group, which applies beta, bias +
// ReLU and stores.  One launch, no workspace.
constexpr int SMALL_BM = 32, SMALL_BN = 32, SMALL_THREADS = 256, SMALL_KMAX = 512;
constexpr int SMALL_AP = SMALL_BM + 4;    // padded row of the transposed A slab As[k][m]
// the two slabs, or the three partial tiles that later take their place, whichever is larger
__host__ __device__ constexpr int simt_small_smem_bytes(int K) {
    return K * (SMALL_AP + SMALL_BN) * 4 > 3 * 64 * 16 * 4 ? K * (SMALL_AP + SMALL_BN) * 4 : 3 * 64 * 16 * 4;
}

struct SmallParams {
    int M, N, K;
    int beta, epilogue;
    const float* A;    // [M][K]
    const float* B;    // [K][N]
    const float* bias; // [N] or null
    float* C;          // [M][N]
};

__global__ void __launch_bounds__(SMALL_THREADS, 2) simt_f32_small_kernel(const SmallParams p) {
    extern __shared__ __align__(16) float small_smem[];
    float* As = small_smem;                       // [K][AP]
    float* Bs = small_smem + p.K * SMALL_AP;      // [K][BN]
    const uint32_t as_u32 = smem_u32(As), bs_u32 = smem_u32(Bs);
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int m0 = blockIdx.y * SMALL_BM, n0 = blockIdx.x * SMALL_BN;

    // A: 4-byte copies that transpose on the way.  A warp copies 8 consecutive k of 4 consecutive
    // rows per instruction (whole 32-byte sectors of global memory; the 32 shared-memory words
    // k * 36 + row fall into 32 different banks).  Warp w takes rows 4 w .. 4 w + 3, one k octet per step.
    {
        const int kq = lane & 7, r4 = lane >> 3;
        const int octets = (p.K + 7) >> 3;
        for (int idx = warp; idx < 8 * octets; idx += SMALL_THREADS / 32) {   // idx = row group (0..7) + 8 * k octet
            const int row = (idx & 7) * 4 + r4, k = (idx >> 3) * 8 + kq;
            const bool ok = m0 + row < p.M && k < p.K;
            if (k < p.K)
                cp_async_4(as_u32 + (k * SMALL_AP + row) * 4, ok ? p.A + static_cast<size_t>(m0 + row) * p.K + k : p.A, ok ? 4u : 0u);
        }
        // B: 16-byte copies, a row of the slab (32 columns) per 8 lanes
        const int nq = (t & 7) * 4;
        const bool col_ok = n0 + nq < p.N;          // N is a multiple of 4
        for (int k = t >> 3; k < p.K; k += SMALL_THREADS / 8)
            cp_async_16(bs_u32 + (k * SMALL_BN + nq) * 4, col_ok ? p.B + static_cast<size_t>(k) * p.N + n0 + nq : p.B, col_ok ? 16u : 0u);
        cp_async_commit();
        cp_async_wait_group<0>();
    }
    __syncthreads();

    const int g = t >> 6, tt = t & 63, ty = tt >> 3, tx = tt & 7;
    const int kper = (p.K + 3) >> 2;
    const int k0 = g * kper, k1 = min(p.K, k0 + kper);
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
#pragma unroll 4
    for (int k = k0; k < k1; ++k) {
        const float4 a = *reinterpret_cast<const float4*>(As + k * SMALL_AP + ty * 4);
        const float4 b = *reinterpret_cast<const float4*>(Bs + k * SMALL_BN + tx * 4);
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();                                // the slabs are consumed: the partial tiles take their place
    float* red = small_smem;                        // [3][64][16]
    if (g > 0) {
        float4* dst = reinterpret_cast<float4*>(red + ((g - 1) * 64 + tt) * 16);
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    }
    __syncthreads();
    if (g > 0) return;
#pragma unroll
    for (int s = 0; s < 3; ++s) {
        const float4* src = reinterpret_cast<const float4*>(red + (s * 64 + tt) * 16);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 v = src[i];
            acc[i][0] += v.x; acc[i][1] += v.y; acc[i][2] += v.z; acc[i][3] += v.w;
        }
    }
    const int gn = n0 + tx * 4;
    if (gn >= p.N) return;
    float4 bias4 = make_float4(0.f, 0.f, 0.f, 0.f);
    if (p.epilogue) bias4 = __ldg(reinterpret_cast<const float4*>(p.bias + gn));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int gm = m0 + ty * 4 + i;
        if (gm >= p.M) break;
        float4 v = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        float* dst = p.C + static_cast<size_t>(gm) * p.N + gn;
        if (p.beta) {       // beta = 1: the accumulation tile starts from the stored C
            const float4 cv = *reinterpret_cast<const float4*>(dst);
            v.x += cv.x; v.y += cv.y; v.z += cv.z; v.w += cv.w;
        }
        if (p.epilogue) {
            v.x = fmaxf(v.x + bias4.x, 0.f);
            v.y = fmaxf(v.y + bias4.y, 0.f);
            v.z = fmaxf(v.z + bias4.z, 0.f);
            v.w = fmaxf(v.w + bias4.w, 0.f);
        }
        *reinterpret_cast<float4*>(dst) = v;
    }
}

}  // namespace nk
