// Skinny GEMM (M <= 64 rows) on the tensor cores with the operands' roles swapped.
//
// With few rows of A a 128-row MMA tile is mostly zero padding, and what the kernel really does
// is stream B once.  Here the MMA computes C^T: its 128 "rows" are 128 COLUMNS of B (n), its N
// extent is M rounded up to 16, 32 or 64, so one MMA instruction (which costs the issuing thread
// the same whatever its shape) covers 128 columns of B instead of 64, a stage holds 16 KB of B and
// only MP x 128 bytes of A, and the accumulator (128 x MP FP32) is small enough for K splits to
// meet in one CTA of a cluster at almost no cost.  This is the tile loop's swap-AB decision
// (Algorithm 1's tile loop, re-aimed at a hardware tile that is 128 rows tall).
//
//   MMA A operand   B tile: 64 k x 128 n of the row-major B[K][N] (N contiguous: an MN-major
//                   operand, two 64-column slabs 8 KB apart), or 128 n x 64 k of the transposed
//                   Bt[N][K] (K-major)
//   MMA B operand   A tile: MP rows (m) x 64 k, K-major; rows beyond M arrive as zeros
//   accumulator     tensor-memory lane = n, column = m; the epilogue stores a column at a time,
//                   which is a row of C: 32 lanes write 32 consecutive n (coalesced)
//
// One unit (column tile, K split) per CTA; warp 0 produces, warp 1 issues MMAs, warps 2-5 drain.
// K splits are the CTAs of a cluster: splits 1..S-1 write their accumulators into the stage ring
// of split 0 (remote shared-memory stores), which adds them in split order and stores C; or,
// where that is not possible, FP32 partials go to the workspace and the split-K kernel adds them.
#pragma once
#include "umma_bf16.cuh"

namespace nk {

struct SwapParams {
    int M, N, K;
    int tiles_n;        // ceil(N / 128)
    int splits, kb_total, kb_per_split;
    int cluster;        // the K splits of a tile are the CTAs of one cluster
    int b_3d, b_kmajor;
    int epilogue, out_bf16, f16, bias_f32, beta;
    uint32_t idesc;
    const void* bias;
    void* C;
    float* partial;     // [splits][M][N] when the splits do not meet in a cluster
    unsigned int* status;
};

__host__ __device__ constexpr int swap_stage_bytes(int MP) { return 16384 + MP * 128; }
__host__ __device__ constexpr int swap_smem_bytes(int MP, int stages) { return stages * swap_stage_bytes(MP) + 1024 + 512; }
__host__ __device__ constexpr int swap_stages(int MP) { return MP == 64 ? 8 : 10; }

// One 32-row x 32-column piece of the accumulator (lane = n, v[j] = column m0 + j) -> rows m0 + j of C.
__device__ __forceinline__ void swap_store_piece(const SwapParams& p, uint32_t (&v)[32], int n, int m0, int mcount, float bias_n,
                                                 float* partial_dst) {
    if (n >= p.N) return;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (j >= mcount) break;                      // warp-uniform
        const int m = m0 + j;
        if (m >= p.M) break;
        float x = __uint_as_float(v[j]);
        const size_t o = static_cast<size_t>(m) * p.N + n;
        if (partial_dst) {
            partial_dst[o] = x;
            continue;
        }
        if (p.beta) {
            x += p.out_bf16 ? half_bits_to_f32(static_cast<const uint16_t*>(p.C)[o], p.f16) : static_cast<const float*>(p.C)[o];
        }
        if (p.epilogue) x = fmaxf(x + bias_n, 0.0f);
        if (p.out_bf16) static_cast<uint16_t*>(p.C)[o] = static_cast<uint16_t>(pack_half2(x, 0.0f, p.f16) & 0xFFFFu);
        else static_cast<float*>(p.C)[o] = x;
    }
}

template <int MP, bool CLUSTER>
__global__ void __launch_bounds__(192, 1)
umma_swap_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const SwapParams p) {
    static_assert(MP == 16 || MP == 32 || MP == 64, "padded M");
    constexpr int STAGES = swap_stages(MP);
    constexpr int STAGE = swap_stage_bytes(MP);
    constexpr int A_BYTES = MP * 128;                 // the A tile comes first in a stage (1024-byte aligned: MP >= 16 -> 2 KB)
    constexpr uint32_t TMEM_COLS = MP < 32 ? 32 : MP;
    constexpr int NCH = (MP + 31) / 32;               // 32-column pieces of the accumulator per warp

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + STAGES * STAGE;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    const uint32_t tfull_bar = bar_base + 8u * (2 * STAGES);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * STAGE + 8 * (2 * STAGES + 2));
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) {
        constexpr int NB = 2 * STAGES + 1;
        static_assert(NB <= 32, "one barrier per lane");
        if (lane < NB) mbar_init(bar_base + 8u * lane, 1);
        if (lane == 0) *abort_flag = 0;
        fence_mbar_init();
        __syncwarp();
    } else if (warp == 2 && lane == 0) {
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
        tmem_relinquish();
    }
    const uint32_t nthreads = blockDim.x;
    uint32_t tmem_base = 0;
    if (warp == 0) {
        asm volatile("bar.arrive 0, %0;" ::"r"(nthreads) : "memory");
    } else {
        tc_fence_before_sync();
        asm volatile("bar.sync 0, %0;" ::"r"(nthreads) : "memory");
        tc_fence_after_sync();
        tmem_base = *tmem_slot;
    }

    // unit = blockIdx.x: tile = unit / splits, split = unit % splits (the splits of a tile are consecutive CTAs: one cluster)
    const int tile = p.splits > 1 ? div_small(blockIdx.x, p.splits) : static_cast<int>(blockIdx.x);
    const int split = static_cast<int>(blockIdx.x) - tile * p.splits;
    const int kb0 = split * p.kb_per_split;
    const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
    const int n0 = tile * 128;

    auto give_up = [&](unsigned int code) {
        *abort_flag = 1;
        if (p.status) atomicCAS(p.status, 0u, code);
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer (warp-uniform issue, see elect_one)
        const uint32_t elected = elect_one();
        const bool b3d = p.b_3d != 0, b_kmajor = p.b_kmajor != 0;
        int stage = 0;
        uint32_t phase = 0;
        uint32_t sa = smem_base, fb = full_bar(0);
        bool ok = true;
        for (int kb = kb0; kb < kb1; ++kb) {
            const int kx = kb * UMMA_BK;
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
                if (lane == 0) give_up(0x100u + stage);
                ok = false;
                break;
            }
            const uint32_t sb = sa + A_BYTES;
            mbar_arrive_expect_tx_if(fb, STAGE, elected);
            tma_load_3d_if(sa, &tmap_a, fb, kx, 0, 0, elected);                   // MP rows of A, 128 bytes of k
            if (b_kmajor) {
                tma_load_3d_if(sb, &tmap_b, fb, kx, n0, 0, elected);              // 128 rows (n) of Bt, 128 bytes of k
            } else if (b3d) {
                tma_load_4d_if(sb, &tmap_b, fb, 0, kx, n0 >> 6, 0, elected);      // 64 k-rows of two 64-column slabs
            } else {
                tma_load_3d_if(sb, &tmap_b, fb, n0, kx, 0, elected);
                tma_load_3d_if(sb + 8192, &tmap_b, fb, n0 + 64, kx, 0, elected);
            }
            __syncwarp();
            sa += STAGE;
            fb += 8;
            if (++stage == STAGES) { stage = 0; phase ^= 1u; sa = smem_base; fb = full_bar(0); }
        }
        if (ok) {   // drain: every stage this warp filled has been consumed (a stage never filled passes at once)
            for (int s = 0; s < STAGES; ++s) {
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) break;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        const uint32_t elected = elect_one();
        const bool b_k = p.b_kmajor != 0;
        // MMA A operand = the B tile of the GEMM (after the A tile in the stage); MMA B operand = the A tile
        const uint64_t dw0 = b_k ? make_smem_desc(smem_base + A_BYTES, 16, 1024, 2) : make_smem_desc(smem_base + A_BYTES, 8192, 1024, 2);
        const uint64_t dx0 = make_smem_desc(smem_base, 16, 1024, 2);
        const uint32_t w_hi = static_cast<uint32_t>(dw0 >> 32), x_hi = static_cast<uint32_t>(dx0 >> 32);
        const uint32_t w_lo0 = static_cast<uint32_t>(dw0), x_lo0 = static_cast<uint32_t>(dx0);
        const uint32_t w_s = b_k ? 2u : 128u;
        constexpr uint32_t STAGE16 = STAGE >> 4;
        int stage = 0;
        uint32_t phase = 0, soff = 0, accumulate = 0u;
        for (int kb = kb0; kb < kb1; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) {
                if (lane == 0) give_up(0x300u + stage);
                break;
            }
            tc_fence_after_sync();
            const uint32_t w_lo = w_lo0 + soff, x_lo = x_lo0 + soff;
            umma_if<0>(tmem_base, w_lo, w_hi, x_lo, x_hi, p.idesc, accumulate, elected);
            umma_if<0>(tmem_base, w_lo + w_s, w_hi, x_lo + 2u, x_hi, p.idesc, 1u, elected);
            umma_if<0>(tmem_base, w_lo + 2 * w_s, w_hi, x_lo + 4u, x_hi, p.idesc, 1u, elected);
            umma_if<0>(tmem_base, w_lo + 3 * w_s, w_hi, x_lo + 6u, x_hi, p.idesc, 1u, elected);
            umma_commit_if(empty_bar(stage), elected);
            if (kb == kb1 - 1) umma_commit_if(tfull_bar, elected);
            accumulate = 1u;
            __syncwarp();
            soff += STAGE16;
            if (++stage == STAGES) { stage = 0; phase ^= 1u; soff = 0; }
        }
        if (kb1 <= kb0) umma_commit_if(tfull_bar, elected);      // empty K range
    } else {
        // ------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;
        const int n = n0 + quarter * 32 + lane;
        float bias_n = 0.0f;
        if (p.epilogue && n < p.N)
            bias_n = p.bias_f32 ? __ldg(static_cast<const float*>(p.bias) + n)
                                : half_bits_to_f32(__ldg(static_cast<const uint16_t*>(p.bias) + n), p.f16);
        bool ok = true;
        if (!mbar_wait(tfull_bar, 0u, abort_flag)) {
            if (lane == 0) give_up(0x400u);
            ok = false;
        }
        tc_fence_after_sync();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const bool empty_k = kb1 <= kb0;
        if (CLUSTER) {
            const uint32_t S = static_cast<uint32_t>(p.splits), rank = cluster_ctarank();
            cluster_arrive();
            cluster_wait();                          // every K loop of the cluster is over: split 0's ring may be overwritten
            if (ok && rank != 0) {
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(taddr + c * 32, v);
                    tmem_ld_wait();
                    if (empty_k) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = 0u;
                    }
                    const uint32_t dst = map_to_cta(smem_base + (((rank - 1u) * 4u + quarter) * NCH + c) * 4096u, 0u);
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        if (c * 32 + 4 * g < MP)
                            st_cluster_v4(dst + g * 512 + ((lane ^ g) << 4), v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                }
            }
            cluster_arrive();
            cluster_wait();                          // every accumulator has landed in split 0
            if (ok && rank == 0) {
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(taddr + c * 32, v);
                    tmem_ld_wait();
                    if (empty_k) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = 0u;
                    }
                    // split order 1 .. S-1 after split 0's own sum
#pragma unroll 1
                    for (uint32_t r = 1; r < S; ++r) {
                        const uint8_t* slot = gen_base + (((r - 1u) * 4u + quarter) * NCH + c) * 4096u;
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            if (c * 32 + 4 * g < MP) {
                                const uint4 t4 = *reinterpret_cast<const uint4*>(slot + g * 512 + ((lane ^ g) << 4));
                                add2_f32(v[4 * g], v[4 * g + 1], t4.x, t4.y);
                                add2_f32(v[4 * g + 2], v[4 * g + 3], t4.z, t4.w);
                            }
                    }
                    swap_store_piece(p, v, n, c * 32, MP - c * 32 < 32 ? MP - c * 32 : 32, bias_n, nullptr);
                }
            }
        } else if (ok) {
            float* pdst = p.splits > 1 ? p.partial + static_cast<size_t>(split) * p.M * p.N : nullptr;
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(taddr + c * 32, v);
                tmem_ld_wait();
                if (empty_k) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0u;
                }
                swap_store_piece(p, v, n, c * 32, MP - c * 32 < 32 ? MP - c * 32 : 32, bias_n, pdst);
            }
        }
    }
    if (CLUSTER && warp < 2) {
        // the cluster barriers count every thread: the producer and the issuer pass both of them here
        cluster_arrive();
        cluster_wait();
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace nk
