// BF16 x BF16 -> FP32 GEMM on the 5th-generation tensor cores.
//
// Structure (Algorithm 1 of the paper, re-expressed for sm_100a): a persistent
// CTA walks output tiles; for each tile the accumulator stays resident in tensor
// memory over the whole K loop (Algorithm 1: the C sub-block is held across the
// batch-reduce and K loops), operands are staged by TMA into a ring of swizzled
// shared-memory tiles while earlier stages are being multiplied (the software
// pipelining of Algorithm 3, AMX branch), and bias + ReLU are applied to the
// accumulator before the single store of C (Section 6, "MLP").
//
// Warp roles (320 threads):
//   warp 0      TMA producer: A tile 128 x 64 (K-major), B tile 64 x BN (N-major)
//   warp 1      MMA issuer and TMEM owner: 4 x tcgen05.mma 128 x BN x 16 per stage
//   warps 2-5   epilogue: tcgen05.ld -> (+bias, ReLU, cvt) -> global stores; two
//               TMEM accumulators so tile t's epilogue overlaps tile t+1's K loop
//   warps 6-9   with VNNI-blocked B, re-layout: the producer's TMA box brings the
//               [k/2][n][2] blocks of a stage as they are; these warps transpose them
//               as 32-bit words, in place, into the K-major swizzled stage (the
//               in-kernel counterpart of the paper's software-pipelined pack step,
//               in the opposite direction); warps 6-7 take the even stages, 8-9 the odd
//               ones.  In a CTA that delivers a single tile they are also the second
//               half of the epilogue (half of the columns each)
//
// Every mbarrier wait is bounded; a role that gives up raises the CTA's abort
// flag and the device status word, the other roles fall out of their loops, and
// the CTA frees its TMEM and exits.
//
// Split-K inside a thread-block cluster (CLUSTER_REDUCE): the K splits of one tile are the CTAs
// of one cluster, one unit per CTA.  After its K loop every CTA sends the 32 x 32 pieces of its
// accumulator that other CTAs own straight into their shared memory (distributed shared memory;
// they land in the stage ring, which is idle by then) and counts them in on the receiving warp's
// mbarrier; every CTA adds the pieces it owns in split order, applies the epilogue and stores them.  No partial ever
// goes to global memory and there is no second kernel.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include "aux_kernels.cuh"
#include "ptx.cuh"

namespace nk {

constexpr int UMMA_BM = 128;
constexpr int UMMA_BK = 64;
constexpr int UMMA_A_STAGE_BYTES = UMMA_BM * UMMA_BK * 2;  // 16 KB
constexpr int UMMA_THREADS = 320;   // producer, MMA issuer, 4 epilogue warps, 4 re-layout / second-epilogue warps

struct UmmaParams {
    int M, N, K;
    int tiles_m, tiles_n;
    int splits;         // K splits; > 1 writes FP32 partials to `partial`
    int kb_total;       // batch * kb_per_item: k-blocks of the whole reduction
    int kb_per_item;    // ceil(K / 64): k-blocks of one (A_b, B_b) pair of the batch-reduce
    int beta;           // 1: the old C is added before the epilogue (Algorithm 1's beta.C)
    int gemms;          // independent GEMMs in one launch (batched matmul): C_g = A_g . B_g; else 1
    long long stride_c; // elements from C_g to C_g+1
    int c_blocked;      // C is stored as [M/32][N/32][32][32]: each 32 x 32 chunk is one block
    int tma_store;      // C (row-major, no beta, no partials) leaves through TMA stores of 32 x 32 boxes
    int cluster_reduce; // the K splits of a tile are the CTAs of one cluster and meet in shared memory
    int kb_per_split;   // ceil(kb_total / splits)
    int group_m;        // raster: this many M tiles sweep N together
    int serpentine;     // raster: every other group of M tiles sweeps N in the opposite direction
    int k_serpentine;   // pair kernel, no batch: every other whole tile of a pair walks K downwards, so that a
                        // wave begins with the part of the shared strips that the wave before it read last
    int a_blocked;      // A tensor map is the 4-D blocked view
    int b_3d;           // B tensor map is the 3-D (n-in-slab, k, slab) view: one box per stage
    int b_kmajor;       // B is stored transposed, Bt[N][K]: its tiles are K-major like A's, one box per stage
    int epilogue;       // 0 none, 1 bias + ReLU
    int out_bf16;       // C is 16 bits wide (the operands' type), else FP32
    int f16;            // the 16-bit type of A, B, bias (and C) is IEEE binary16 instead of BF16
    uint32_t idesc;     // tcgen05 instruction descriptor
    const void* bias;   // BF16 [N] or null
    void* C;            // [M][N] FP32 or BF16
    float* partial;     // [splits][M][N] when splits > 1; [tail tile][segment][tile rows][BN] in tail mode
    int tail_from;      // stream-K tail (pair kernel): tiles >= tail_from, the last, partial wave, are shared out by k-blocks; else -1
    int sk_share;       // k-blocks of the tail each pair takes: pair i has [i * sk_share, (i + 1) * sk_share) of the tail tiles' k-blocks laid end to end
    int sk_max_segs;    // partial slabs reserved per tail tile (a tile is cut into at most this many segments)
    int bias_f32;       // the bias vector is FP32 although the operands are not (split-FP32 and quantised plans)
    int dequant;        // the accumulator holds INT32 sums: convert to FP32 and multiply by `scale` before the epilogue
    float scale;
    int acc_s32;        // the accumulator holds INT32 sums (INT8 operands): K splits are added as integers
    int item_remap;     // batch item i multiplies A item (item_map_a >> 4i) & 15 by B item (item_map_b >> 4i) & 15
    uint32_t item_map_a, item_map_b;
    unsigned int* status;
};

// The (A item, B item) pair of batch item `item`: the item itself, or, for plans that multiply
// cross terms of split operands, the pair the plan's 4-bit tables name.
__device__ __forceinline__ void umma_item_pair(const UmmaParams& p, int item, int& ia, int& ib) {
    ia = ib = item;
    if (p.item_remap) {
        ia = static_cast<int>((p.item_map_a >> (4 * item)) & 15u);
        ib = static_cast<int>((p.item_map_b >> (4 * item)) & 15u);
    }
}

__host__ __device__ constexpr int umma_b_stage_bytes(int BN) { return BN * UMMA_BK * 2; }
__host__ __device__ constexpr int umma_stage_bytes(int BN) {
    return UMMA_A_STAGE_BYTES + umma_b_stage_bytes(BN);
}
constexpr uint32_t UMMA_RECV_BAR_OFFSET = 264;    // in the barrier block, after the raw-block barriers: one per epilogue warp of a cluster split-K CTA
constexpr uint32_t UMMA_RAW_BAR_OFFSET = 200;     // in the barrier block: after full/empty/tmem barriers (<= 168 B) and the cluster barrier (192)
constexpr int UMMA_EPI_STAGING = 4 * 2 * 4096;   // two 32 x 32 FP32 chunks per epilogue warp (1024-byte aligned: TMA store source)
__host__ __device__ constexpr int umma_smem_bytes(int BN, int stages) {
    return stages * umma_stage_bytes(BN) + 1024 /*alignment slack*/ + UMMA_EPI_STAGING + 384 /*barriers*/;
}
// cluster split-K: one 4 KB slot per (32 x 32 piece this CTA owns, split it comes from); the pieces of
// a CTA's 128 x BN accumulator are shared out over the splits, so a CTA's slots never exceed one
// accumulator (BN * 512 bytes), which fits the stage ring of every variant

// a / b for 0 <= a < 2^24, 0 < b < 2^24 without the integer-division routine (some forty dependent
// instructions; the producer decodes its first unit before it can issue the first load, and on a
// short problem that wait is visible): a single-precision estimate, then one exact correction step.
__device__ __forceinline__ int div_small(int a, int b) {
    int q = __float2int_rz(__fdividef(__int2float_rz(a), __int2float_rz(b)));
    int r = a - q * b;             // the estimate is off by one at most (the loops run once or not at all)
    while (r < 0) { --q; r += b; }
    while (r >= b) { ++q; r -= b; }
    return q;
}

// tile id -> (m block, n block): groups of `group_m` M tiles sweep across N so
// that CTAs running at the same time share A rows and B columns in L2.
__device__ __forceinline__ void umma_tile_coords(const UmmaParams& p, int tile, int& mb, int& nb) {
    const int per_group = p.group_m * p.tiles_n;
    const int g = div_small(tile, per_group);
    const int within = tile - g * per_group;
    const int first_m = g * p.group_m;
    const int gm = min(p.group_m, p.tiles_m - first_m);
    nb = div_small(within, gm);
    mb = first_m + within - nb * gm;
    // odd groups sweep N backwards: the B columns a group ends on are the ones the next group starts with
    if (p.serpentine && (g & 1)) nb = p.tiles_n - 1 - nb;
}

// unit id -> (independent GEMM, tile, K split)
__device__ __forceinline__ void umma_decode_unit(const UmmaParams& p, int unit, int& tile, int& split, int& gemm) {
    gemm = 0;
    int u = unit;
    if (p.gemms > 1) {
        const int per_gemm = p.tiles_m * p.tiles_n * p.splits;
        gemm = div_small(unit, per_gemm);
        u = unit - gemm * per_gemm;
    }
    tile = u;
    split = 0;
    if (p.splits > 1) {
        tile = div_small(u, p.splits);
        split = u - tile * p.splits;
    }
}

// Where the FP32 partial of a chunk goes: base[(row0 + r) * ld + col0 + c], clipped to rows x cols.
struct PartialDst {
    float* base;
    int ld, row0, col0, rows, cols;
};

// Two FP32 adds in one instruction (add.rn.f32x2: the same IEEE results as two scalar adds).
__device__ __forceinline__ void add2_f32(uint32_t& a0, uint32_t& a1, uint32_t b0, uint32_t b1) {
    asm("{\n\t.reg .b64 x, y;\n\tmov.b64 x, {%0, %1};\n\tmov.b64 y, {%2, %3};\n\tadd.rn.f32x2 x, x, y;\n\tmov.b64 {%0, %1}, x;\n\t}"
        : "+r"(a0), "+r"(a1)
        : "r"(b0), "r"(b1));
}

// bias + ReLU (Section 6, the MLP layer) on one 32 x 32 chunk held as a row per lane.  `bias_sm`:
// the chunk's 32 bias values as FP32 in shared memory (parked there by umma_park_bias while the K
// loop was still running); without it the values come from global memory, 16-bit or FP32.
__device__ __forceinline__ void umma_chunk_bias_relu(const UmmaParams& p, uint32_t (&v)[32], int col0,
                                                     const float* bias_sm) {
    if (!p.epilogue) return;
    if (bias_sm) {
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const uint4 b = reinterpret_cast<const uint4*>(bias_sm)[g];
            add2_f32(v[4 * g], v[4 * g + 1], b.x, b.y);
            add2_f32(v[4 * g + 2], v[4 * g + 3], b.z, b.w);
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(fmaxf(__uint_as_float(v[i]), 0.0f));
    } else if (p.bias_f32) {
        const float4* bsrc = reinterpret_cast<const float4*>(static_cast<const float*>(p.bias) + col0);
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            if (col0 + 4 * g >= p.N) break;
            const float4 b = __ldg(bsrc + g);
            v[4 * g] = __float_as_uint(fmaxf(__uint_as_float(v[4 * g]) + b.x, 0.0f));
            v[4 * g + 1] = __float_as_uint(fmaxf(__uint_as_float(v[4 * g + 1]) + b.y, 0.0f));
            v[4 * g + 2] = __float_as_uint(fmaxf(__uint_as_float(v[4 * g + 2]) + b.z, 0.0f));
            v[4 * g + 3] = __float_as_uint(fmaxf(__uint_as_float(v[4 * g + 3]) + b.w, 0.0f));
        }
    } else {
        const uint4* bsrc = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(p.bias) + col0);
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            if (col0 + 8 * g >= p.N) break;
            const uint4 b = __ldg(bsrc + g);
            const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float x0 = __uint_as_float(v[8 * g + 2 * j]) + half_bits_to_f32(w[j] & 0xFFFFu, p.f16);
                float x1 = __uint_as_float(v[8 * g + 2 * j + 1]) + half_bits_to_f32(w[j] >> 16, p.f16);
                v[8 * g + 2 * j] = __float_as_uint(fmaxf(x0, 0.0f));
                v[8 * g + 2 * j + 1] = __float_as_uint(fmaxf(x1, 0.0f));
            }
        }
    }
}

// One 32 x 32 chunk in the layout a TMA store of a 32 x 32 box reads: FP32 rows of 128 bytes with the
// 128-byte swizzle (16-byte group g of row t at group g ^ (t & 7)), 16-bit rows of 64 bytes with the
// 64-byte swizzle (group g at g ^ ((t >> 1) & 3)); both conflict-free for a row per lane.
template <bool F16>
__device__ __forceinline__ void umma_write_tile16(const uint32_t (&v)[32], int lane, uint8_t* tile) {
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint4 o;
        o.x = pack_half2(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1]), F16);
        o.y = pack_half2(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]), F16);
        o.z = pack_half2(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]), F16);
        o.w = pack_half2(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]), F16);
        *reinterpret_cast<uint4*>(tile + lane * 64 + ((g ^ ((lane >> 1) & 3)) << 4)) = o;
    }
}
__device__ __forceinline__ void umma_write_store_tile(const UmmaParams& p, const uint32_t (&v)[32], int lane, uint8_t* tile) {
    if (p.out_bf16) {
        if (p.f16) umma_write_tile16<true>(v, lane, tile);
        else umma_write_tile16<false>(v, lane, tile);
    } else {
#pragma unroll
        for (int g = 0; g < 8; ++g)
            *reinterpret_cast<uint4*>(tile + lane * 128 + ((g ^ (lane & 7)) << 4)) =
                make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
    }
}

// Epilogue for one 32 x 32 chunk of the accumulator: lane t holds row `row0 + t`, columns
// col0 .. col0+31 as FP32 bit patterns.  Either the raw FP32 partial of a K split, or bias +
// ReLU (Section 6, "MLP") followed by the single store of C as FP32 or BF16 (one RNE rounding).
// FP32 rows are transposed through a 4 KB per-warp shared-memory buffer (16-byte chunk g of
// row t kept at chunk g ^ (t & 7): conflict-free both ways) so that every store instruction
// writes four whole 128-byte row segments instead of 32 scattered 16-byte pieces.  BF16 rows
// (64 bytes each) are stored directly.  Columns are predicated in groups (N is a multiple of 8).
//
// `staging` is the warp's 8 KB of shared memory: two 4 KB (FP32) or two 2 KB (BF16) tiles used
// alternately (`parity`) as TMA-store sources; with BF16 output the bias slice of the tile
// (`bias_smem`, one FP32 value per tile column, fetched while the K loop was still running) sits
// behind them.
__device__ __forceinline__ void umma_store_chunk(const UmmaParams& p, const CUtensorMap* tmap_c, uint32_t (&v)[32],
                                                 int row0, int lane, int col0, int split, int gemm, bool empty_k,
                                                 uint8_t* staging, int parity, const float* bias_smem,
                                                 const PartialDst* pd) {
    const bool to_partial = pd != nullptr;      // a K split's FP32 partial instead of the final C
    const bool tma_store = p.tma_store && !to_partial;
    if (col0 >= p.N || row0 >= p.M) return;           // warp-uniform
    const int row = row0 + lane;
    const size_t c_base = static_cast<size_t>(gemm) * p.stride_c;   // this GEMM's C inside the batch
    // element offset of (row0 + r, col0 + c) inside C: row-major, or one 32 x 32 block per chunk
    const size_t blk_base = (static_cast<size_t>(row0 >> 5) * (p.N >> 5) + (col0 >> 5)) * 1024;
    auto c_off = [&](int r, int c) -> size_t {
        return p.c_blocked ? blk_base + r * 32 + c : static_cast<size_t>(row0 + r) * p.N + col0 + c;
    };
    if (empty_k) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = 0u;
    }
    if (p.dequant && !to_partial) {   // a K split's partial stays an INT32 sum; the reduce kernel converts
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__int2float_rn(static_cast<int>(v[i])) * p.scale);
    }
    if (!to_partial && p.beta && row < p.M) {
        // beta = 1: the accumulation tile starts from the stored C (Algorithm 1 loads the C
        // sub-block before the K loop; adding it here, in FP32, gives the same sum)
        if (p.out_bf16) {
            const uint4* csrc = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(p.C) + c_base + c_off(lane, 0));
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                if (col0 + 8 * g >= p.N) break;
                const uint4 c = csrc[g];
                const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    v[8 * g + 2 * j] = __float_as_uint(__uint_as_float(v[8 * g + 2 * j]) + half_bits_to_f32(w[j] & 0xFFFFu, p.f16));
                    v[8 * g + 2 * j + 1] = __float_as_uint(__uint_as_float(v[8 * g + 2 * j + 1]) + half_bits_to_f32(w[j] >> 16, p.f16));
                }
            }
        } else {
            const uint4* csrc = reinterpret_cast<const uint4*>(static_cast<const float*>(p.C) + c_base + c_off(lane, 0));
#pragma unroll
            for (int g = 0; g < 8; ++g) {
                if (col0 + 4 * g >= p.N) break;
                const uint4 c = csrc[g];
                v[4 * g] = __float_as_uint(__uint_as_float(v[4 * g]) + __uint_as_float(c.x));
                v[4 * g + 1] = __float_as_uint(__uint_as_float(v[4 * g + 1]) + __uint_as_float(c.y));
                v[4 * g + 2] = __float_as_uint(__uint_as_float(v[4 * g + 2]) + __uint_as_float(c.z));
                v[4 * g + 3] = __float_as_uint(__uint_as_float(v[4 * g + 3]) + __uint_as_float(c.w));
            }
        }
    }
    if (!to_partial) umma_chunk_bias_relu(p, v, col0, bias_smem);
    if (!to_partial && p.out_bf16 && tma_store) {
        // BF16 rows (64 bytes) -> staging, 16-byte chunk g of row t at chunk g ^ ((t >> 1) & 3) (the
        // 64-byte swizzle: conflict-free stores) -> one TMA store of the 32 x 32 box
        uint8_t* tile = staging + parity * 2048;
        if (lane == 0) bulk_wait_read<1>();          // the store issued two chunks ago has read this tile
        __syncwarp();
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            uint4 o;
            o.x = pack_half2(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1]), p.f16);
            o.y = pack_half2(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]), p.f16);
            o.z = pack_half2(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]), p.f16);
            o.w = pack_half2(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]), p.f16);
            *reinterpret_cast<uint4*>(tile + lane * 64 + ((g ^ ((lane >> 1) & 3)) << 4)) = o;
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            tma_store_3d(tmap_c, smem_u32(tile), col0, row0, gemm);
            bulk_commit();
        }
        return;
    }
    if (!to_partial && p.out_bf16) {
        if (row >= p.M) return;
        uint16_t* dst = static_cast<uint16_t*>(p.C) + c_base + c_off(lane, 0);
#pragma unroll
        for (int g = 0; g < 4; ++g)
            if (col0 + 8 * g < p.N) {
                uint4 o;
                o.x = pack_half2(__uint_as_float(v[8 * g]), __uint_as_float(v[8 * g + 1]), p.f16);
                o.y = pack_half2(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]), p.f16);
                o.z = pack_half2(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]), p.f16);
                o.w = pack_half2(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]), p.f16);
                *reinterpret_cast<uint4*>(dst + 8 * g) = o;
            }
        return;
    }
    // FP32: registers -> staging (row per lane, 16-byte chunk g of row t at chunk g ^ (t & 7): the
    // 128-byte swizzle) -> global, either as one TMA store of the 32 x 32 box (the TMA unit writes
    // whole lines and clips the ragged edge; the warp only pays eight shared-memory stores), or with
    // per-thread stores of four 128-byte row segments per instruction.
    staging += parity * 4096;
    if (tma_store) {
        // two tiles used alternately: the store issued two chunks ago has read this one
        if (lane == 0) bulk_wait_read<1>();
        __syncwarp();
    } else if (p.tma_store) {
        // a K split's partial in a plan whose whole tiles leave by TMA store (tail-wave mode): the
        // stores of the previous whole tile may still be reading either staging tile (16-bit C keeps
        // both inside the first 4 KB), so all of them must have read their source first
        if (lane == 0) bulk_wait_read<0>();
        __syncwarp();
    }
#pragma unroll
    for (int g = 0; g < 8; ++g)
        *reinterpret_cast<uint4*>(staging + lane * 128 + ((g ^ (lane & 7)) << 4)) =
            make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
    if (tma_store) {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            tma_store_3d(tmap_c, smem_u32(staging), col0, row0, gemm);
            bulk_commit();
        }
        return;
    }
    __syncwarp();
    const int c = lane & 7, rsub = lane >> 3;
    if (to_partial) {
        const bool col_in = pd->col0 + 4 * c < pd->cols;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = 4 * i + rsub;
            const uint4 val = *reinterpret_cast<const uint4*>(staging + r * 128 + ((c ^ (r & 7)) << 4));
            if (col_in && pd->row0 + r < pd->rows)
                *reinterpret_cast<uint4*>(pd->base + static_cast<size_t>(pd->row0 + r) * pd->ld + pd->col0 + 4 * c) = val;
        }
        __syncwarp();
        return;
    }
    float* out = static_cast<float*>(p.C) + c_base;
    const bool col_ok = col0 + 4 * c < p.N;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + rsub;
        const uint4 val = *reinterpret_cast<const uint4*>(staging + r * 128 + ((c ^ (r & 7)) << 4));
        if (col_ok && row0 + r < p.M) *reinterpret_cast<uint4*>(out + c_off(r, 4 * c)) = val;
    }
    __syncwarp();   // the buffer is reused by the next chunk
}

// The bias slice of a tile (BN values from column col_tile0 on), widened to FP32 and parked at `dst`
// in shared memory (BN * 4 bytes) before the wait for the accumulator, so that its global latency
// hides behind the K loop and the chunks pay shared-memory reads only.  Null without an epilogue.
template <int BN>
__device__ __forceinline__ const float* umma_park_bias(const UmmaParams& p, float* dst, int col_tile0, int lane) {
    if (!p.epilogue) return nullptr;
    if (lane < BN / 8) {
        const int col = col_tile0 + 8 * lane;        // N is a multiple of 8: eight columns are in or out together
        float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
        if (col < p.N) {
            if (p.bias_f32) {
                lo = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(p.bias) + col));
                hi = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(p.bias) + col) + 1);
            } else {
                const uint4 b = __ldg(reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(p.bias) + col));
                lo = make_float4(half_bits_to_f32(b.x & 0xFFFFu, p.f16), half_bits_to_f32(b.x >> 16, p.f16),
                                 half_bits_to_f32(b.y & 0xFFFFu, p.f16), half_bits_to_f32(b.y >> 16, p.f16));
                hi = make_float4(half_bits_to_f32(b.z & 0xFFFFu, p.f16), half_bits_to_f32(b.z >> 16, p.f16),
                                 half_bits_to_f32(b.w & 0xFFFFu, p.f16), half_bits_to_f32(b.w >> 16, p.f16));
            }
        }
        reinterpret_cast<float4*>(dst)[2 * lane] = lo;
        reinterpret_cast<float4*>(dst)[2 * lane + 1] = hi;
    }
    __syncwarp();
    return dst;
}

// In the chunk-at-a-time epilogue the slice fits behind the staging tiles only with a 16-bit C
// (two 2 KB tiles): parked at staging + 4096, else read from global memory chunk by chunk.
template <int BN>
__device__ __forceinline__ const float* umma_fetch_bias(const UmmaParams& p, uint8_t* staging, int col_tile0, int lane) {
    if (!p.out_bf16 || p.splits > 1) return nullptr;
    return umma_park_bias<BN>(p, reinterpret_cast<float*>(staging + 4096), col_tile0, lane);
}

// Epilogue of a CTA that has a single tile to deliver (a problem of one wave or less), C row-major and
// stored by TMA.  By the time the accumulator is complete every stage of the operand ring has been
// consumed and nothing will be loaded again, so the ring serves as store staging: a warp converts
// ALL its chunks first (a tile each, `tiles` = the warp's region of the ring, 1024-byte aligned), pays
// one proxy fence and one warp barrier, and then issues its box stores back to back as one bulk
// group.  The chunk-at-a-time scheme costs ~550 clocks per chunk in fence, barrier, issue and
// buffer-reuse waits; this one ~150 per chunk plus ~300 once.  Two warps share each quarter of the
// accumulator's rows (tensor-memory lanes are tied to warp % 4): this one takes chunks c0 .. c1-1.
template <int BN>
__device__ __forceinline__ void umma_epilogue_oneshot(const UmmaParams& p, const CUtensorMap* tmap_c, uint32_t taddr,
                                                      uint8_t* tiles, int row0, int col_tile0, int gemm, int lane,
                                                      bool empty_k, const float* bias_sm, int c0, int c1) {
    const uint32_t tile_bytes = p.out_bf16 ? 2048u : 4096u;
    if (row0 >= p.M) return;
#pragma unroll 1
    for (int c = c0; c < c1; c += 2) {
        if (col_tile0 + c * 32 >= p.N) break;        // warp-uniform
        const bool two = c + 1 < c1 && col_tile0 + c * 32 + 32 < p.N;
        uint32_t v0[32], v1[32];
        tmem_ld_32x32(taddr + c * 32, v0);
        if (two) tmem_ld_32x32(taddr + c * 32 + 32, v1);
        tmem_ld_wait();
        if (empty_k) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v0[i] = v1[i] = 0u;
        }
        if (p.dequant) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                v0[i] = __float_as_uint(__int2float_rn(static_cast<int>(v0[i])) * p.scale);
                v1[i] = __float_as_uint(__int2float_rn(static_cast<int>(v1[i])) * p.scale);
            }
        }
        umma_chunk_bias_relu(p, v0, col_tile0 + c * 32, bias_sm ? bias_sm + c * 32 : nullptr);
        umma_write_store_tile(p, v0, lane, tiles + (c - c0) * tile_bytes);
        if (two) {
            umma_chunk_bias_relu(p, v1, col_tile0 + c * 32 + 32, bias_sm ? bias_sm + c * 32 + 32 : nullptr);
            umma_write_store_tile(p, v1, lane, tiles + (c - c0 + 1) * tile_bytes);
        }
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
#pragma unroll 1
        for (int c = c0; c < c1; ++c)
            if (col_tile0 + c * 32 < p.N) tma_store_3d(tmap_c, smem_u32(tiles + (c - c0) * tile_bytes), col_tile0 + c * 32, row0, gemm);
        bulk_commit();
    }
}

// Epilogue of a cluster split-K CTA.  Its accumulator (128 rows x BN columns, tensor-memory
// columns 0..BN-1) is cut into 4 * BN / 32 pieces, piece u = quarter * (BN / 32) + chunk; the CTAs
// that hold the S splits of the same rows have cluster ranks rank0 + s * rank_step.  Piece u
// belongs to split u % S; the other splits write theirs into slot (u / S) * S + source split of
// the owner's stage ring (idle by then), the owner's own contribution stays in tensor memory.
//   barrier  every CTA of the cluster has finished its K loop: the rings may be overwritten
//   send     tcgen05.ld -> asynchronous remote shared-memory stores straight from the registers, a
//            warp writing 512 contiguous bytes per instruction (16-byte group g of row t at
//            g * 512 + (t ^ g) * 16: conflict-free when the owner reads it back), every store counted
//            in on the receiving warp's mbarrier `recv_bar`.  The SM-to-SM path moves 16-23 bytes per
//            clock per CTA whatever the method (bulk copies, remote loads, remote stores; measured),
//            so what counts is that all the pieces are in flight at once and nothing waits in between
//   wait     each warp waits on its own mbarrier for the pieces it owns (armed with their byte
//            count before the first barrier); no second barrier of the whole cluster
//   reduce   every owned piece is summed in split order (the result does not depend on timing;
//            INT32 sums are added as integers), gets the epilogue, and all the owned chunks leave
//            as one batch of TMA stores staged behind the slots
// Every thread of the cluster passes the barrier, also in a CTA where a wait gave up (`ok` false);
// the warps that then wait for its pieces give up after their bounded wait.  A CTA leaves only
// after all its warps have what they wait for, so nothing is written into an exited CTA.
// `bias_sm`: the tile's bias slice as FP32 in shared memory (umma_park_bias), or null.
template <int BN>
__host__ __device__ constexpr uint32_t umma_cluster_slot_bytes() { return BN * 512u; }

// Eight warps run this, two per quarter of the accumulator's rows (tensor-memory lanes are tied to
// warp % 4); `half` (0 or 1) picks the warp's half of the BN / 32 chunks.  Plans that cannot store
// by TMA (beta, blocked C) let the second set of warps send only: the first set then reduces and
// stores all the owned chunks one at a time through its staging tiles.
template <int BN>
__device__ __forceinline__ bool umma_cluster_epilogue(const UmmaParams& p, const CUtensorMap* tmap_c, uint32_t tmem_base,
                                                      uint32_t ring, uint8_t* ring_gen, uint8_t* staging,
                                                      const float* bias_sm, int quarter, int half, int lane, uint32_t S,
                                                      uint32_t split, uint32_t rank0, uint32_t rank_step, int row_cta0,
                                                      int col_tile0, int gemm, bool ok, uint32_t recv_bar0,
                                                      volatile uint32_t* abort_flag) {
    constexpr uint32_t NC = BN / 32, HC = NC / 2;
    const uint32_t lane_tmem = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t c_lo = half * HC, c_hi = c_lo + HC;
    const uint32_t my_bar = recv_bar0 + 8u * (quarter * 2 + half);
    // pieces of this warp's chunk range that this CTA owns: each brings 4 KB from every other split
    uint32_t owned = 0;
#pragma unroll
    for (uint32_t c = 0; c < HC; ++c) owned += ((quarter * NC + c_lo + c) & (S - 1u)) == split ? 1u : 0u;
    if (lane == 0) mbar_arrive_expect_tx(my_bar, owned * (S - 1u) * 4096u);
    cluster_arrive();
    cluster_wait();
    if (ok) {
#pragma unroll 1
        for (uint32_t c = c_lo; c < c_hi; ++c) {
            const uint32_t u = quarter * NC + c, owner = u & (S - 1u);      // S is 2, 4 or 8
            if (owner == split) continue;                // mine: stays in tensor memory (warp-uniform)
            uint32_t v[32];
            tmem_ld_32x32(tmem_base + c * 32 + lane_tmem, v);
            tmem_ld_wait();
            const uint32_t orank = rank0 + owner * rank_step;
            const uint32_t dst = map_to_cta(ring + ((u & ~(S - 1u)) + split) * 4096u, orank);
            const uint32_t obar = map_to_cta(my_bar, orank);     // the same (quarter, half) warp of the owner
#pragma unroll
            for (int g = 0; g < 8; ++g)
                st_async_cluster_v4(dst + g * 512 + ((lane ^ g) << 4), v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3], obar);
        }
    }
    if (!ok) return false;
    const bool batched = p.tma_store != 0;
    // the pieces this warp will reduce have landed: its own range, and without batched stores (set 0
    // reduces every chunk of its rows) the other half's range as well
    if (!mbar_wait_cluster(my_bar, 0u, abort_flag)) return false;
    if (!batched && !mbar_wait_cluster(recv_bar0 + 8u * (quarter * 2 + (half ^ 1)), 0u, abort_flag)) return false;
    if (!batched && half != 0) return true;
    const uint32_t r_lo = batched ? c_lo : 0u, r_hi = batched ? c_hi : NC;
    // store tiles of the owned chunks: behind the receive slots, max(1, HC / S) per warp
    constexpr uint32_t kSlots = umma_cluster_slot_bytes<BN>();
    const uint32_t per_warp = HC / S > 0 ? HC / S : 1u;
    const uint32_t tile_bytes = p.out_bf16 ? 2048u : 4096u;
    uint8_t* tiles = ring_gen + kSlots + (quarter * 2 + half) * per_warp * 4096u;
    const int row0 = row_cta0 + quarter * 32;
    uint32_t ntiles = 0;
    int parity = 0;
    bool reduced = false;
    if constexpr (HC >= 4) {
        if (batched && S == 2u) {
            // Two splits, two owned chunks per warp (c_lo + split and the next but one; quarter * NC and
            // c_lo are even): both are reduced side by side, so that the loads of one hide behind the
            // arithmetic of the other.  With two terms the order of the sum does not matter (a + b is
            // b + a bit for bit), so the result is the one the general loop below gives.
            reduced = true;
            const uint32_t ca = c_lo + split, cb = ca + 2u;
            const int cola = col_tile0 + static_cast<int>(ca) * 32, colb = cola + 64;
            if (row0 < p.M && cola < p.N) {
                const bool two = colb < p.N;
                uint32_t v0[32], v1[32];
                tmem_ld_32x32(tmem_base + ca * 32 + lane_tmem, v0);
                if (two) tmem_ld_32x32(tmem_base + cb * 32 + lane_tmem, v1);
                tmem_ld_wait();
                const uint8_t* sa = ring_gen + (((quarter * NC + ca) & ~1u) + (split ^ 1u)) * 4096u;   // the other split's piece
                const uint8_t* sb = sa + 2u * 4096u;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const uint32_t off = g * 512 + ((lane ^ g) << 4);
                    const uint4 ta = *reinterpret_cast<const uint4*>(sa + off);
                    if (p.acc_s32) {
                        v0[4 * g] += ta.x; v0[4 * g + 1] += ta.y; v0[4 * g + 2] += ta.z; v0[4 * g + 3] += ta.w;
                    } else {
                        add2_f32(v0[4 * g], v0[4 * g + 1], ta.x, ta.y);
                        add2_f32(v0[4 * g + 2], v0[4 * g + 3], ta.z, ta.w);
                    }
                    if (two) {
                        const uint4 tb = *reinterpret_cast<const uint4*>(sb + off);
                        if (p.acc_s32) {
                            v1[4 * g] += tb.x; v1[4 * g + 1] += tb.y; v1[4 * g + 2] += tb.z; v1[4 * g + 3] += tb.w;
                        } else {
                            add2_f32(v1[4 * g], v1[4 * g + 1], tb.x, tb.y);
                            add2_f32(v1[4 * g + 2], v1[4 * g + 3], tb.z, tb.w);
                        }
                    }
                }
                if (p.dequant) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v0[i] = __float_as_uint(__int2float_rn(static_cast<int>(v0[i])) * p.scale);
                }
                umma_chunk_bias_relu(p, v0, cola, bias_sm ? bias_sm + ca * 32 : nullptr);
                umma_write_store_tile(p, v0, lane, tiles);
                ntiles = 1;
                if (two) {
                    if (p.dequant) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v1[i] = __float_as_uint(__int2float_rn(static_cast<int>(v1[i])) * p.scale);
                    }
                    umma_chunk_bias_relu(p, v1, colb, bias_sm ? bias_sm + cb * 32 : nullptr);
                    umma_write_store_tile(p, v1, lane, tiles + tile_bytes);
                    ntiles = 2;
                }
            }
        }
    }
#pragma unroll 1
    for (uint32_t c = r_lo; c < r_hi && !reduced; ++c) {
        const uint32_t u = quarter * NC + c;
        if ((u & (S - 1u)) != split) continue;           // warp-uniform
        const int col0 = col_tile0 + static_cast<int>(c) * 32;
        if (batched && (col0 >= p.N || row0 >= p.M)) continue;
        uint32_t own[32], v[32];
        tmem_ld_32x32(tmem_base + c * 32 + lane_tmem, own);
        tmem_ld_wait();
        const uint8_t* slot0 = ring_gen + (u & ~(S - 1u)) * 4096u;
        // split order s = 0, 1, .., S-1, this CTA's own accumulator taking its place in the row
#pragma unroll 1
        for (uint32_t sp = 0; sp < S; ++sp) {
            if (sp == split) {
                if (sp == 0) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = own[i];
                } else if (p.acc_s32) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] += own[i];
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) add2_f32(v[i], v[i + 1], own[i], own[i + 1]);
                }
                continue;
            }
            const uint8_t* slot = slot0 + sp * 4096u;
            if (sp == 0) {
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const uint4 t4 = *reinterpret_cast<const uint4*>(slot + g * 512 + ((lane ^ g) << 4));
                    v[4 * g] = t4.x; v[4 * g + 1] = t4.y; v[4 * g + 2] = t4.z; v[4 * g + 3] = t4.w;
                }
            } else if (p.acc_s32) {
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const uint4 t4 = *reinterpret_cast<const uint4*>(slot + g * 512 + ((lane ^ g) << 4));
                    v[4 * g] += t4.x; v[4 * g + 1] += t4.y; v[4 * g + 2] += t4.z; v[4 * g + 3] += t4.w;
                }
            } else {
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const uint4 t4 = *reinterpret_cast<const uint4*>(slot + g * 512 + ((lane ^ g) << 4));
                    add2_f32(v[4 * g], v[4 * g + 1], t4.x, t4.y);
                    add2_f32(v[4 * g + 2], v[4 * g + 3], t4.z, t4.w);
                }
            }
        }
        if (!batched) {
            // beta, blocked C: the chunk-at-a-time path through the warp's staging tiles
            umma_store_chunk(p, tmap_c, v, row0, lane, col0, 0, gemm, false, staging, parity, nullptr, nullptr);
            __syncwarp();
            parity ^= 1;
            continue;
        }
        if (p.dequant) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__int2float_rn(static_cast<int>(v[i])) * p.scale);
        }
        umma_chunk_bias_relu(p, v, col0, bias_sm ? bias_sm + c * 32 : nullptr);
        umma_write_store_tile(p, v, lane, tiles + ntiles * tile_bytes);
        ++ntiles;
    }
    if (batched && ntiles > 0) {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            // the owned chunks of the range, in the order their tiles were filled
            uint32_t k = 0;
#pragma unroll 1
            for (uint32_t c = r_lo; c < r_hi && k < ntiles; ++c) {
                if (((quarter * NC + c) & (S - 1u)) != split) continue;
                tma_store_3d(tmap_c, smem_u32(tiles + k * tile_bytes), col_tile0 + static_cast<int>(c) * 32, row0, gemm);
                ++k;
            }
            bulk_commit();
        }
    }
    if (lane == 0) bulk_wait_read<0>();
    __syncwarp();
    return true;
}

// Re-layout of a VNNI-blocked B operand (Figure 1 of the paper: [k/2][n][2] inside every 32 x 32
// block) into the K-major stage tile the tensor core reads: COLS columns n x 64 k, 128-byte
// rows, 16-byte chunk c of row n stored at chunk c ^ (n & 7) (the 128-byte swizzle).
//
// The producer brings the blocks of a stage with one TMA box: seen as 16-bit elements the
// operand is a 3-D tensor (64 elements = the 32 words of one k-pair row, K/2 pair rows, N/32
// column blocks), and a box of 64 x 32 x COLS/32 lands as COLS/32 regions of 4 KB, region j
// holding the 32 pair rows of column block j, 128 bytes each, 16-byte chunk c of row R at
// chunk c ^ (R & 7).  Seen as 32-bit words a region is 32 rows (k/2) x 32 words (n), and the
// stage tile wants its word transpose: word (R, n) belongs at row n, word R.  One warp
// transposes one region in place: a lane reads eight 4 x 4 word blocks with 16-byte loads
// (four rows R x four columns n each), the warp synchronises, and the lane writes each
// block's four columns as 16-byte stores (one column n, four consecutive R = eight
// consecutive k).  The lane -> block map below makes the eight lanes of a quarter warp touch
// eight different 16-byte bank groups in the loads and in the stores, so neither side has
// bank conflicts.  This is the paper's software-pipelined pack (Algorithm 3, AMX branch) in the
// opposite direction: the copies of later stages are in flight while a stage is re-laid.
// Who does what: with ALT the four warps take turns by stage (warps 6-7 the even stages, 8-9 the
// odd ones; STAGES is even), two warps sharing the regions of a stage, so that a warp has two stage
// times for its fixed costs (barrier wait, warp barriers, proxy fence, arrive); without it all four
// warps work on every stage.  Measured: ALT wins where a stage has two regions (64 columns per CTA:
// the other scheme leaves two warps idle) and in the pair kernel (+4.5 % on 8-bit 8192^3), and
// loses on single CTAs with four or more regions per stage (8-bit 512 x 4096 x 4096: 19.0 against
// 17.5 us), where the short stage time makes the longer per-stage latency count.
template <int COLS, bool PAIR>
__host__ __device__ constexpr bool vnni_alt() { return COLS / 32 == 2 || PAIR; }

template <int COLS, int WARPS>
__device__ __forceinline__ void vnni_relayout_stage(uint32_t sb, int first, int lane) {
    // This warp's regions of the stage: first, first + WARPS, ...  Regions go two at a time: all
    // loads of both, one warp barrier, all stores.
    // block (q, nq): pair rows 16h + 4q .. + 3 (h = 0, 1), columns 4nq .. 4nq + 3
    constexpr int REGIONS = COLS / 32;
    constexpr int MINE = (REGIONS + WARPS - 1) / WARPS;
    if (first >= REGIONS) return;           // 64 columns shared by four warps: two have nothing to move
    const uint32_t l0 = lane & 1, l1 = (lane >> 1) & 1, l2 = (lane >> 2) & 1, l3 = (lane >> 3) & 1, l4 = lane >> 4;
    const uint32_t q = l2 * 2 + l1;
    const uint32_t nq = l3 * 4 + (l2 ^ l4) * 2 + l0;
#pragma unroll
    for (int b = 0; b < MINE; b += 2) {
        const bool two = b + 1 < MINE;      // compile-time after unrolling
        const uint32_t rb0 = sb + (first + WARPS * b) * 4096;
        const uint32_t rb1 = rb0 + WARPS * 4096;
        uint32_t w0[2][4][4], w1[2][4][4];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint32_t R = 16 * h + 4 * q + r;
                const uint32_t off = R * 128 + ((nq ^ (R & 7)) << 4);
                ld_shared_v4(rb0 + off, w0[h][r]);
                if (two) ld_shared_v4(rb1 + off, w1[h][r]);
            }
        __syncwarp();
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t n = 4 * nq + c;
                const uint32_t off = n * 128 + (((4 * h + q) ^ (n & 7)) << 4);
                st_shared_v4(rb0 + off, w0[h][0][c], w0[h][1][c], w0[h][2][c], w0[h][3][c]);
                if (two) st_shared_v4(rb1 + off, w1[h][0][c], w1[h][1][c], w1[h][2][c], w1[h][3][c]);
            }
    }
}

template <int BN, int STAGES, bool B_VNNI, bool CLUSTER_REDUCE = false, int KIND = 0>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
umma_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_c, const UmmaParams p) {
    static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "tile N");
    constexpr int B_STAGE = umma_b_stage_bytes(BN);
    constexpr int STAGE = umma_stage_bytes(BN);
    constexpr uint32_t TMEM_COLS = (2 * BN <= 32) ? 32 : (2 * BN <= 64) ? 64 : (2 * BN <= 128) ? 128
                                   : (2 * BN <= 256) ? 256 : 512;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_base = smem_base + STAGES * STAGE + UMMA_EPI_STAGING;
    // after the stages: epilogue staging, then the barrier block: full[STAGES], empty[STAGES],
    // tmem_full[2], tmem_empty[2], then 2 words
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    auto raw_bar = [&](int s) { return bar_base + UMMA_RAW_BAR_OFFSET + 8u * s; };   // VNNI B: blocks of stage s have landed
    const uint32_t recv_bar0 = bar_base + UMMA_RECV_BAR_OFFSET;   // cluster split-K: pieces for epilogue warp w have landed
    uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot =
        reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * STAGE + UMMA_EPI_STAGING + 8 * (2 * STAGES + 4));
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (warp == 0) {
        // one barrier per lane: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2] (and raw[STAGES])
        constexpr int NB = 2 * STAGES + 4;
        static_assert(NB <= 32, "one barrier per lane");
        static_assert(!B_VNNI || STAGES % 2 == 0, "the re-layout warps take alternate stages");
        if (lane < NB)
            mbar_init(bar_base + 8u * lane, lane < STAGES ? (B_VNNI ? 1 + (vnni_alt<BN, false>() ? 2 : 4) : 1)
                                                          : lane < 2 * STAGES + 2 ? 1 : 128);
        if (B_VNNI && lane < STAGES) mbar_init(raw_bar(lane), 1);
        if (CLUSTER_REDUCE && lane >= 24) mbar_init(recv_bar0 + 8u * (lane - 24), 1);   // one per epilogue warp
        if (lane == 0) *abort_flag = 0;
        fence_mbar_init();
        __syncwarp();
    } else if (warp == 2 && lane == 0) {
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
        if (p.tma_store) tma_prefetch_desc(&tmap_c);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
        tmem_relinquish();
    }
    // The producer warp needs nothing but the barriers its own lanes have just initialised: it
    // signals the CTA barrier without waiting on it and starts fetching while tensor memory is
    // still being allocated (on a short problem this start-up is a visible part of the run).
    const uint32_t nthreads = blockDim.x;
    uint32_t tmem_base = 0;
    if (warp == 0) {
        __syncwarp();
        asm volatile("bar.arrive 0, %0;" ::"r"(nthreads) : "memory");
    } else {
        tc_fence_before_sync();
        asm volatile("bar.sync 0, %0;" ::"r"(nthreads) : "memory");
        tc_fence_after_sync();
        tmem_base = *tmem_slot;
    }

    const int total_units = p.gemms * p.tiles_m * p.tiles_n * p.splits;
    // a CTA with a single tile to deliver, stored by TMA: its epilogue is batched through the idle ring
    const bool one_shot = !CLUSTER_REDUCE && p.tma_store && p.splits == 1 && total_units <= static_cast<int>(gridDim.x);

    auto give_up = [&](unsigned int code) {
        *abort_flag = 1;
        if (p.status) atomicCAS(p.status, 0u, code);
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        // One lane issues, but the whole warp runs the loop (see elect_one); like the MMA issuer
        // its instruction stream paces the pipeline, so addresses advance by adds and the layout
        // decisions are taken outside the loops.
        const bool a_blk = p.a_blocked != 0;
        const bool b3d = p.b_3d != 0;
        const bool b_kmajor = p.b_kmajor != 0;
        const uint32_t elected = elect_one();
        int stage = 0;
        uint32_t phase = 0;
        uint32_t sa = smem_base, fb = full_bar(0);
        bool ok = true;
        for (int unit = blockIdx.x; ok && unit < total_units; unit += gridDim.x) {
            int tile, split, gemm;
            umma_decode_unit(p, unit, tile, split, gemm);
            int mb, nb;
            umma_tile_coords(p, tile, mb, nb);
            const int kb0 = split * p.kb_per_split;
            const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
            const int row0 = mb * UMMA_BM, col0 = nb * BN;
            // k-block kb of the reduction = k-block (kb % kb_per_item) of batch item kb / kb_per_item
            int item = kb0 == 0 ? 0 : div_small(kb0, p.kb_per_item);
            int kbl = kb0 - item * p.kb_per_item;
            item += gemm;   // independent batch: the unit's own (A, B) pair
            int ia, ib;
            umma_item_pair(p, item, ia, ib);
            for (int kb = kb0; kb < kb1; ++kb) {
                const int kx = kbl * (KIND != 0 ? 2 * UMMA_BK : UMMA_BK);   // a stage row is 128 bytes: 64 16-bit or 128 8-bit elements
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
                    if (lane == 0) give_up(0x100u + stage);
                    ok = false;
                    break;
                }
                {
                    // issued by the elected lane; the warp stays convergent (see elect_one)
                    const uint32_t sb = sa + UMMA_A_STAGE_BYTES;
                    mbar_arrive_expect_tx_if(fb, UMMA_A_STAGE_BYTES + (B_VNNI ? 0 : B_STAGE), elected);
                    if (a_blk) {
                        // two 32-wide K slabs, each 128 rows x 64 B (64-byte swizzle)
                        tma_load_5d_if(sa, &tmap_a, fb, 0, 0, kbl * 2, mb * 4, ia, elected);
                        tma_load_5d_if(sa + 8192, &tmap_a, fb, 0, 0, kbl * 2 + 1, mb * 4, ia, elected);
                    } else {
                        tma_load_3d_if(sa, &tmap_a, fb, kx, row0, ia, elected);
                    }
                    if (B_VNNI) {
                        // the stage's blocks as they are; warps 6-9 re-lay them in place
                        mbar_arrive_expect_tx_if(raw_bar(stage), B_STAGE, elected);
                        tma_load_4d_if(sb, &tmap_b, raw_bar(stage), 0, kbl * (UMMA_BK / 2), col0 >> 5, ib, elected);
                    } else if (b_kmajor) {
                        tma_load_3d_if(sb, &tmap_b, fb, kx, col0, ib, elected);   // BN rows (n) of 128 bytes of k
                    } else {
                        if (b3d) {
                            tma_load_4d_if(sb, &tmap_b, fb, 0, kx, col0 >> 6, ib, elected);
                        } else {
#pragma unroll
                            for (int j = 0; j < BN / 64; ++j)
                                tma_load_3d_if(sb + j * 8192, &tmap_b, fb, col0 + j * 64, kx, ib, elected);
                        }
                    }
                }
                if (++kbl == p.kb_per_item) { kbl = 0; ++item; umma_item_pair(p, item, ia, ib); }
                __syncwarp();
                sa += STAGE;
                fb += 8;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; sa = smem_base; fb = full_bar(0); }
            }
        }
        // Drain: wait (bounded) until the consumer has released every stage this warp
        // filled, so no TMA write is in flight when the CTA's shared memory is freed.
        if (ok) {
            for (int s = 0; s < STAGES; ++s) {
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) break;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        // One lane issues (the whole warp runs the loop, see elect_one); its instruction stream is the critical path of the K loop, so the
        // descriptors are kept as 32-bit halves and advanced with adds, and everything that
        // does not change per stage is computed here, once.
        //   A row-major: K-major tile, 128-byte swizzle, 8-row groups 1024 B apart; the four
        //     k-steps of a stage are 32 B apart.
        //   A blocked: two K-major slabs of 32 k (8192 B apart), 64-byte swizzle, 8-row groups
        //     512 B apart; k-steps at 0, 32 B, 8192 B, 8192 + 32 B.
        //   B row-major [K][N]: N-major, 64-column atoms 8192 B apart (leading), 8-k groups
        //     1024 B apart (stride); k-steps 2048 B apart.  B re-laid from VNNI, or stored transposed: K-major like A.
        const bool a_blk = p.a_blocked != 0;
        const uint64_t da0 = a_blk ? make_smem_desc(smem_base, 16, 512, 4) : make_smem_desc(smem_base, 16, 1024, 2);
        const bool b_k = B_VNNI || p.b_kmajor != 0;
        const uint64_t db0 = b_k ? make_smem_desc(smem_base + UMMA_A_STAGE_BYTES, 16, 1024, 2)
                                 : make_smem_desc(smem_base + UMMA_A_STAGE_BYTES, 8192, 1024, 2);
        const uint32_t a_hi = static_cast<uint32_t>(da0 >> 32), b_hi = static_cast<uint32_t>(db0 >> 32);
        const uint32_t a_lo0 = static_cast<uint32_t>(da0), b_lo0 = static_cast<uint32_t>(db0);
        const uint32_t a_s1 = 2u, a_s2 = a_blk ? 512u : 4u, a_s3 = a_blk ? 514u : 6u;
        const uint32_t b_s = b_k ? 2u : 128u, b_s2 = 2 * b_s, b_s3 = 3 * b_s;
        constexpr uint32_t STAGE16 = STAGE >> 4;
        const uint32_t idesc = p.idesc;
        const uint32_t elected = elect_one();
        int stage = 0;
        uint32_t phase = 0;
        uint32_t soff = 0;  // stage * STAGE / 16
        int local = 0;
        bool ok = true;
        for (int unit = blockIdx.x; ok && unit < total_units; unit += gridDim.x, ++local) {
            int tile, split, gemm;
            umma_decode_unit(p, unit, tile, split, gemm);
            const int kb0 = split * p.kb_per_split;
            const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
            const int acc = local & 1;
            if (!mbar_wait(tempty_bar(acc), ((local >> 1) & 1u) ^ 1u, abort_flag)) {
                if (lane == 0) give_up(0x200u + acc);
                ok = false;
                break;
            }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + acc * BN;
            uint32_t accumulate = 0u;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(full_bar(stage), phase, abort_flag)) {
                    if (lane == 0) give_up(0x300u + stage);
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                {
                    const uint32_t a_lo = a_lo0 + soff, b_lo = b_lo0 + soff;
                    umma_if<KIND>(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc, accumulate, elected);
                    umma_if<KIND>(d_tmem, a_lo + a_s1, a_hi, b_lo + b_s, b_hi, idesc, 1u, elected);
                    umma_if<KIND>(d_tmem, a_lo + a_s2, a_hi, b_lo + b_s2, b_hi, idesc, 1u, elected);
                    umma_if<KIND>(d_tmem, a_lo + a_s3, a_hi, b_lo + b_s3, b_hi, idesc, 1u, elected);
                    umma_commit_if(empty_bar(stage), elected);
                    if (kb == kb1 - 1) umma_commit_if(tfull_bar(acc), elected);
                }
                accumulate = 1u;
                __syncwarp();
                soff += STAGE16;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; soff = 0; }
            }
            if (kb1 <= kb0) umma_commit_if(tfull_bar(acc), elected);  // empty K range
        }
    } else {
        // ------------------------------------------------ warps 2..9
        // Warps 2-5 are the epilogue.  Warps 6-9 first re-lay VNNI B (if that is the operand form),
        // then join the epilogue of a CTA that delivers a single tile (one-shot, cluster split-K):
        // tensor-memory lanes are tied to warp % 4, so each quarter of the rows has two warps,
        // which take half of the columns each.
        const int set = warp >= 6 ? 1 : 0;
        const int quarter = warp & 3;  // TMEM lanes 32*quarter .. +31 belong to this warp
        uint8_t* staging = gen_base + STAGES * STAGE + quarter * 8192;   // set 0: two store tiles; bias slices behind them
        if (set == 1 && B_VNNI) {
            // -------------------------------------------- VNNI re-layout
            const int tw = warp - 6;
            constexpr bool ALT = vnni_alt<BN, false>();
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int unit = blockIdx.x; ok && unit < total_units; unit += gridDim.x) {
                int tile, split, gemm;
                umma_decode_unit(p, unit, tile, split, gemm);
                const int kb0 = split * p.kb_per_split;
                const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!ALT || (stage & 1) == (tw >> 1)) {
                        if (!mbar_wait(raw_bar(stage), phase, abort_flag)) {
                            if (lane == 0) give_up(0x500u + stage);
                            ok = false;
                            break;
                        }
                        vnni_relayout_stage<BN, ALT ? 2 : 4>(smem_base + stage * STAGE + UMMA_A_STAGE_BYTES, ALT ? (tw & 1) : tw, lane);
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(full_bar(stage));
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        if (CLUSTER_REDUCE) {
            // -------------------------------------------- epilogue, K splits reduced inside the cluster
            // One unit per CTA (grid = units); cluster rank = K split.
            int tile, split, gemm;
            umma_decode_unit(p, blockIdx.x, tile, split, gemm);
            int mb, nb;
            umma_tile_coords(p, tile, mb, nb);
            bool ok = blockIdx.x < total_units;
            const float* bias_sm = p.tma_store ? umma_park_bias<BN>(p, reinterpret_cast<float*>(staging + set * 2048), nb * BN, lane)
                                               : nullptr;
            if (ok && !mbar_wait(tfull_bar(0), 0u, abort_flag)) {
                if (lane == 0) give_up(0x400u);
                ok = false;
            }
            tc_fence_after_sync();
            umma_cluster_epilogue<BN>(p, &tmap_c, tmem_base, smem_base, gen_base, staging, bias_sm, quarter, set, lane,
                                      static_cast<uint32_t>(p.splits), cluster_ctarank(), 0u, 1u, mb * UMMA_BM, nb * BN, gemm, ok,
                                      recv_bar0, abort_flag);
        } else if (set == 1) {
            // -------------------------------------------- second half of a one-shot epilogue
            if (one_shot && static_cast<int>(blockIdx.x) < total_units) {
                int tile, split, gemm;
                umma_decode_unit(p, blockIdx.x, tile, split, gemm);
                int mb, nb;
                umma_tile_coords(p, tile, mb, nb);
                const float* bias_sm = umma_park_bias<BN>(p, reinterpret_cast<float*>(staging + 6144), nb * BN, lane);
                if (!mbar_wait(tfull_bar(0), 0u, abort_flag)) {
                    if (lane == 0) give_up(0x480u);
                } else {
                    tc_fence_after_sync();
                    umma_epilogue_oneshot<BN>(p, &tmap_c, tmem_base + (static_cast<uint32_t>(quarter * 32) << 16),
                                              gen_base + (quarter * 2 + 1) * (BN * 64), mb * UMMA_BM + quarter * 32, nb * BN, gemm,
                                              lane, p.kb_total <= 0, bias_sm, BN / 64, BN / 32);
                }
                if (lane == 0) bulk_wait_read<0>();
                __syncwarp();
            }
        } else {
            // -------------------------------------------- epilogue
            int local = 0;
            bool ok = true;
            for (int unit = blockIdx.x; ok && unit < total_units; unit += gridDim.x, ++local) {
                int tile, split, gemm;
                umma_decode_unit(p, unit, tile, split, gemm);
                int mb, nb;
                umma_tile_coords(p, tile, mb, nb);
                const int kb0 = split * p.kb_per_split;
                const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
                const int acc = local & 1;
                const float* bias_smem = one_shot ? umma_park_bias<BN>(p, reinterpret_cast<float*>(staging + 4096), nb * BN, lane)
                                                  : umma_fetch_bias<BN>(p, staging, nb * BN, lane);
                if (!mbar_wait(tfull_bar(acc), (local >> 1) & 1u, abort_flag)) {
                    if (lane == 0) give_up(0x400u + acc);
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const int row0 = mb * UMMA_BM + quarter * 32;
                const bool empty_k = kb1 <= kb0;
                if (one_shot) {
                    // the only tile of this CTA: the ring is idle, batch the stores through it (first half
                    // of the columns; warps 6-9 take the second)
                    umma_epilogue_oneshot<BN>(p, &tmap_c, tmem_base + acc * BN + (static_cast<uint32_t>(quarter * 32) << 16),
                                              gen_base + (quarter * 2) * (BN * 64), row0, nb * BN, gemm, lane, empty_k, bias_smem,
                                              0, BN / 64);
                    tc_fence_before_sync();
                    mbar_arrive(tempty_bar(acc));
                    continue;
                }
                PartialDst pdst = {p.partial + (static_cast<size_t>(split) * p.gemms + gemm) * p.M * p.N, p.N, row0, 0, p.M, p.N};
                const PartialDst* pd = p.splits > 1 ? &pdst : nullptr;
                // two 32-column chunks per round: one wait for both tensor-memory loads
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 64) {
                    uint32_t v0[32], v1[32];
                    const uint32_t taddr = tmem_base + acc * BN + c0 + (static_cast<uint32_t>(quarter * 32) << 16);
                    tmem_ld_32x32(taddr, v0);
                    tmem_ld_32x32(taddr + 32, v1);
                    tmem_ld_wait();
                    pdst.col0 = nb * BN + c0;
                    umma_store_chunk(p, &tmap_c, v0, row0, lane, nb * BN + c0, split, gemm, empty_k, staging, 0,
                                     bias_smem ? bias_smem + c0 : nullptr, pd);
                    __syncwarp();
                    pdst.col0 = nb * BN + c0 + 32;
                    umma_store_chunk(p, &tmap_c, v1, row0, lane, nb * BN + c0 + 32, split, gemm, empty_k, staging, 1,
                                     bias_smem ? bias_smem + c0 + 32 : nullptr, pd);
                    __syncwarp();
                }
                tc_fence_before_sync();
                mbar_arrive(tempty_bar(acc));
            }
            // the TMA stores of this warp must have read their staging buffers before the CTA's shared
            // memory goes away; their global writes are part of the grid's work and complete with it
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
        }
    }

    if (CLUSTER_REDUCE && warp < 2) {
        // the cluster barrier counts every thread: the other roles pass it here, once their part
        // of the K loop is over (the producer has seen every stage consumed)
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
