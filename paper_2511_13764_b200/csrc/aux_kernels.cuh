// Small kernels around the two GEMM mainloops: the one-thread-per-output debug
// kernel, the deterministic split-K reduction with the fused epilogue, and the
// unpacking of a VNNI-blocked B operand into row-major scratch.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace nk {

// A 16-bit element is BF16 (its bits are the upper half of the FP32 pattern) or, with `f16`
// set, IEEE binary16.  Both widen exactly to FP32; a result is rounded once (RNE) on the way out.
__device__ __forceinline__ float half_bits_to_f32(uint32_t h, int f16) {
    return f16 ? __half2float(__ushort_as_half(static_cast<unsigned short>(h))) : __uint_as_float(h << 16);
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi, int f16) {
    if (f16) {
        const __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&v);
    }
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

struct NaiveParams {
    int M, N, K;
    int in_bf16, out_bf16, a_blocked, b_blocked, epilogue;   // in_bf16 / out_bf16: 16-bit elements (BF16 or FP16)
    int batch, beta;
    long long stride_a, stride_b;
    int gemms;             // batched matmul: gridDim.z independent GEMMs
    long long stride_c;
    int c_blocked;         // C stored as [M/32][N/32][32][32]
    const void *A, *B, *bias;
    void* C;
    int f16;               // the 16-bit type is IEEE binary16, not BF16
};

__device__ __forceinline__ float ld_elem(const void* p, int is16, int f16, size_t i) {
    return is16 ? half_bits_to_f32(static_cast<const uint16_t*>(p)[i], f16) : static_cast<const float*>(p)[i];
}

// Debug cross-check only: one thread per C element, FP32 accumulation in k order,
// operands addressed through the layout index functions (Figure 1 for blocked B).
__global__ void naive_gemm_kernel(const NaiveParams p) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = blockIdx.y;
    if (j >= p.N || i >= p.M) return;
    const size_t kb32 = p.K / 32;
    const int g = blockIdx.z;
    const size_t o = static_cast<size_t>(g) * p.stride_c +
                     (p.c_blocked ? ((static_cast<size_t>(i / 32) * (p.N / 32) + j / 32) * 32 + i % 32) * 32 + j % 32
                                  : static_cast<size_t>(i) * p.N + j);
    float acc = 0.f;
    if (p.beta) acc = ld_elem(p.C, p.out_bf16, p.f16, o);
    for (int b = 0; b < p.batch; ++b)
    for (int k = 0; k < p.K; ++k) {
        const size_t ia = p.a_blocked
            ? (((static_cast<size_t>(i / 32) * kb32 + k / 32) * 32 + i % 32) * 32 + k % 32)
            : static_cast<size_t>(i) * p.K + k;
        const size_t ib = p.b_blocked
            ? (((((static_cast<size_t>(j / 32) * kb32 + k / 32) * 16 + (k % 32) / 2) * 32 + j % 32) * 2) + k % 2)
            : static_cast<size_t>(k) * p.N + j;
        acc = fmaf(ld_elem(p.A, p.in_bf16, p.f16, (g + b) * p.stride_a + ia), ld_elem(p.B, p.in_bf16, p.f16, (g + b) * p.stride_b + ib), acc);
    }
    if (p.epilogue) acc = fmaxf(acc + ld_elem(p.bias, p.in_bf16, p.f16, j), 0.f);
    if (p.out_bf16)
        static_cast<uint16_t*>(p.C)[o] = static_cast<uint16_t>(pack_half2(acc, 0.f, p.f16) & 0xFFFFu);
    else
        static_cast<float*>(p.C)[o] = acc;
}

struct ReduceParams {
    size_t MN;          // elements of C
    int N;
    int splits;
    int epilogue, bias_bf16, out_bf16;
    int beta;              // 1: add the old C before the epilogue
    int c_blocked;         // C stored as [M/32][N/32][32][32] (per GEMM of M_rows rows)
    int M;                 // rows of one GEMM
    const float* partial;  // [splits][M][N]
    const void* bias;
    void* C;
    int f16;               // the 16-bit type (bias_bf16 / out_bf16) is IEEE binary16, not BF16
    int int_partials;      // the partials are INT32 sums (INT8 operands): added as integers, exactly
    int dequant;           // ... then converted to FP32 and multiplied by `scale` before the epilogue
    float scale;
};

// Sum of the splits of four consecutive elements, in split order: FP32 adds, or exact INT32 adds (the
// result then either keeps its integer bit pattern or becomes scale * sum in FP32).
__device__ __forceinline__ float4 sum_partials(const float* first, size_t stride, int splits, int int_partials,
                                               int dequant, float scale) {
    if (!int_partials) {
        float4 s = __ldcs(reinterpret_cast<const float4*>(first));
        for (int sp = 1; sp < splits; ++sp) {
            const float4 v = __ldcs(reinterpret_cast<const float4*>(first + sp * stride));
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        return s;
    }
    int4 a = __ldcs(reinterpret_cast<const int4*>(first));
    for (int sp = 1; sp < splits; ++sp) {
        const int4 v = __ldcs(reinterpret_cast<const int4*>(first + sp * stride));
        a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    if (dequant)
        return make_float4(__int2float_rn(a.x) * scale, __int2float_rn(a.y) * scale, __int2float_rn(a.z) * scale,
                           __int2float_rn(a.w) * scale);
    return make_float4(__int_as_float(a.x), __int_as_float(a.y), __int_as_float(a.z), __int_as_float(a.w));
}

// C = epilogue(sum over splits, in split order): fixed order, so the result does
// not depend on how CTAs were scheduled.  Four consecutive columns per thread.
__global__ void splitk_reduce_kernel(const ReduceParams p) {
    const size_t q = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t e = q * 4;
    if (e >= p.MN) return;
    // where the four elements live in C: same index, or inside their 32 x 32 block
    size_t ce = e;
    if (p.c_blocked) {
        const size_t per = static_cast<size_t>(p.M) * p.N;
        const size_t g = e / per, r = e - g * per;
        const size_t i = r / p.N, j = r - i * p.N;
        ce = g * per + ((i / 32 * (p.N / 32) + j / 32) * 32 + i % 32) * 32 + j % 32;
    }
    float4 s = sum_partials(p.partial + e, p.MN, p.splits, p.int_partials, p.dequant, p.scale);
    if (p.beta) {
        if (p.out_bf16) {
            const uint2 w = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.C) + ce);
            s.x += half_bits_to_f32(w.x & 0xFFFFu, p.f16); s.y += half_bits_to_f32(w.x >> 16, p.f16);
            s.z += half_bits_to_f32(w.y & 0xFFFFu, p.f16); s.w += half_bits_to_f32(w.y >> 16, p.f16);
        } else {
            const float4 c = *reinterpret_cast<const float4*>(static_cast<const float*>(p.C) + ce);
            s.x += c.x; s.y += c.y; s.z += c.z; s.w += c.w;
        }
    }
    if (p.epilogue) {
        const int n = static_cast<int>(e % p.N);
        float b0, b1, b2, b3;
        if (p.bias_bf16) {
            const uint2 w = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.bias) + n));
            b0 = half_bits_to_f32(w.x & 0xFFFFu, p.f16); b1 = half_bits_to_f32(w.x >> 16, p.f16);
            b2 = half_bits_to_f32(w.y & 0xFFFFu, p.f16); b3 = half_bits_to_f32(w.y >> 16, p.f16);
        } else {
            const float4 w = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(p.bias) + n));
            b0 = w.x; b1 = w.y; b2 = w.z; b3 = w.w;
        }
        s.x = fmaxf(s.x + b0, 0.f); s.y = fmaxf(s.y + b1, 0.f);
        s.z = fmaxf(s.z + b2, 0.f); s.w = fmaxf(s.w + b3, 0.f);
    }
    if (p.out_bf16) {
        uint2 o;
        o.x = pack_half2(s.x, s.y, p.f16);
        o.y = pack_half2(s.z, s.w, p.f16);
        *reinterpret_cast<uint2*>(static_cast<uint16_t*>(p.C) + ce) = o;
    } else {
        *reinterpret_cast<float4*>(static_cast<float*>(p.C) + ce) = s;
    }
}

struct TailReduceParams {
    int M, N;
    int tile_rows, tile_cols;   // 256 x BN
    int tiles_m, tiles_n, group_m, first_tile;   // raster of the GEMM kernel; first_tile = id of tail tile 0
    int serpentine;             // raster: odd groups of M tiles sweep N backwards
    int kb_total, sk_share;     // k-blocks of a tile; k-blocks of the tail each pair took (segment boundaries)
    int max_segs;               // slabs reserved per tail tile
    int epilogue, bias_bf16, out_bf16, beta, c_blocked, f16;
    const float* partial;       // [tail tile][segment][tile_rows][tile_cols]
    const void* bias;
    void* C;
    int int_partials, dequant;  // as in ReduceParams
    float scale;
};

// Sums the segments of the tail tiles (the last, partial wave of a large GEMM, shared out by
// k-blocks over all the CTA pairs: see the pair kernel) in segment order, which is k order, and
// applies the epilogue: blockIdx.y = tail tile, four consecutive columns per thread.  Pair i took
// the k-blocks [i * sk_share, (i + 1) * sk_share) of the tail tiles laid end to end, so tile t was
// cut by the pairs t * kb_total / sk_share .. ((t + 1) * kb_total - 1) / sk_share.
__global__ void tail_reduce_kernel(const TailReduceParams p) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    const int per_row = p.tile_cols / 4;
    const int r = q / per_row, c = (q - r * per_row) * 4;
    if (r >= p.tile_rows) return;
    // tile id -> (m block, n block), as in the GEMM kernel's raster
    const int tile = p.first_tile + blockIdx.y;
    const int per_group = p.group_m * p.tiles_n;
    const int g = tile / per_group;
    const int within = tile - g * per_group;
    const int first_m = g * p.group_m;
    const int gm = min(p.group_m, p.tiles_m - first_m);
    const int mb = first_m + within % gm;
    int nb = within / gm;
    if (p.serpentine && (g & 1)) nb = p.tiles_n - 1 - nb;
    const int i = mb * p.tile_rows + r, j = nb * p.tile_cols + c;
    if (i >= p.M || j >= p.N) return;
    const int t = blockIdx.y;
    const int segs = ((t + 1) * p.kb_total - 1) / p.sk_share - (t * p.kb_total) / p.sk_share + 1;
    const size_t slab = static_cast<size_t>(p.tile_rows) * p.tile_cols;
    const float* src = p.partial + static_cast<size_t>(t) * p.max_segs * slab + static_cast<size_t>(r) * p.tile_cols + c;
    float4 s = sum_partials(src, slab, segs, p.int_partials, p.dequant, p.scale);
    const size_t ce = p.c_blocked ? ((static_cast<size_t>(i / 32) * (p.N / 32) + j / 32) * 32 + i % 32) * 32 + j % 32
                                  : static_cast<size_t>(i) * p.N + j;
    if (p.beta) {
        if (p.out_bf16) {
            const uint2 w = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.C) + ce);
            s.x += half_bits_to_f32(w.x & 0xFFFFu, p.f16); s.y += half_bits_to_f32(w.x >> 16, p.f16);
            s.z += half_bits_to_f32(w.y & 0xFFFFu, p.f16); s.w += half_bits_to_f32(w.y >> 16, p.f16);
        } else {
            const float4 cv = *reinterpret_cast<const float4*>(static_cast<const float*>(p.C) + ce);
            s.x += cv.x; s.y += cv.y; s.z += cv.z; s.w += cv.w;
        }
    }
    if (p.epilogue && !p.bias_bf16) {
        const float4 w = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(p.bias) + j));
        s.x = fmaxf(s.x + w.x, 0.f); s.y = fmaxf(s.y + w.y, 0.f);
        s.z = fmaxf(s.z + w.z, 0.f); s.w = fmaxf(s.w + w.w, 0.f);
    } else if (p.epilogue) {
        const uint2 w = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.bias) + j));
        s.x = fmaxf(s.x + half_bits_to_f32(w.x & 0xFFFFu, p.f16), 0.f); s.y = fmaxf(s.y + half_bits_to_f32(w.x >> 16, p.f16), 0.f);
        s.z = fmaxf(s.z + half_bits_to_f32(w.y & 0xFFFFu, p.f16), 0.f); s.w = fmaxf(s.w + half_bits_to_f32(w.y >> 16, p.f16), 0.f);
    }
    if (p.out_bf16) {
        uint2 o;
        o.x = pack_half2(s.x, s.y, p.f16);
        o.y = pack_half2(s.z, s.w, p.f16);
        *reinterpret_cast<uint2*>(static_cast<uint16_t*>(p.C) + ce) = o;
    } else {
        *reinterpret_cast<float4*>(static_cast<float*>(p.C) + ce) = s;
    }
}

// FP32 -> three BF16 planes whose sum is the FP32 value (to within 2^-27 of it): hi = bf16(x),
// mid = bf16(x - hi), lo = bf16(x - hi - mid), every rounding to nearest even, the subtractions
// exact in FP32.  Products of BF16 values are exact in FP32, so a GEMM over cross terms of the
// planes of A and B, accumulated in FP32, reproduces the FP32 product on the tensor cores.  A
// value whose hi plane is not finite (inf, NaN, or beyond the largest BF16, 3.39e38) keeps that
// plane only (inf - inf would poison the others).
// Plane q of element i is P[q * plane + i]; four elements per thread and iteration.  One launch
// splits both operands: the first `blocks_a` CTAs take A, the others B.
struct SplitOperand {
    const float* X;
    uint16_t* P;
    long long count, plane;
};

__global__ void split_f32_bf16x3_kernel(const SplitOperand a, const SplitOperand b, unsigned blocks_a) {
    const bool is_a = blockIdx.x < blocks_a;
    const SplitOperand& o = is_a ? a : b;
    const long long block = is_a ? blockIdx.x : blockIdx.x - blocks_a;
    const long long nblocks = is_a ? blocks_a : gridDim.x - blocks_a;
    const long long step = nblocks * blockDim.x * 4;
    for (long long i = (block * blockDim.x + threadIdx.x) * 4; i < o.count; i += step) {
        const float4 x4 = __ldcs(reinterpret_cast<const float4*>(o.X + i));
        const float x[4] = {x4.x, x4.y, x4.z, x4.w};
        uint32_t hi[4], mid[4], lo[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            hi[j] = pack_half2(x[j], 0.f, false) & 0xFFFFu;
            const float r1 = x[j] - __uint_as_float(hi[j] << 16);
            mid[j] = pack_half2(r1, 0.f, false) & 0xFFFFu;
            const float r2 = r1 - __uint_as_float(mid[j] << 16);
            lo[j] = pack_half2(r2, 0.f, false) & 0xFFFFu;
            if ((hi[j] & 0x7F80u) == 0x7F80u) mid[j] = lo[j] = 0u;
        }
        *reinterpret_cast<uint2*>(o.P + i) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
        *reinterpret_cast<uint2*>(o.P + o.plane + i) = make_uint2(mid[0] | (mid[1] << 16), mid[2] | (mid[3] << 16));
        *reinterpret_cast<uint2*>(o.P + 2 * o.plane + i) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
    }
}

// VNNI-blocked B[N/32][K/32][16][32][2] -> row-major B[K][N] (BF16).  One CTA per
// 32 x 32 block; thread (r, lane) reads word (k2 = r.., n = lane) and writes the two
// k rows.  Reads are 128-byte rows; writes are 64-byte row segments.
__global__ void unpack_vnni_b_kernel(const uint32_t* __restrict__ Bblk, uint16_t* __restrict__ Brow,
                                     int N, int K) {
    const int kb = blockIdx.x, nb = blockIdx.y;
    const int lane = threadIdx.x & 31, r = threadIdx.x >> 5;  // 8 warps
    const size_t blk = (static_cast<size_t>(nb) * (K / 32) + kb) * 512;
    for (int k2 = r; k2 < 16; k2 += 8) {
        const uint32_t w = Bblk[blk + k2 * 32 + lane];
        const size_t row0 = static_cast<size_t>(kb * 32 + 2 * k2) * N + nb * 32 + lane;
        Brow[row0] = static_cast<uint16_t>(w & 0xFFFFu);       // even k: low half
        Brow[row0 + N] = static_cast<uint16_t>(w >> 16);       // odd k: high half
    }
}

// FP32 -> INT8: q = saturate(round-to-nearest-even(x * inv_scale)), the product in FP32 (one
// multiplication: nothing for the compiler to contract); NaN converts to 0.  Four elements per thread.
__global__ void quantize_s8_kernel(const float* __restrict__ x, int8_t* __restrict__ q, size_t n, float inv_scale) {
    const size_t i = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
    if (i >= n) return;
    auto one = [&](float v) { return static_cast<uint32_t>(max(-128, min(127, __float2int_rn(v * inv_scale))) & 0xFF); };
    if (i + 4 <= n) {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(x + i));
        const uint32_t w = one(v.x) | (one(v.y) << 8) | (one(v.z) << 16) | (one(v.w) << 24);
        if ((reinterpret_cast<uintptr_t>(q + i) & 3u) == 0) {
            *reinterpret_cast<uint32_t*>(q + i) = w;
        } else {
            for (int j = 0; j < 4; ++j) q[i + j] = static_cast<int8_t>((w >> (8 * j)) & 0xFF);
        }
    } else {
        for (size_t j = i; j < n; ++j) q[j] = static_cast<int8_t>(one(x[j]));
    }
}

// Self-test of the bounded-wait path: one warp waits on an mbarrier that nothing ever
// arrives on, with a short limit; the wait gives up, the kernel records the code in the
// status word and returns normally (no trap, no fault, the context stays usable).
__global__ void wait_timeout_probe_kernel(unsigned int* status, long long limit_clocks) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t abort_flag;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncwarp();
    const bool done = mbar_wait(b, 0u, &abort_flag, limit_clocks);
    if (!done && threadIdx.x == 0 && status) atomicCAS(status, 0u, 0x900u);
}

}  // namespace nk
