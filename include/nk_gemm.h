/*
 * nk_gemm — dense GEMM for NVIDIA B200 (sm_100a) behind a plain C ABI.
 *
 * The operation is the batch-reduce GEMM of the paper's Algorithm 1
 * (C = beta*C + sum_i A_i x B_i) taken with beta = 0 and the batch folded into K:
 *
 *     C[M][N] = A[M][K] . B[K][N]                     FP32 accumulation
 *     C[M][N] = ReLU(A.B + bias[N])                   optional fused epilogue
 *                                                     (Section 6, the MLP benchmark: bias and ReLU are
 *                                                     applied before the single store of C)
 *
 * Element types (Section 2.3): FP32 operands, or 16-bit operands (BF16; or FP16, the
 * packed type Section 5 names next) widened exactly to FP32 with the products
 * accumulated in FP32.  C is FP32, or has the operands' 16-bit type, rounded to
 * nearest-even once, after the epilogue.  Wherever a rule below says BF16 it holds
 * for FP16 as well.  8-bit operands (NK_S8 with exact INT32 accumulation, the Int8 dot
 * product Section 5 names among the next packed types; NK_E4M3 / NK_E5M2 with FP32
 * accumulation) take A row-major and B blocked with four k per group; see nk_dtype_t.
 *
 * Operand layouts (Section 2.3, Figure 1 and Listing 1):
 *   NK_ROW_MAJOR   A[M][K], B[K][N]                      ("flat")
 *   NK_BLOCKED32   A[M/32][K/32][32][32]                 (m-block, k-block, m, k)
 *                  B[N/32][K/32][16][32][2]              (n-block, k-block, k/2, n, k%2):
 *                  every 32x32 block of B is VNNI-2 packed as in Figure 1,
 *                  packed[k/2][n][k%2] = flat[k][n] (16-bit operands);
 *                  B[N/32][K/32][8][32][4], packed[k/4][n][k%4] = flat[k][n] (8-bit operands:
 *                  four k per 32-bit group, the INT8 packing Section 2 describes).
 *   NK_TRANSPOSED  (layout_b only) Bt[N][K]: B kept as its transpose, K contiguous.
 * C is row-major [M][N] unless desc.layout_c asks for the blocked form; bias is [N] in the
 * operand type (FP32 for 8-bit operands).
 *
 * All data pointers are DEVICE pointers on the plan's device unless a function
 * says otherwise.  The library never allocates or frees device memory, never
 * synchronises inside nk_gemm_run, and reports every failure as a status code
 * (nothing is printed, nothing is thrown).  No CPU fallback exists: without a
 * usable sm_100 device every call that needs one returns NK_ERR_DEVICE.
 */
#ifndef NK_GEMM_H
#define NK_GEMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct nk_gemm_s* nk_gemm_t; /* opaque plan; host memory only */

typedef enum {
    NK_OK = 0,
    NK_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bad enum                */
    NK_ERR_UNSUPPORTED = 2, /* legal request this build has no kernel for               */
    NK_ERR_MISALIGNED = 3,  /* pointer not 16-byte aligned / size not a required multiple */
    NK_ERR_WORKSPACE = 4,   /* workspace null or smaller than nk_gemm_workspace_bytes   */
    NK_ERR_DEVICE = 5,      /* no CUDA device, wrong device, or not compute capability 10.x */
    NK_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed                        */
    NK_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out (see nk_gemm_check)    */
} nk_status_t;

typedef enum {
    NK_F32 = 0,
    NK_BF16 = 1,
    NK_F16 = 2, /* IEEE binary16: the other 16-bit packed type (Section 5 names FP16 as the next one); same
                   kernels, layouts and rules as BF16, FP32 accumulation, one RNE rounding of a 16-bit C */
    NK_S8 = 3, /* signed 8-bit integers: the Int8 dot product Section 5 names among the next packed types.  A is
                  row-major; B is NK_BLOCKED32 with four k per 32-bit group (the INT8 packing of Section 2):
                  B[N/32][K/32][8][32][4], packed[k/4][n][k%4] = flat[k][n] inside each 32 x 32 block;
                  or NK_TRANSPOSED (8-bit operands have no row-major [K][N] form here).
                  The result is exact: INT32 accumulation of at most 2^17 - 1 products (K splits add their
                  INT32 partial sums as integers).  No epilogue with an INT32 C, no beta, no batch; N and K
                  multiples of 32 */
    NK_S32 = 4, /* signed 32-bit integers: the type of C for NK_S8 operands (and only for them).  NK_S8
                  operands may also have an NK_F32 C: the INT32 sum is converted (round to nearest even),
                  multiplied by desc.scale and given the epilogue (FP32 bias + ReLU) before the store */
    NK_E4M3 = 5, /* 8-bit floating point, 4 exponent bits (bias 7), 3 fraction bits, no infinities, largest finite
                    value 448 (the OCP FP8 E4M3 format) */
    NK_E5M2 = 6  /* 8-bit floating point, 5 exponent bits (bias 15), 2 fraction bits, IEEE infinities and NaNs.
                    Both: the 8-bit floating-point counterpart on this hardware of the packed types Section 5
                    lists; A row-major, B NK_BLOCKED32 with four k per group or NK_TRANSPOSED like NK_S8, FP32 accumulation, FP32 C,
                    FP32 bias; N and K multiples of 32; no batch */
} nk_dtype_t;
typedef enum {
    NK_ROW_MAJOR = 0,
    NK_BLOCKED32 = 1,
    NK_TRANSPOSED = 2 /* layout_b only: B is stored transposed, Bt[N][K] with K contiguous (the way a linear layer's
                         weight [out][in] is usually kept).  16-bit and 8-bit operands; K a multiple of 16, N of 8.
                         Not one of the paper's layouts (flat [K][N] and VNNI-blocked): on this hardware
                         it is the operand form the tensor core reads without any re-layout */
} nk_layout_t;
typedef enum { NK_EPI_NONE = 0, NK_EPI_BIAS_RELU = 1 } nk_epilogue_t;

/* desc.flags: 0 lets the plan choose.  The rest are tuning/debug overrides. */
#define NK_FLAG_KERNEL_MASK 0x0000000Fu
#define NK_FLAG_KERNEL_AUTO 0x0u
#define NK_FLAG_KERNEL_NAIVE 0x1u /* one thread per output element; debug cross-check only   */
#define NK_FLAG_KERNEL_SIMT 0x2u  /* register-blocked FFMA kernel (FP32 operands)             */
#define NK_FLAG_KERNEL_UMMA 0x3u  /* TMA + tcgen05.mma + TMEM pipeline (BF16 operands)        */
#define NK_FLAG_REPACK_B 0x10u    /* blocked B: unpack to row-major in the workspace first,
                                     instead of re-laying it out inside the GEMM kernel      */
#define NK_FLAG_SINGLE_CTA 0x20u  /* BF16: never pair CTAs (one CTA per 128-row tile)            */
#define NK_FLAG_CTA_PAIR 0x40u    /* BF16: always pair CTAs (256-row tiles, cta_group::2 MMA)      */
#define NK_FLAG_SCALAR_FMA 0x80u  /* FP32 128 x 128 tile: scalar FFMA instead of packed fma.f32x2   */
#define NK_FLAG_SEPARATE_REDUCE 0x100000u /* BF16 split-K: always write FP32 partials to the workspace and sum
                                             them in a second kernel, never inside a thread-block cluster  */
#define NK_FLAG_LSU_STORE 0x200000u /* BF16 kernels: store C with per-thread stores, never by TMA             */
#define NK_FLAG_NO_TAIL_SPLIT 0x400000u /* BF16 pair kernel: never cut the tiles of the last, partial wave along K */
#define NK_FLAG_F32_TENSOR 0x800000u /* FP32 operands (row-major, no batch): multiply on the tensor cores.  A and B
                                       are each split into three BF16 planes, x = hi + mid + lo to within 2^-27
                                       of x (a first kernel; the planes take 6 bytes per element of A and B in the
                                       workspace), and the six cross terms that weigh more than 2^-25 of |a||b|
                                       are multiplied by the BF16 kernels as a batch-reduce GEMM with FP32
                                       accumulation, smallest terms first.  BF16 x BF16 products are exact in
                                       FP32, so the result differs from the FP32 product by the dropped terms
                                       (< 2^-24 of sum |a||b|) and the accumulation's rounding: the same error
                                       class as the FMA kernels, not bit-identical to them.  The paper's FP32
                                       path is FMA arithmetic (Algorithm 1); this flag is an opt-in departure
                                       for compute-bound shapes.  Needs N and K multiples of 8.  A value beyond
                                       the largest BF16 (3.39e38) counts as infinite.                        */
#define NK_FLAG_TAIL_SPLIT_SHIFT 24 /* bits 24..27: cut every tile of the last, partial wave into this many equal K
                                      splits (2..8) instead of sharing its k-blocks out evenly over the pairs; 15: share
                                      them out evenly even where the plan's cost model would not */
#define NK_FLAG_RASTER_SHIFT 28 /* bits 28..30: M tiles that sweep N together in the tile raster of the tensor-core
                                   kernels: 0 = 8 (default), 1 = 4, 2 = 6, 3 = 12, 4 = 16, 5 = 24, 6 = 2; 7 = 8 with
                                   every tile's K walked upwards (by default a CTA pair walks K downwards on every
                                   other of its whole tiles, so that a wave of tiles starts on the part of the shared
                                   operand strips that the wave before it read last and finds it in L2; FP32 sums
                                   then differ in their last bits from the upward order, integer sums do not);
                                   bit 31: switch off the serpentine sweep (every other group sweeps N backwards) */
#define NK_FLAG_SPLITK_SHIFT 8    /* bits 8..15: force this many K splits (0 = auto)          */
#define NK_FLAG_TILE_N_SHIFT 16   /* bits 16..19: force tile N: 1=32 2=64 3=128 4=256 (0 = auto) */

typedef struct {
    int64_t M, N, K;
    int32_t in_dtype;  /* nk_dtype_t of A, B and bias                        */
    int32_t out_dtype; /* nk_dtype_t of C: NK_F32, or the operands' 16-bit type      */
    int32_t layout_a;  /* nk_layout_t                                         */
    int32_t layout_b;  /* nk_layout_t                                         */
    int32_t epilogue;  /* nk_epilogue_t                                       */
    int32_t device;    /* CUDA device ordinal                                 */
    uint32_t flags;    /* NK_FLAG_*                                           */
    /* Batch-reduce form of Algorithm 1, C = beta*C + sum_b A_b . B_b (all zero = plain GEMM): */
    int32_t beta;      /* 0: C's old contents are never read; 1: they are added (FP32)  */
    int64_t batch;     /* number of (A_b, B_b) pairs reduced into C; 0 means 1          */
    int64_t stride_a;  /* elements from A_b to A_b+1; 0 means M*K (contiguous)          */
    int64_t stride_b;  /* elements from B_b to B_b+1; 0 means K*N                       */
    /* Batched matmul (Section 5(b): the same nanokernels serve batch.matmul): */
    int64_t stride_c;  /* elements from C_b to C_b+1; 0 means M*N                       */
    int32_t batch_independent; /* 0: the batch is reduced into one C; 1: C_b = A_b . B_b for
                                  every b (bias shared; beta applies to each C_b)        */
    int32_t layout_c;  /* nk_layout_t of C: NK_ROW_MAJOR, or NK_BLOCKED32 = C[M/32][N/32][32][32],
                          the layout a following layer reads as its blocked A (BF16 operands;
                          M and N multiples of 32)                                        */
    float scale;       /* NK_S8 operands with an NK_F32 C (quantised layer: Section 5c names Int8 with
                          quantisation as the next type): C = scale * (A.B), then the epilogue, in FP32;
                          scale is the product of the two operands' quantisation steps and must be
                          finite and non-zero.  The bias of such a plan is FP32.  Ignored otherwise. */
} nk_gemm_desc_t;

/*
 * Build a plan (Section 3.1, register tiling; Section 5(a), tile-size selection:
 * here the choice of kernel, output tile and K split is made once, from the
 * shape).  Validates the descriptor, queries the device, and keeps only host
 * state.  Requirements: M, N, K > 0; blocked layouts need 16-bit or 8-bit operands and the
 * blocked operand's two dimensions to be multiples of 32; row-major BF16 needs N and K
 * to be multiples of 8, row-major FP32 needs N and K to be multiples of 4
 * (16-byte rows); BF16 output needs BF16 inputs.  batch > 1 (Section 2.1: the source tiles
 * of a batch-reduce GEMM need not be contiguous, the accumulation tile is C) takes every
 * item in the operand's layout (row-major, blocked / VNNI-packed as in Listing 1, or B
 * transposed; 16-bit and FP32 operands) and needs strides that are multiples of 8 (16-bit)
 * or 4 (FP32) elements; with
 * beta = 1, y = epilogue(C_old + sum_b A_b.B_b), C_old read in C's own layout.  A blocked C
 * needs BF16 operands and M, N multiples of 32.  On failure *out is NULL.
 */
nk_status_t nk_gemm_create(const nk_gemm_desc_t* desc, nk_gemm_t* out);

/*
 * Bytes of device scratch nk_gemm_run needs for this plan: 0 unless the plan
 * splits K through global memory (FP32 partial tiles, reduced by a second kernel
 * in a fixed order: deterministic; 16-bit plans whose K splits are the CTAs of one
 * thread-block cluster sum them in shared memory instead, in the same order, and
 * need none) or unpacks a blocked operand first.  The caller allocates it; contents need not
 * be initialised and are undefined afterwards.
 */
size_t nk_gemm_workspace_bytes(nk_gemm_t plan);

/*
 * Enqueue C = A.B (+ epilogue) on `cuda_stream` (a cudaStream_t; NULL is the
 * default stream) and return without synchronising (Algorithm 1: tile loop,
 * accumulator resident over the whole K loop, epilogue, one store of C).
 * With desc.beta = 0 C's previous contents are never read; with desc.beta = 1 they
 * are read once and added, in FP32, before the epilogue.  A, B, C (and bias, workspace when
 * used) must be 16-byte aligned device pointers on the plan's device, must not
 * overlap, and must stay valid until the stream reaches the end of the work.
 * bias may be NULL only when the plan has no epilogue.  Nothing is launched
 * when an error is returned.  A plan must not be run from two host threads at
 * once; distinct plans may be.
 */
nk_status_t nk_gemm_run(nk_gemm_t plan, const void* A, const void* B, const void* bias, void* C,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same operation for callers holding HOST buffers (pageable or pinned):
 * copies hA, hB (and hbias) into the caller-provided device staging buffers
 * dA, dB, dbias, runs the plan, copies dC back into hC, and waits for the
 * stream.  Sizes are those implied by the plan's descriptor.  Returns after the
 * result is in hC.  Large single GEMMs (no batch, no beta, row-major C, M a multiple
 * of 2048) are cut into eight chunks of rows and, when N is a multiple of 1024, four
 * panels of columns: uploads of A chunks and B panels alternate, each of the 8 x 4
 * blocks of C is multiplied as soon as its chunk and its panel are on the device and
 * copied back while later uploads are still running, on two internal copy streams
 * (created on the first such call and kept by the plan; pinned host buffers are
 * needed for the overlap to happen).  The staging buffers are scratch: afterwards dB
 * holds B as dense column panels and dC holds C as dense blocks, not the row-major
 * matrices.
 */
nk_status_t nk_gemm_run_host(nk_gemm_t plan, const void* hA, const void* hB, const void* hbias,
                             void* hC, void* dA, void* dB, void* dbias, void* dC, void* workspace,
                             size_t workspace_bytes, void* cuda_stream);

/*
 * Synchronise the plan's device and read the plan's device status word.
 * Every wait inside the kernels (on a TMA or MMA completion barrier) is
 * bounded; a wait that runs out records itself in that word, the kernel drains
 * and exits, and this call returns NK_ERR_TIMEOUT once (the word is cleared;
 * results of the affected run are undefined).  NK_OK otherwise.  The word is a
 * slot of a static device table of the library (1024 slots per device, taken
 * round robin at nk_gemm_create and cleared there; nothing is allocated): a
 * plan reports the waits of its own kernels, unless more than 1024 plans were
 * created on the device since it was.
 */
nk_status_t nk_gemm_check(nk_gemm_t plan);

/*
 * Quantise FP32 values to INT8 for an NK_S8 operand (the quantisation step Section 5c leaves to
 * future work): q[i] = saturate_to_[-128,127](round_to_nearest_even(x[i] * inv_scale)), the product
 * taken in FP32; NaN gives 0.  x and q are device pointers on `device` (x 16-byte aligned when
 * n >= 4), n elements each, they must not overlap; the kernel is enqueued on `cuda_stream` and the
 * call returns without synchronising.  Row-major values in, the same order out: packing B into
 * its blocked layout is the caller's business, like every other operand layout.
 */
nk_status_t nk_quantize_s8(const float* x, int8_t* q, size_t n, float inv_scale, int device, void* cuda_stream);

/*
 * nk_gemm_run for callers that cannot allocate device memory.  (The paper has
 * no counterpart; this is a convenience of the library.)
 *
 * Some callers of a GEMM library may not call cudaMalloc when they need the
 * result: code running inside a region where device allocation is forbidden
 * or would stall (a latency-critical serving loop, a plug-in that is handed
 * buffers but owns no allocator, a process whose memory pool was sized up
 * front and is now full).  A plan that splits K needs scratch for its FP32
 * partial tiles, and nk_gemm_run makes the caller provide it.  This entry
 * point runs the same plan with the scratch taken from a fixed array that is
 * part of the library image instead: NK_STATIC_SCRATCH_BYTES (16 MiB) of
 * device memory, present on every GPU that loads the library, from load until
 * the process exits.  The caller passes only inputs and outputs.
 *
 * - Plans whose nk_gemm_workspace_bytes() exceeds NK_STATIC_SCRATCH_BYTES are
 *   refused with NK_ERR_WORKSPACE and nothing is launched.  Plans that need no
 *   scratch run exactly as with nk_gemm_run.
 * - No cudaMalloc, cudaFree or other allocating call is made, here or in
 *   anything this calls.
 * - The first call on each device looks up the array's device address (once
 *   per device, with that device current).  Make that first call outside any
 *   stream capture.
 * - All calls on a device share the one array, and it keeps whatever the last
 *   call left in it.  The kernels overwrite every partial they later read, so
 *   nothing has to be cleared between calls; but two calls whose GPU work can
 *   overlap (different streams, or different plans run concurrently) race on
 *   it.  Serialise them on one stream.
 * Arguments, alignment rules, asynchrony and error codes are otherwise those of
 * nk_gemm_run.
 */
#define NK_STATIC_SCRATCH_BYTES (16u << 20)
nk_status_t nk_gemm_run_static(nk_gemm_t plan, const void* A, const void* B, const void* bias,
                               void* C, void* cuda_stream);

/*
 * Self-test of the failure path, without a failure: enqueues a one-warp kernel that waits on
 * a barrier nothing signals, with a limit of a few milliseconds.  The wait runs out, the
 * kernel records it in the status word and exits normally, so the next nk_gemm_check
 * returns NK_ERR_TIMEOUT (once) and the context stays usable.  This is how the bounded waits
 * of the GEMM kernels (Algorithm 1's K loop, re-expressed as an mbarrier pipeline) report.
 */
nk_status_t nk_gemm_selftest_timeout(nk_gemm_t plan, void* cuda_stream);

/* Free the plan's host state.  NULL is accepted. */
nk_status_t nk_gemm_destroy(nk_gemm_t plan);

/* Static strings; never NULL. */
const char* nk_status_str(nk_status_t s);
/* Name of the kernel variant the plan selected, e.g. "umma_bf16_128x256x64_s4". */
const char* nk_gemm_kernel_name(nk_gemm_t plan);
/* Number of kernel launches one nk_gemm_run of this plan enqueues. */
int nk_gemm_launches_per_run(nk_gemm_t plan);
/* Message of the last CUDA error a call on this plan captured ("" if none). */
const char* nk_gemm_last_cuda_error(nk_gemm_t plan);

#ifdef __cplusplus
}
#endif
#endif /* NK_GEMM_H */
