/*
 * CPU oracle for the dense GEMM path.  TEST INFRASTRUCTURE ONLY: nothing on the
 * product path may call, link or import this file; it shares no code, header,
 * table or constant with the CUDA library.
 *
 * What it computes is the plain definition the method reaches up to summation
 * order (Algorithm 1: C = beta*C + sum_i A_i x B_i, taken with beta = 0):
 *
 *     C[i][j] = sum_{k=0}^{K-1} a(i,k) * b(k,j)       accumulated in FP64, k ascending
 *     y[i][j] = C[i][j]                               (no epilogue)
 *     y[i][j] = max(C[i][j] + bias[j], 0)             (bias + ReLU fused before the store,
 *                                                      Section 6 "MLP")
 *     S[i][j] = sum_k |a(i,k) * b(k,j)| (+ |bias[j]|) (scale of the error bound)
 *
 * a, b are the stored operand values: FP32, or BF16 widened exactly to FP32 (the
 * appendix kernels' scalar body: extf, extf, mulf, addf), or FP16 (IEEE binary16, the
 * other 16-bit type the paper's Section 5 names as the next packed type) widened
 * exactly.  y is returned unrounded, as double; a BF16- or FP16-storing
 * implementation rounds once afterwards.
 *
 * Layouts: row-major A[M][K], B[K][N] (B may also be kept as its transpose Bt[N][K], an
 * indexing variant of the same matrix); or 32x32-blocked with the VNNI-2
 * interleave of Figure 1 inside each B block:
 *     A_blk[M/32][K/32][32][32]         (m-block, k-block, m-in-block, k-in-block)
 *     B_blk[N/32][K/32][16][32][2]      (n-block, k-block, k-pair, n-in-block, k-parity)
 *
 * INT8 (Section 5c, "other packed types": the Int8 dot product, whose operands Section 2
 * packs in groups of four): nko_gemm_s8 computes C[i][j] = sum_k a(i,k) * b(k,j) in integers,
 * exactly (int64 accumulation; results fit int32 while K < 2^17).  A is row-major; B is
 * row-major or 32x32-blocked with Figure 1's rule at group size four:
 *     B_blk4[N/32][K/32][8][32][4]      (n-block, k-block, k-quad, n-in-block, k mod 4)
 *
 * Pins (tests/test_oracle_*.py): Figure 1's printed packing, identity /
 * permutation / diagonal / rank-1 / all-ones closed forms, brute force in a
 * different loop order, numpy float64 matmul on small shapes, blocked-vs-flat
 * bit equality, epilogue closed forms, exhaustive BF16 codec round trip, exhaustive FP16
 * decode against the IEEE reading.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { NKO_F32 = 0, NKO_BF16 = 1, NKO_F16 = 2, NKO_E4M3 = 5, NKO_E5M2 = 6 };
enum { NKO_ROW = 0, NKO_BLOCKED32 = 1, NKO_TRANSPOSED = 2 };   /* TRANSPOSED: layout_b only, Bt[N][K] */
enum { NKO_EPI_NONE = 0, NKO_EPI_BIAS_RELU = 1 };
enum { NKO_ACC_F64 = 0, NKO_ACC_F32_SEQ = 1 };

typedef struct {
    int64_t M, N, K;
    int32_t in_dtype;   /* NKO_F32 | NKO_BF16 | NKO_F16: element type of A, B and bias;
                           NKO_E4M3 | NKO_E5M2: 8-bit floating-point A and B, FP32 bias */
    int32_t layout_a;   /* NKO_ROW | NKO_BLOCKED32 */
    int32_t layout_b;
    int32_t epilogue;
    int32_t acc_mode;   /* NKO_ACC_F64 (the oracle) | NKO_ACC_F32_SEQ (tolerance sanity only) */
} nko_desc_t;

/* BF16 -> FP32 is a 16-bit left shift of the bit pattern (Algorithm 2, fallback branch). */
float nko_bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* IEEE 754 binary16 -> FP32, written from the format's definition: 1 sign bit, 5 exponent bits
   (bias 15), 10 fraction bits; exponent 0 is zero or a subnormal (fraction * 2^-24), exponent 31
   is infinity or NaN, otherwise (1 + fraction / 1024) * 2^(exponent - 15).  Every binary16 value
   is exactly representable in FP32. */
float nko_f16_to_f32(uint16_t h) {
    int sign = (h >> 15) & 1, e = (h >> 10) & 0x1F, m = h & 0x3FF;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)m / 1024.0, e - 15);
    return (float)(sign ? -v : v);
}

/* The two 8-bit floating-point formats of the OCP FP8 specification, written from their
   definitions; every value is exactly representable in FP32.
   E4M3: 1 sign bit, 4 exponent bits (bias 7), 3 fraction bits; exponent 0 is zero or a subnormal
   (fraction * 2^-9); there are no infinities, and only exponent 15 with fraction 7 is NaN, so the
   largest finite value is 1.75 * 2^8 = 448.
   E5M2: 1 sign bit, 5 exponent bits (bias 15), 2 fraction bits, IEEE rules: exponent 0 is zero or
   a subnormal (fraction * 2^-16), exponent 31 is infinity (fraction 0) or NaN. */
float nko_e4m3_to_f32(uint8_t h) {
    int sign = (h >> 7) & 1, e = (h >> 3) & 0xF, m = h & 7;
    double v;
    if (e == 0) v = ldexp((double)m, -9);
    else if (e == 15 && m == 7) v = NAN;
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return (float)(sign ? -v : v);
}

float nko_e5m2_to_f32(uint8_t h) {
    int sign = (h >> 7) & 1, e = (h >> 2) & 0x1F, m = h & 3;
    double v;
    if (e == 0) v = ldexp((double)m, -16);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)m / 4.0, e - 15);
    return (float)(sign ? -v : v);
}

/* FP32 -> BF16, round to nearest, ties to even (finite inputs). */
uint16_t nko_f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t keep = u >> 16, rest = u & 0xFFFFu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1;
    return (uint16_t)keep;
}

/* Figure 1: packed[k/2][n][k%2] = flat[k][n]; K even. */
void nko_pack_vnni2(const uint16_t* flat, int64_t K, int64_t N, uint16_t* packed) {
    for (int64_t k = 0; k < K; ++k)
        for (int64_t n = 0; n < N; ++n)
            packed[((k / 2) * N + n) * 2 + (k % 2)] = flat[k * N + n];
}

void nko_unpack_vnni2(const uint16_t* packed, int64_t K, int64_t N, uint16_t* flat) {
    for (int64_t k = 0; k < K; ++k)
        for (int64_t n = 0; n < N; ++n)
            flat[k * N + n] = packed[((k / 2) * N + n) * 2 + (k % 2)];
}

static int64_t a_index(const nko_desc_t* d, int64_t i, int64_t k) {
    if (d->layout_a == NKO_ROW) return i * d->K + k;
    return (((i / 32) * (d->K / 32) + k / 32) * 32 + i % 32) * 32 + k % 32;
}

static int is_8bit(int32_t dtype) { return dtype == NKO_E4M3 || dtype == NKO_E5M2; }

static int64_t b_index(const nko_desc_t* d, int64_t k, int64_t j) {
    if (d->layout_b == NKO_ROW) return k * d->N + j;
    if (d->layout_b == NKO_TRANSPOSED) return j * d->K + k;   /* B kept as its transpose, K contiguous */
    if (is_8bit(d->in_dtype))   /* 8-bit elements are packed in groups of four (Section 2) */
        return ((((j / 32) * (d->K / 32) + k / 32) * 8 + (k % 32) / 4) * 32 + j % 32) * 4 + k % 4;
    return ((((j / 32) * (d->K / 32) + k / 32) * 16 + (k % 32) / 2) * 32 + j % 32) * 2 + k % 2;
}

/* Storage index of logical element (i,k) of A / (k,j) of B: exported so tests can pack. */
int64_t nko_a_index(const nko_desc_t* d, int64_t i, int64_t k) { return a_index(d, i, k); }
int64_t nko_b_index(const nko_desc_t* d, int64_t k, int64_t j) { return b_index(d, k, j); }

static double load(const void* p, int32_t dtype, int64_t idx) {
    if (dtype == NKO_F32) return (double)((const float*)p)[idx];
    if (dtype == NKO_F16) return (double)nko_f16_to_f32(((const uint16_t*)p)[idx]);
    if (dtype == NKO_E4M3) return (double)nko_e4m3_to_f32(((const uint8_t*)p)[idx]);
    if (dtype == NKO_E5M2) return (double)nko_e5m2_to_f32(((const uint8_t*)p)[idx]);
    return (double)nko_bf16_to_f32(((const uint16_t*)p)[idx]);
}

typedef struct {
    const nko_desc_t* d;
    const void *A, *B, *bias;
    const int64_t *rows, *cols;
    int64_t r0, r1, ncols;
    double *Y, *S;
} job_t;

static void* worker(void* arg) {
    job_t* w = (job_t*)arg;
    const nko_desc_t* d = w->d;
    int64_t nc = w->ncols;
    float* accf = NULL;
    if (d->acc_mode == NKO_ACC_F32_SEQ) accf = (float*)malloc(sizeof(float) * (size_t)nc);
    for (int64_t r = w->r0; r < w->r1; ++r) {
        int64_t i = w->rows ? w->rows[r] : r;
        double* y = w->Y + r * nc;
        double* s = w->S ? w->S + r * nc : NULL;
        for (int64_t c = 0; c < nc; ++c) y[c] = 0.0;
        if (s) for (int64_t c = 0; c < nc; ++c) s[c] = 0.0;
        if (accf) for (int64_t c = 0; c < nc; ++c) accf[c] = 0.0f;
        /* k outermost of the two inner loops: every y[c] still receives its
           products in ascending k, exactly as the definition's sum is written. */
        for (int64_t k = 0; k < d->K; ++k) {
            double a = load(w->A, d->in_dtype, a_index(d, i, k));
            for (int64_t c = 0; c < nc; ++c) {
                int64_t j = w->cols ? w->cols[c] : c;
                double p = a * load(w->B, d->in_dtype, b_index(d, k, j));
                if (accf) accf[c] = accf[c] + (float)p; else y[c] += p;
                if (s) s[c] += fabs(p);
            }
        }
        if (accf) for (int64_t c = 0; c < nc; ++c) y[c] = (double)accf[c];
        if (d->epilogue == NKO_EPI_BIAS_RELU) {
            for (int64_t c = 0; c < nc; ++c) {
                int64_t j = w->cols ? w->cols[c] : c;
                double b = load(w->bias, is_8bit(d->in_dtype) ? NKO_F32 : d->in_dtype, j);
                double v = y[c] + b;
                y[c] = v > 0.0 ? v : 0.0;
                if (s) s[c] += fabs(b);
            }
        }
    }
    free(accf);
    return NULL;
}

/*
 * rows: list of nrows row indices, or NULL for rows 0..nrows-1.
 * cols: list of ncols column indices, or NULL for columns 0..ncols-1.
 * Y, S: [nrows][ncols] doubles (S may be NULL).  Threads split the row list
 * statically; the result does not depend on nthreads.  Returns 0, or -1 on
 * invalid arguments.
 */
int nko_gemm(const nko_desc_t* d, const void* A, const void* B, const void* bias,
             const int64_t* rows, int64_t nrows, const int64_t* cols, int64_t ncols,
             double* Y, double* S, int nthreads) {
    if (!d || !A || !B || !Y || d->M <= 0 || d->N <= 0 || d->K <= 0) return -1;
    if (d->epilogue == NKO_EPI_BIAS_RELU && !bias) return -1;
    if (d->layout_a == NKO_BLOCKED32 && (d->M % 32 || d->K % 32)) return -1;
    if (d->layout_b == NKO_BLOCKED32 && (d->N % 32 || d->K % 32)) return -1;
    if (nrows <= 0 || ncols <= 0) return -1;
    if (nthreads < 1) nthreads = 1;
    if (nthreads > nrows) nthreads = (int)nrows;
    pthread_t* th = (pthread_t*)malloc(sizeof(pthread_t) * (size_t)nthreads);
    job_t* jobs = (job_t*)malloc(sizeof(job_t) * (size_t)nthreads);
    for (int t = 0; t < nthreads; ++t) {
        job_t j = { d, A, B, bias, rows, cols, nrows * t / nthreads, nrows * (t + 1) / nthreads,
                    ncols, Y, S };
        jobs[t] = j;
        if (t > 0) pthread_create(&th[t], NULL, worker, &jobs[t]);
    }
    worker(&jobs[0]);
    for (int t = 1; t < nthreads; ++t) pthread_join(th[t], NULL);
    free(th);
    free(jobs);
    return 0;
}

/*
 * Batch-reduce GEMM, the output line of Algorithm 1 written out:
 *
 *     C[i][j] = beta * C0[i][j] + sum_{b=0}^{batch-1} sum_{k=0}^{K-1} a_b(i,k) * b_b(k,j)
 *
 * with the batch-reduce loop outside the K loop, as in the algorithm.  Row-major
 * operands; A_b starts stride_a elements after A_{b-1}, B_b stride_b after B_{b-1} (the
 * tiles need not be contiguous, Section 2.1).  beta is 0 or 1 (C0 may be NULL when 0);
 * C0 holds the stored values of C widened to double.  FP64 accumulation, then the same
 * epilogue as nko_gemm.  S receives sum |a.b| + |beta.C0| (+ |bias|).  Plain loops, one
 * thread: this is the definition, used on test sizes only.
 */
int nko_brgemm_layout(int64_t M, int64_t N, int64_t K, int64_t batch, int64_t stride_a, int64_t stride_b,
                      int32_t in_dtype, int32_t layout_a, int32_t layout_b, int32_t epilogue, double beta,
                      const void* A, const void* B, const void* bias, const double* C0, double* Y, double* S) {
    if (!A || !B || !Y || M <= 0 || N <= 0 || K <= 0 || batch <= 0) return -1;
    if (beta != 0.0 && beta != 1.0) return -1;
    if (beta != 0.0 && !C0) return -1;
    if (epilogue == NKO_EPI_BIAS_RELU && !bias) return -1;
    if (layout_a == NKO_BLOCKED32 && (M % 32 || K % 32)) return -1;
    if (layout_b == NKO_BLOCKED32 && (N % 32 || K % 32)) return -1;
    /* every batch item is one operand in the given layout (Listing 1: VNNI-packed items), item b
     * starting b * stride elements into the buffer; inside an item the index formulas of nko_gemm */
    nko_desc_t d = {M, N, K, in_dtype, layout_a, layout_b, epilogue, NKO_ACC_F64};
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double acc = beta != 0.0 ? beta * C0[i * N + j] : 0.0;
            double s = fabs(acc);
            for (int64_t b = 0; b < batch; ++b) {
                for (int64_t k = 0; k < K; ++k) {
                    double p = load(A, in_dtype, b * stride_a + a_index(&d, i, k)) *
                               load(B, in_dtype, b * stride_b + b_index(&d, k, j));
                    acc += p;
                    s += fabs(p);
                }
            }
            if (epilogue == NKO_EPI_BIAS_RELU) {
                double bv = load(bias, in_dtype, j);
                acc += bv;
                s += fabs(bv);
                if (!(acc > 0.0)) acc = 0.0;
            }
            Y[i * N + j] = acc;
            if (S) S[i * N + j] = s;
        }
    }
    return 0;
}

/* The row-major form (the first interface): the same loops with row-major index formulas. */
int nko_brgemm(int64_t M, int64_t N, int64_t K, int64_t batch, int64_t stride_a, int64_t stride_b,
               int32_t in_dtype, int32_t epilogue, double beta, const void* A, const void* B,
               const void* bias, const double* C0, double* Y, double* S) {
    return nko_brgemm_layout(M, N, K, batch, stride_a, stride_b, in_dtype, NKO_ROW, NKO_ROW, epilogue, beta,
                             A, B, bias, C0, Y, S);
}

/* ------------------------------------------------------------------ INT8
 * Figure 1's packing rule with groups of four along k (Section 2: "INT8 elements in groups
 * of four"): packed[k/4][n][k%4] = flat[k][n]. */
void nko_pack_vnni4(const int8_t* flat, int64_t K, int64_t N, int8_t* packed) {
    for (int64_t k = 0; k < K; ++k)
        for (int64_t n = 0; n < N; ++n)
            packed[((k / 4) * N + n) * 4 + (k % 4)] = flat[k * N + n];
}

void nko_unpack_vnni4(const int8_t* packed, int64_t K, int64_t N, int8_t* flat) {
    for (int64_t k = 0; k < K; ++k)
        for (int64_t n = 0; n < N; ++n)
            flat[k * N + n] = packed[((k / 4) * N + n) * 4 + (k % 4)];
}

/* Storage index of logical element (k,j) of an INT8 B operand. */
int64_t nko_b_index_s8(int64_t K, int64_t N, int32_t layout_b, int64_t k, int64_t j) {
    if (layout_b == NKO_ROW) return k * N + j;
    if (layout_b == NKO_TRANSPOSED) return j * K + k;
    return ((((j / 32) * (K / 32) + k / 32) * 8 + (k % 32) / 4) * 32 + j % 32) * 4 + k % 4;
}

typedef struct {
    int64_t M, N, K;
    int32_t layout_b;
    const int8_t *A, *B;
    const int64_t* rows;
    int64_t r0, r1;
    int64_t* Y;
} job_s8_t;

static void* worker_s8(void* arg) {
    job_s8_t* w = (job_s8_t*)arg;
    for (int64_t r = w->r0; r < w->r1; ++r) {
        const int64_t i = w->rows ? w->rows[r] : r;
        for (int64_t j = 0; j < w->N; ++j) {
            int64_t acc = 0;
            for (int64_t k = 0; k < w->K; ++k)
                acc += (int64_t)w->A[i * w->K + k] * (int64_t)w->B[nko_b_index_s8(w->K, w->N, w->layout_b, k, j)];
            w->Y[r * w->N + j] = acc;
        }
    }
    return NULL;
}

/* Y[r][j] (int64) for the listed rows (all M rows when rows == NULL).  Returns 0, or -1 on bad arguments. */
int nko_gemm_s8(int64_t M, int64_t N, int64_t K, int32_t layout_b, const int8_t* A, const int8_t* B,
                const int64_t* rows, int64_t nrows, int64_t* Y, int nthreads) {
    if (M <= 0 || N <= 0 || K <= 0 || !A || !B || !Y) return -1;
    if (layout_b != NKO_ROW && layout_b != NKO_TRANSPOSED && (layout_b != NKO_BLOCKED32 || N % 32 || K % 32)) return -1;
    const int64_t nr = rows ? nrows : M;
    if (rows)
        for (int64_t r = 0; r < nr; ++r)
            if (rows[r] < 0 || rows[r] >= M) return -1;
    if (nthreads < 1) nthreads = 1;
    if (nthreads > 64) nthreads = 64;
    if (nthreads > nr) nthreads = (int)nr;
    pthread_t th[64];
    job_s8_t jobs[64];
    for (int t = 0; t < nthreads; ++t) {
        job_s8_t j = {M, N, K, layout_b, A, B, rows, nr * t / nthreads, nr * (t + 1) / nthreads, Y};
        jobs[t] = j;
        if (pthread_create(&th[t], NULL, worker_s8, &jobs[t]) != 0) return -1;
    }
    for (int t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
    return 0;
}

/* Quantisation to INT8 (Section 5c leaves "quantization support" to future work; the reading taken
 * here is the usual symmetric one): q = the FP32 product x * inv_scale, rounded to the nearest
 * integer with ties to even, saturated to [-128, 127]; NaN gives 0. */
void nko_quantize_s8(const float* x, int64_t n, float inv_scale, int8_t* q) {
    for (int64_t i = 0; i < n; ++i) {
        volatile float p = x[i] * inv_scale;      /* one FP32 rounding, kept out of wider registers */
        if (p != p) { q[i] = 0; continue; }
        if (p >= 127.0f) { q[i] = 127; continue; }
        if (p <= -128.0f) { q[i] = -128; continue; }
        q[i] = (int8_t)lrintf(p);                 /* default rounding mode: to nearest, ties to even */
    }
}
