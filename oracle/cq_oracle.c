/*
 * CrossQuant CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, by-eye-checkable implementation of the activation cross-quantizer
 * (paper Section 4.2, the CrossQuant equation), of per-token quantization (Eq. 1), of
 * per-channel weight quantization (Eq. 2) and of the quantization kernel (Definition 1).
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may use it.  It
 * shares no code with the CUDA library: its own 16-bit decoders and encoders are written
 * here from the IEEE binary16 / bfloat16 bit layouts.
 *
 * Arithmetic (one rounding per line unless stated), for b-bit codes and 0 <= alpha <= 1:
 *
 *   qmax = 2^(b-1) - 1                                  CrossQuant equation, denominator
 *   x_ij = exact float value of the 16-bit input
 *   t_i  = max_j |x_ij| ,  c_j = max_i |x_ij|           exact (Eq. 1; CrossQuant equation)
 *   alpha == 1 :  a_i = fl32(t_i / qmax),  b_j = 1      exactly Eq. 1 (Table 1 caption:
 *                                                       alpha = 1 is per-token quantization)
 *   alpha == 0 :  a_i = 1,  b_j = fl32(c_j / qmax)      per-column quantization of X
 *   otherwise  :  a_i = fl32( pow_fp64(t_i, alpha) / qmax )
 *                 b_j = fl32( pow_fp64(c_j, 1 - alpha) )
 *                 (the row factor carries 1/qmax, as in the Appendix B.1 listing)
 *   s_ij = fl32(a_i * b_j)                              the per-element scale
 *   s_ij == 0 :  q_ij = 0, xhat_ij = 0                  all-zero row or column
 *   else      :  u = fl32(x_ij / s_ij)
 *                q_ij = round-half-even(u), clamped to [-qmax, qmax]
 *                xhat_ij = fl32(q_ij * s_ij)            then RN-even to 16 bit if asked
 *   |K(CQ)| = #{ (i,j) : q_ij == 0 }                    Definition 1
 *
 * Weights (Eq. 2), per stored row r:  m_r = max_k |w_rk| ; d_r = fl32(m_r / qmax) ;
 *   d_r == 0 -> zeros ; q = round-half-even(fl32(w / d_r)) ; what = fl32(q * d_r).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define CQO_F16 0
#define CQO_BF16 1

/* ---------------------------------------------------------------- 16-bit formats --- */

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static float f16_to_float(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int m = h & 0x3FF;
    float v;
    if (e == 0) {
        v = ldexpf((float)m, -24);                 /* subnormal: m * 2^-24 */
    } else if (e == 31) {
        v = m ? NAN : INFINITY;
    } else {
        v = ldexpf((float)(1024 + m), e - 25);     /* (1 + m/1024) * 2^(e-15) */
    }
    return sign ? -v : v;
}

/* bfloat16: the upper 16 bits of an IEEE binary32. */
static float bf16_to_float(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float v;
    memcpy(&v, &u, 4);
    return v;
}

static float decode16(uint16_t bits, int dtype) {
    return dtype == CQO_F16 ? f16_to_float(bits) : bf16_to_float(bits);
}

/* float -> binary16, round to nearest, ties to even. */
static uint16_t float_to_f16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    float af = fabsf(f);
    if (isnan(f)) return (uint16_t)(sign | 0x7E00u);
    if (af >= 65520.0f) return (uint16_t)(sign | 0x7C00u);   /* midpoint of 65504 and 2^16 rounds up */
    if (af < 6.103515625e-05f) {                             /* below 2^-14: subnormal result */
        /* value = k * 2^-24 with k = round-half-even(af * 2^24); k == 1024 is the smallest normal */
        float k = nearbyintf(ldexpf(af, 24));
        return (uint16_t)(sign | (uint16_t)k);
    }
    uint32_t au = u & 0x7FFFFFFFu;
    uint32_t e32 = au >> 23;                 /* biased by 127 */
    uint32_t m = au & 0x7FFFFFu;
    uint32_t keep = m >> 13;                 /* 10 kept fraction bits */
    uint32_t rest = m & 0x1FFFu;             /* 13 dropped bits */
    uint32_t h = ((e32 - 127u + 15u) << 10) | keep;
    if (rest > 0x1000u || (rest == 0x1000u && (keep & 1u))) h += 1u;  /* carry may bump the exponent */
    return (uint16_t)(sign | (uint16_t)h);
}

/* float -> bfloat16, round to nearest, ties to even. */
static uint16_t float_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if (isnan(f)) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t keep = u >> 16;
    uint32_t rest = u & 0xFFFFu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1u;
    return (uint16_t)keep;
}

static uint16_t encode16(float f, int dtype) {
    return dtype == CQO_F16 ? float_to_f16(f) : float_to_bf16(f);
}

/* exported for the format pins */
void cqo_decode16(const uint16_t* bits, int dtype, int64_t n, float* out) {
    for (int64_t k = 0; k < n; ++k) out[k] = decode16(bits[k], dtype);
}
void cqo_encode16(const float* x, int dtype, int64_t n, uint16_t* out) {
    for (int64_t k = 0; k < n; ++k) out[k] = encode16(x[k], dtype);
}

static int qmax_of(int bits) { return (1 << (bits - 1)) - 1; }

/* ---------------------------------------------------------------- absmax vectors --- */

/* t_i = max_j |x_ij|  (Eq. 1) */
void cqo_absmax_rows(const uint16_t* X, int dtype, int64_t T, int64_t I, int64_t ld, float* t) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < T; ++i) {
        float m = 0.0f;
        for (int64_t j = 0; j < I; ++j) {
            float ax = fabsf(decode16(X[i * ld + j], dtype));
            if (ax > m) m = ax;
        }
        t[i] = m;
    }
}

/* c_j = max_i |x_ij|  (CrossQuant equation) */
void cqo_absmax_cols(const uint16_t* X, int dtype, int64_t T, int64_t I, int64_t ld, float* c) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < I; ++j) {
        float m = 0.0f;
        for (int64_t i = 0; i < T; ++i) {
            float ax = fabsf(decode16(X[i * ld + j], dtype));
            if (ax > m) m = ax;
        }
        c[j] = m;
    }
}

/* ---------------------------------------------------------------- scale vectors ---- */

/* The two factors of the per-element scale: s_ij = fl32(a_i * b_j). */
void cqo_scale_vectors(const float* t, const float* c, int64_t T, int64_t I, double alpha, int bits,
                       float* a, float* b) {
    int qmax = qmax_of(bits);
    for (int64_t i = 0; i < T; ++i) {
        if (alpha == 1.0) a[i] = t[i] / (float)qmax;
        else if (alpha == 0.0) a[i] = 1.0f;
        else a[i] = (float)(pow((double)t[i], alpha) / (double)qmax);
    }
    for (int64_t j = 0; j < I; ++j) {
        if (alpha == 1.0) b[j] = 1.0f;
        else if (alpha == 0.0) b[j] = c[j] / (float)qmax;
        else b[j] = (float)pow((double)c[j], 1.0 - alpha);
    }
}

/* ---------------------------------------------------------------- one element ------ */

static int quantize_one(float x, float s, int qmax, int clamp) {
    if (s == 0.0f) return 0;
    float u = x / s;
    int q = (int)nearbyintf(u);          /* default rounding mode: ties to even */
    if (clamp) {
        if (q > qmax) q = qmax;
        if (q < -qmax) q = -qmax;
    }
    return q;
}

/* ---------------------------------------------------------------- CrossQuant ------- */

/*
 * Activation cross-quantizer.  Every output pointer may be NULL.
 *   codes  : int8 [T*I], one code per element (INT4 codes are also stored one per byte here;
 *            cqo_pack_int4 produces the packed form)
 *   deq32  : float [T*I]     xhat in fp32
 *   deq16  : uint16 [T*I]    xhat rounded to X's 16-bit type
 *   clamp  : 1 = clamp codes to [-qmax, qmax]; 0 = leave them (used by the range pin)
 * Returns 0, or -1 on bad arguments.
 */
int cqo_quantize_act(const uint16_t* X, int dtype, int64_t T, int64_t I, int64_t ld,
                     double alpha, int bits,
                     float* t, float* c, float* a, float* b,
                     int8_t* codes, float* deq32, uint16_t* deq16,
                     uint64_t* zero_count, int clamp) {
    if ((bits != 4 && bits != 8) || !(alpha >= 0.0 && alpha <= 1.0) || ld < I) return -1;
    int qmax = qmax_of(bits);
    float* tt = t ? t : (float*)malloc(sizeof(float) * (size_t)(T > 0 ? T : 1));
    float* cc = c ? c : (float*)malloc(sizeof(float) * (size_t)(I > 0 ? I : 1));
    float* aa = a ? a : (float*)malloc(sizeof(float) * (size_t)(T > 0 ? T : 1));
    float* bb = b ? b : (float*)malloc(sizeof(float) * (size_t)(I > 0 ? I : 1));
    cqo_absmax_rows(X, dtype, T, I, ld, tt);
    cqo_absmax_cols(X, dtype, T, I, ld, cc);
    cqo_scale_vectors(tt, cc, T, I, alpha, bits, aa, bb);
    uint64_t zeros = 0;
#pragma omp parallel for schedule(static) reduction(+ : zeros)
    for (int64_t i = 0; i < T; ++i) {
        for (int64_t j = 0; j < I; ++j) {
            float x = decode16(X[i * ld + j], dtype);
            float s = aa[i] * bb[j];
            int q = quantize_one(x, s, qmax, clamp);
            float xhat = (s == 0.0f) ? 0.0f : (float)q * s;
            if (q == 0) zeros += 1;
            if (codes) codes[i * I + j] = (int8_t)q;
            if (deq32) deq32[i * I + j] = xhat;
            if (deq16) deq16[i * I + j] = encode16(xhat, dtype);
        }
    }
    if (zero_count) *zero_count = zeros;
    if (!t) free(tt);
    if (!c) free(cc);
    if (!a) free(aa);
    if (!b) free(bb);
    return 0;
}

/* INT4 storage: element (i, 2k) in the low nibble and (i, 2k+1) in the high nibble of byte
 * i*(I/2)+k, two's-complement nibbles. */
int cqo_pack_int4(const int8_t* codes, int64_t T, int64_t I, uint8_t* packed) {
    if (I % 2) return -1;
    for (int64_t i = 0; i < T; ++i)
        for (int64_t k = 0; k < I / 2; ++k) {
            uint8_t lo = (uint8_t)codes[i * I + 2 * k] & 0xF;
            uint8_t hi = (uint8_t)codes[i * I + 2 * k + 1] & 0xF;
            packed[i * (I / 2) + k] = (uint8_t)(lo | (hi << 4));
        }
    return 0;
}

static int code_at(const void* codes, int bits, int64_t I, int64_t i, int64_t j) {
    if (bits == 8) return ((const int8_t*)codes)[i * I + j];
    uint8_t byte = ((const uint8_t*)codes)[i * (I / 2) + j / 2];
    int nib = (j & 1) ? (byte >> 4) : (byte & 0xF);
    return nib >= 8 ? nib - 16 : nib;
}

/* xhat_ij = fl32(q_ij * fl32(a_i * b_j)) from stored codes (INT8, or packed INT4). */
void cqo_dequantize(const void* codes, int bits, int64_t T, int64_t I, const float* a, const float* b,
                    float* out32, uint16_t* out16, int dtype16) {
    for (int64_t i = 0; i < T; ++i)
        for (int64_t j = 0; j < I; ++j) {
            float s = a[i] * b[j];
            int q = code_at(codes, bits, I, i, j);
            float xhat = (s == 0.0f) ? 0.0f : (float)q * s;
            if (out32) out32[i * I + j] = xhat;
            if (out16) out16[i * I + j] = encode16(xhat, dtype16);
        }
}

/* |K| = number of zero codes (Definition 1), from stored codes. */
uint64_t cqo_kernel_count(const void* codes, int bits, int64_t T, int64_t I) {
    uint64_t n = 0;
    for (int64_t i = 0; i < T; ++i)
        for (int64_t j = 0; j < I; ++j)
            if (code_at(codes, bits, I, i, j) == 0) n += 1;
    return n;
}

/* ---------------------------------------------------------------- weights (Eq. 2) -- */

int cqo_quantize_weight_per_channel(const uint16_t* W, int dtype, int64_t R, int64_t C, int64_t ld, int bits,
                                    int8_t* codes, float* scale, float* deq32, uint16_t* deq16,
                                    uint64_t* zero_count) {
    if ((bits != 4 && bits != 8) || ld < C) return -1;
    int qmax = qmax_of(bits);
    uint64_t zeros = 0;
#pragma omp parallel for schedule(static) reduction(+ : zeros)
    for (int64_t r = 0; r < R; ++r) {
        float m = 0.0f;
        for (int64_t k = 0; k < C; ++k) {
            float aw = fabsf(decode16(W[r * ld + k], dtype));
            if (aw > m) m = aw;
        }
        float d = m / (float)qmax;
        if (scale) scale[r] = d;
        for (int64_t k = 0; k < C; ++k) {
            float w = decode16(W[r * ld + k], dtype);
            int q = quantize_one(w, d, qmax, 1);
            float what = (d == 0.0f) ? 0.0f : (float)q * d;
            if (q == 0) zeros += 1;
            if (codes) codes[r * C + k] = (int8_t)q;
            if (deq32) deq32[r * C + k] = what;
            if (deq16) deq16[r * C + k] = encode16(what, dtype);
        }
    }
    if (zero_count) *zero_count = zeros;
    return 0;
}

/* ---------------------------------------------------------------- diagnostics ------ */

static int64_t ulp_distance(float p, float q) {
    int32_t ip, iq;
    memcpy(&ip, &p, 4);
    memcpy(&iq, &q, 4);
    int64_t d = (int64_t)ip - (int64_t)iq;
    return d < 0 ? -d : d;
}

/*
 * Compare the fp32 factored evaluation with the CrossQuant equation evaluated in fp64:
 *   s_ideal = pow(t_i, alpha) * pow(c_j, 1-alpha) / qmax ,  q_ideal = round-half-even(x / s_ideal).
 * out[0] = largest fp32-ulp distance between s_ij and fl32(s_ideal) over non-zero scales
 * out[1] = number of elements whose code differs from q_ideal
 * out[2] = of those, how many have |x / s_ideal| farther than `rel` (relative) from every k + 1/2
 */
void cqo_compare_with_ideal(const uint16_t* X, int dtype, int64_t T, int64_t I, int64_t ld,
                            double alpha, int bits, const float* t, const float* c,
                            const float* a, const float* b, const int8_t* codes, double rel,
                            int64_t* out) {
    int qmax = qmax_of(bits);
    int64_t max_ulp = 0, differ = 0, far = 0;
    for (int64_t i = 0; i < T; ++i)
        for (int64_t j = 0; j < I; ++j) {
            float s = a[i] * b[j];
            double s_ideal = pow((double)t[i], alpha) * pow((double)c[j], 1.0 - alpha) / (double)qmax;
            if (s == 0.0f || s_ideal == 0.0) continue;
            int64_t d = ulp_distance(s, (float)s_ideal);
            if (d > max_ulp) max_ulp = d;
            double u = (double)decode16(X[i * ld + j], dtype) / s_ideal;
            int q_ideal = (int)nearbyint(u);
            if (q_ideal != codes[i * I + j]) {
                differ += 1;
                double au = fabs(u);
                double boundary = floor(au) + 0.5;
                if (fabs(au - boundary) > rel * boundary) far += 1;
            }
        }
    out[0] = max_ulp;
    out[1] = differ;
    out[2] = far;
}

/* ---------------------------------------------------------------- Remove Kernel ---- */

/*
 * The "Remove Kernel" operator of Figure 1 and Appendix B: the elements of the quantization kernel are
 * set to zero and every other element is left as it is (not quantized).
 *   removed  <=>  |u_ij| <= bound_scale / 2,  u_ij = fl32(x_ij / s_ij)  (s_ij == 0 counts as removed);
 *   bound_scale = 1 removes exactly K(CQ) for this alpha (|u| <= 1/2  <=>  round-half-even(u) == 0);
 *   other values scale the zero bound B~ and so sweep the removed proportion (Section 4.3).
 * out16[T*I]: x or +0.  counts[0] = removed, counts[1] = |K(Q)| of per-token quantization (Eq. 1),
 * counts[2] = |K(CQ)| for this alpha -- all three from one pass over X.
 */
int cqo_remove_kernel(const uint16_t* X, int dtype, int64_t T, int64_t I, int64_t ld, double alpha, int bits,
                      float bound_scale, uint16_t* out16, uint64_t* counts) {
    if ((bits != 4 && bits != 8) || !(alpha >= 0.0 && alpha <= 1.0) || ld < I || !(bound_scale >= 0.0f)) return -1;
    int qmax = qmax_of(bits);
    float* t = (float*)malloc(sizeof(float) * (size_t)(T > 0 ? T : 1));
    float* c = (float*)malloc(sizeof(float) * (size_t)(I > 0 ? I : 1));
    float* a = (float*)malloc(sizeof(float) * (size_t)(T > 0 ? T : 1));
    float* b = (float*)malloc(sizeof(float) * (size_t)(I > 0 ? I : 1));
    cqo_absmax_rows(X, dtype, T, I, ld, t);
    cqo_absmax_cols(X, dtype, T, I, ld, c);
    cqo_scale_vectors(t, c, T, I, alpha, bits, a, b);
    float half_bound = 0.5f * bound_scale;
    uint64_t removed = 0, k_pt = 0, k_cq = 0;
#pragma omp parallel for schedule(static) reduction(+ : removed, k_pt, k_cq)
    for (int64_t i = 0; i < T; ++i) {
        float s_pt = t[i] / (float)qmax;
        for (int64_t j = 0; j < I; ++j) {
            uint16_t bits16 = X[i * ld + j];
            float x = decode16(bits16, dtype);
            float s = a[i] * b[j];
            float u = (s == 0.0f) ? 0.0f : x / s;
            int gone = fabsf(u) <= half_bound;
            if (gone) removed += 1;
            if (quantize_one(x, s, qmax, 1) == 0) k_cq += 1;
            if (quantize_one(x, s_pt, qmax, 1) == 0) k_pt += 1;
            if (out16) out16[i * I + j] = gone ? (uint16_t)0 : bits16;
        }
    }
    counts[0] = removed;
    counts[1] = k_pt;
    counts[2] = k_cq;
    free(t); free(c); free(a); free(b);
    return 0;
}

/* ---------------------------------------------------------------- Table 1 indicators */

/*
 * The two indicators of Table 1 (Section 4.2, Cases I / II), over all (i, j) pairs of one matrix:
 *   out[0] = #{ (i,j) : c_j >= t_i }                                   (Case II)
 *   out[1] = #{ (i,j) : B~_ij < B_ij } with the zero bounds B~ = s_ij / 2, B = fl32(t_i / qmax) / 2,
 *            s_ij = fl32(a_i * b_j) the scale the quantizer uses for this alpha.
 */
void cqo_case_indicators(const float* t, const float* c, const float* a, const float* b,
                         int64_t T, int64_t I, int bits, uint64_t* out) {
    int qmax = qmax_of(bits);
    uint64_t n_case2 = 0, n_smaller = 0;
#pragma omp parallel for schedule(static) reduction(+ : n_case2, n_smaller)
    for (int64_t i = 0; i < T; ++i) {
        float s_pt = t[i] / (float)qmax;
        for (int64_t j = 0; j < I; ++j) {
            float s = a[i] * b[j];
            if (c[j] >= t[i]) n_case2 += 1;
            if (0.5f * s < 0.5f * s_pt) n_smaller += 1;
        }
    }
    out[0] = n_case2;
    out[1] = n_smaller;
}

/* Number of OpenMP threads later calls may use (timing only: results do not depend on it).  n < 1 is ignored. */
void cqo_set_num_threads(int n) {
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int cqo_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
