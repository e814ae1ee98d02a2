/*
 * Reference (oracle) implementation of the structured contraction ops (and, at the end of the
 * file, of the depthwise convolutions and of the memory-bound 2-D kernels).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a deliberately plain,
 * slow CPU evaluation of each op's definition, used only to check the CUDA
 * library and to be timed beside it as a baseline.  It shares no code with the
 * CUDA path and the CUDA path never calls it.
 *
 * Each op is the literal loop nest over its iteration domain, reading every
 * operand through its indexing map and its element strides, with one f64
 * accumulator per output element:
 *
 *   matmul  (Section 4.6.1, equation "AB"):
 *       C[m,n] = sum_k A[m,k] * B[k,n]
 *       iterators (m,n,k) = (parallel, parallel, reduction)
 *   conv_1d_nwc_wcf  (Section 3, index notation; Section 4.6.2, "(1-D)"):
 *       O[n,w,f] = sum_{kw,c} I[n, w*Sw + kw*Dw, c] * K[kw,c,f]
 *       domain 0<=n<O.0, 0<=w<O.1, 0<=f<O.2, 0<=kw<K.0, 0<=c<K.1
 *   conv_2d_nhwc_hwcf  (Section 4.6.2, "(2-D)"):
 *       O[n,h,w,f] = sum_{kh,kw,c} I[n, h*Sh + kh*Dh, w*Sw + kw*Dw, c] * K[kh,kw,c,f]
 *
 * The "." in the paper's expressions is an implicit sum over every iterator
 * that does not appear on the left-hand side.  The filter is not flipped
 * (index is w + kw) and there is no padding: the domain is bounded by the
 * output and filter sizes and the input must be large enough.
 *
 * Inputs are f32 (for the bf16 path the caller passes bf16-representable
 * values widened to f32).  Outputs are f64.  `S`, when non-NULL, receives
 * sum |a*b| per output element (dense row-major over the output's named dim
 * order); it is the scale of the comparison bound |err| <= 1e-4 * S.
 * `mode` 0 overwrites the output, mode 1 adds to the value already there
 * (destination-passing: the output operand is in/out, Section 3.4).
 *
 * The `_points` variants evaluate only listed output coordinates, for checking
 * sampled elements of full-size problems; they are the same inner loops.
 *
 * Parallelism: the outermost parallel iterator is split across OpenMP threads;
 * nothing else is blocked, fused, reordered or vectorised by hand.
 */
#include <stdint.h>
#include <stddef.h>
#include <math.h>

#include "sg_ref.h"    /* the declarations of everything below: the compiler checks that they agree */
#ifdef _OPENMP
#include <omp.h>
#endif

static int use_threads(int threads) {
#ifdef _OPENMP
    if (threads <= 0) threads = omp_get_max_threads();
    return threads;
#else
    (void)threads;
    return 1;
#endif
}

int sg_ref_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* C[m,n] (+)= sum_k A[m,k]*B[k,n]; strides in elements. */
int sg_ref_matmul(int64_t M, int64_t N, int64_t K,
                  const float *A, int64_t a_sm, int64_t a_sk,
                  const float *B, int64_t b_sk, int64_t b_sn,
                  double *C, int64_t c_sm, int64_t c_sn,
                  double *S, int mode, int threads)
{
    if (M < 0 || N < 0 || K < 0) return 1;
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0, sab = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double p = (double)A[m * a_sm + k * a_sk] * (double)B[k * b_sk + n * b_sn];
                acc += p;
                sab += fabs(p);
            }
            double *c = &C[m * c_sm + n * c_sn];
            *c = (mode ? *c : 0.0) + acc;
            if (S) S[m * N + n] = sab;
        }
    }
    return 0;
}

/*
 * Matmul with a fused pointwise consumer (Section 2.1: tensor operations are fused at the tiled level; Section 3.3,
 * items 1 and 2 of the vectorization cases: a pointwise op has identity indexing maps, a lower-dimensional operand
 * is broadcast).  The consumer is the generic op with maps (m,n)->(m,n) for the product, (m,n)->(n) for the bias
 * and (m,n)->(m,n) for the result, and body  r = act(p + b):
 *     C[m,n] = act( sum_k A[m,k]*B[k,n] + bias[n] ),   act = identity (0) or max(., 0) (1).
 * Evaluated the unfused way: the whole sum first, in f64, then the consumer on it.  bias may be NULL (no bias).
 * S (optional) = sum_k |a*b| + |bias[n]|: the scale of the comparison bound.
 */
int sg_ref_matmul_bias_act(int64_t M, int64_t N, int64_t K,
                           const float *A, int64_t a_sm, int64_t a_sk,
                           const float *B, int64_t b_sk, int64_t b_sn,
                           const float *bias, int64_t bias_sn, int act,
                           double *C, int64_t c_sm, int64_t c_sn,
                           double *S, int threads)
{
    if (M < 0 || N < 0 || K < 0 || (act != 0 && act != 1)) return 1;
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0, sab = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double p = (double)A[m * a_sm + k * a_sk] * (double)B[k * b_sk + n * b_sn];
                acc += p;
                sab += fabs(p);
            }
            double b = bias ? (double)bias[n * bias_sn] : 0.0;
            double r = acc + b;
            if (act == 1 && r < 0.0) r = 0.0;
            C[m * c_sm + n * c_sn] = r;
            if (S) S[m * N + n] = sab + fabs(b);
        }
    }
    return 0;
}

/* Selected elements only: (pm[i], pn[i]) -> out[i], sabs[i]. No accumulate input. */
int sg_ref_matmul_points(int64_t K,
                         const float *A, int64_t a_sm, int64_t a_sk,
                         const float *B, int64_t b_sk, int64_t b_sn,
                         int64_t npts, const int64_t *pm, const int64_t *pn,
                         double *out, double *sabs, int threads)
{
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < npts; ++i) {
        int64_t m = pm[i], n = pn[i];
        double acc = 0.0, sab = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double p = (double)A[m * a_sm + k * a_sk] * (double)B[k * b_sk + n * b_sn];
            acc += p;
            sab += fabs(p);
        }
        out[i] = acc;
        if (sabs) sabs[i] = sab;
    }
    return 0;
}

/* O[n,w,f] (+)= sum_{kw,c} I[n, w*sw + kw*dw, c] * K[kw,c,f] */
int sg_ref_conv1d_nwc_wcf(int64_t N, int64_t Wo, int64_t F, int64_t KW, int64_t C,
                          int64_t W_in, int64_t sw, int64_t dw,
                          const float *I, const int64_t *is /* n,w,c */,
                          const float *Kf, const int64_t *ks /* kw,c,f */,
                          double *O, const int64_t *os /* n,w,f */,
                          double *S, int mode, int threads)
{
    if (N < 0 || Wo < 0 || F < 0 || KW < 0 || C < 0 || sw < 1 || dw < 1) return 1;
    if (Wo > 0 && KW > 0 && W_in < (Wo - 1) * sw + (KW - 1) * dw + 1) return 1;
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static) collapse(2)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t w = 0; w < Wo; ++w) {
            for (int64_t f = 0; f < F; ++f) {
                double acc = 0.0, sab = 0.0;
                for (int64_t kw = 0; kw < KW; ++kw) {
                    for (int64_t c = 0; c < C; ++c) {
                        double p = (double)I[n * is[0] + (w * sw + kw * dw) * is[1] + c * is[2]] *
                                   (double)Kf[kw * ks[0] + c * ks[1] + f * ks[2]];
                        acc += p;
                        sab += fabs(p);
                    }
                }
                double *o = &O[n * os[0] + w * os[1] + f * os[2]];
                *o = (mode ? *o : 0.0) + acc;
                if (S) S[(n * Wo + w) * F + f] = sab;
            }
        }
    }
    return 0;
}

/* O[n,h,w,f] (+)= sum_{kh,kw,c} I[n, h*sh+kh*dh, w*sw+kw*dw, c] * K[kh,kw,c,f] */
int sg_ref_conv2d_nhwc_hwcf(int64_t N, int64_t Ho, int64_t Wo, int64_t F,
                            int64_t KH, int64_t KW, int64_t C, int64_t H_in, int64_t W_in,
                            int64_t sh, int64_t sw, int64_t dh, int64_t dw,
                            const float *I, const int64_t *is /* n,h,w,c */,
                            const float *Kf, const int64_t *ks /* kh,kw,c,f */,
                            double *O, const int64_t *os /* n,h,w,f */,
                            double *S, int mode, int threads)
{
    if (N < 0 || Ho < 0 || Wo < 0 || F < 0 || KH < 0 || KW < 0 || C < 0) return 1;
    if (sh < 1 || sw < 1 || dh < 1 || dw < 1) return 1;
    if (Ho > 0 && KH > 0 && H_in < (Ho - 1) * sh + (KH - 1) * dh + 1) return 1;
    if (Wo > 0 && KW > 0 && W_in < (Wo - 1) * sw + (KW - 1) * dw + 1) return 1;
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static) collapse(2)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t h = 0; h < Ho; ++h) {
            for (int64_t w = 0; w < Wo; ++w) {
                for (int64_t f = 0; f < F; ++f) {
                    double acc = 0.0, sab = 0.0;
                    for (int64_t kh = 0; kh < KH; ++kh) {
                        for (int64_t kw = 0; kw < KW; ++kw) {
                            for (int64_t c = 0; c < C; ++c) {
                                double p =
                                    (double)I[n * is[0] + (h * sh + kh * dh) * is[1] +
                                              (w * sw + kw * dw) * is[2] + c * is[3]] *
                                    (double)Kf[kh * ks[0] + kw * ks[1] + c * ks[2] + f * ks[3]];
                                acc += p;
                                sab += fabs(p);
                            }
                        }
                    }
                    double *o = &O[n * os[0] + h * os[1] + w * os[2] + f * os[3]];
                    *o = (mode ? *o : 0.0) + acc;
                    if (S) S[((n * Ho + h) * Wo + w) * F + f] = sab;
                }
            }
        }
    }
    return 0;
}

/* Selected conv2d outputs: coordinates (pn,ph,pw,pf)[i] -> out[i], sabs[i]. */
int sg_ref_conv2d_points(int64_t KH, int64_t KW, int64_t C,
                         int64_t sh, int64_t sw, int64_t dh, int64_t dw,
                         const float *I, const int64_t *is, const float *Kf, const int64_t *ks,
                         int64_t npts, const int64_t *pn, const int64_t *ph, const int64_t *pw,
                         const int64_t *pf, double *out, double *sabs, int threads)
{
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < npts; ++i) {
        int64_t n = pn[i], h = ph[i], w = pw[i], f = pf[i];
        double acc = 0.0, sab = 0.0;
        for (int64_t kh = 0; kh < KH; ++kh)
            for (int64_t kw = 0; kw < KW; ++kw)
                for (int64_t c = 0; c < C; ++c) {
                    double p = (double)I[n * is[0] + (h * sh + kh * dh) * is[1] +
                                         (w * sw + kw * dw) * is[2] + c * is[3]] *
                               (double)Kf[kh * ks[0] + kw * ks[1] + c * ks[2] + f * ks[3]];
                    acc += p;
                    sab += fabs(p);
                }
        out[i] = acc;
        if (sabs) sabs[i] = sab;
    }
    return 0;
}

/*
 * Depthwise convolution, NHWC input, HWC filter (Section 4.6.3, "(2-D)"; the 1-D op is the
 * case H = KH = 1 with Sh = Dh = 1):
 *     O[n,h,w,c] = sum_{kh,kw} I[n, h*Sh + kh*Dh, w*Sw + kw*Dw, c] * K[kh,kw,c]
 * iterators (n,h,w,c,kh,kw) = (parallel x4, reduction x2): the channel iterator is parallel,
 * only the window is reduced.  No padding, filter not flipped, as for the dense convolutions.
 */
int sg_ref_depthwise_conv2d_nhwc_hwc(int64_t N, int64_t Ho, int64_t Wo, int64_t C,
                                     int64_t KH, int64_t KW, int64_t H_in, int64_t W_in,
                                     int64_t sh, int64_t sw, int64_t dh, int64_t dw,
                                     const float *I, const int64_t *is /* n,h,w,c */,
                                     const float *Kf, const int64_t *ks /* kh,kw,c */,
                                     double *O, const int64_t *os /* n,h,w,c */,
                                     double *S, int mode, int threads)
{
    if (N < 0 || Ho < 0 || Wo < 0 || C < 0 || KH < 0 || KW < 0) return 1;
    if (sh < 1 || sw < 1 || dh < 1 || dw < 1) return 1;
    if (Ho > 0 && KH > 0 && H_in < (Ho - 1) * sh + (KH - 1) * dh + 1) return 1;
    if (Wo > 0 && KW > 0 && W_in < (Wo - 1) * sw + (KW - 1) * dw + 1) return 1;
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static) collapse(2)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t h = 0; h < Ho; ++h) {
            for (int64_t w = 0; w < Wo; ++w) {
                for (int64_t c = 0; c < C; ++c) {
                    double acc = 0.0, sab = 0.0;
                    for (int64_t kh = 0; kh < KH; ++kh) {
                        for (int64_t kw = 0; kw < KW; ++kw) {
                            double p = (double)I[n * is[0] + (h * sh + kh * dh) * is[1] +
                                                 (w * sw + kw * dw) * is[2] + c * is[3]] *
                                       (double)Kf[kh * ks[0] + kw * ks[1] + c * ks[2]];
                            acc += p;
                            sab += fabs(p);
                        }
                    }
                    double *o = &O[n * os[0] + h * os[1] + w * os[2] + c * os[3]];
                    *o = (mode ? *o : 0.0) + acc;
                    if (S) S[((n * Ho + h) * Wo + w) * C + c] = sab;
                }
            }
        }
    }
    return 0;
}

/*
 * The memory-bound 2-D kernels (Section 4.4 "Benchmarks": Copy2D, Transpose2D, ColRed2D,
 * RowRed2D; Section 4.5).  A is an R x C tensor read through its element strides.
 *
 *   Copy2D       dst[i,j] = src[i,j]                      iterators (i,j) parallel
 *   Transpose2D  dst[j,i] = src[i,j]      (dst is C x R)  iterators (i,j) parallel
 *   ColRed2D     out[j]   = sum_i A[i,j]  (out has C elements)   i is the reduction
 *   RowRed2D     out[i]   = sum_j A[i,j]  (out has R elements)   j is the reduction
 *
 * Which reduction is which follows the caption of the L3 bandwidth figure: for a 250 x 960
 * tensor the row reduction writes 250 values and the column reduction 960.  The reductions
 * are sums (the paper ties them to matrix-vector products), accumulated in f64; `S` receives
 * sum |a| per output element, `mode` 1 adds to the output (destination-passing).
 * Copy and transpose move elements of `esize` bytes untouched, so they work on bit patterns.
 */
#include <string.h>

int sg_ref_copy2d(int64_t R, int64_t C, int64_t esize, const void *src, int64_t ss0, int64_t ss1,
                  void *dst, int64_t ds0, int64_t ds1)
{
    if (R < 0 || C < 0 || esize < 1) return 1;
    for (int64_t i = 0; i < R; ++i)
        for (int64_t j = 0; j < C; ++j)
            memcpy((char *)dst + (i * ds0 + j * ds1) * esize,
                   (const char *)src + (i * ss0 + j * ss1) * esize, (size_t)esize);
    return 0;
}

int sg_ref_transpose2d(int64_t R, int64_t C, int64_t esize, const void *src, int64_t ss0, int64_t ss1,
                       void *dst, int64_t ds0, int64_t ds1)
{
    if (R < 0 || C < 0 || esize < 1) return 1;
    for (int64_t i = 0; i < R; ++i)
        for (int64_t j = 0; j < C; ++j)
            memcpy((char *)dst + (j * ds0 + i * ds1) * esize,
                   (const char *)src + (i * ss0 + j * ss1) * esize, (size_t)esize);
    return 0;
}

int sg_ref_colred2d(int64_t R, int64_t C, const float *A, int64_t as0, int64_t as1,
                    double *out, double *S, int mode, int threads)
{
    if (R < 0 || C < 0) return 1;
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t j = 0; j < C; ++j) {
        double acc = 0.0, sab = 0.0;
        for (int64_t i = 0; i < R; ++i) {
            double v = (double)A[i * as0 + j * as1];
            acc += v;
            sab += fabs(v);
        }
        out[j] = (mode ? out[j] : 0.0) + acc;
        if (S) S[j] = sab;
    }
    return 0;
}

int sg_ref_rowred2d(int64_t R, int64_t C, const float *A, int64_t as0, int64_t as1,
                    double *out, double *S, int mode, int threads)
{
    if (R < 0 || C < 0) return 1;
    int nt = use_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < R; ++i) {
        double acc = 0.0, sab = 0.0;
        for (int64_t j = 0; j < C; ++j) {
            double v = (double)A[i * as0 + j * as1];
            acc += v;
            sab += fabs(v);
        }
        out[i] = (mode ? out[i] : 0.0) + acc;
        if (S) S[i] = sab;
    }
    return 0;
}
