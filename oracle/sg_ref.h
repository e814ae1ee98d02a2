/*
 * sg_ref.h: C interface of the CPU oracle (sg_ref.c -> libsgref.so).
 *
 * TEST INFRASTRUCTURE, NOT THE PRODUCT.  These are the reference counterparts of the GPU
 * library's entry points: the same argument order (extents, then each operand with its element
 * strides), HOST pointers, no CUDA.  Only the tests, the smoke check and the benchmark's CPU
 * baseline call them; the GPU library neither includes this header nor links this code.
 *
 * Inputs are f32 (bf16 problems pass bf16-representable values widened to f32), results are
 * f64.  `S`, when non-NULL, receives sum |a*b| per output element (dense row-major in the
 * output's dimension order): the scale of the comparison bound |err| <= 1e-4 * S.
 * `mode` 0 overwrites the output, 1 adds to the value already there.  `threads` <= 0 uses
 * every OpenMP thread; the outermost parallel iterator is split across them.
 * Return value: SG_REF_OK, or SG_REF_INVALID_ARG (negative extent, stride or dilation < 1,
 * input smaller than the window needs); nothing is written in that case.
 */
#ifndef SG_REF_H_
#define SG_REF_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { SG_REF_OK = 0, SG_REF_INVALID_ARG = 1 };

int sg_ref_max_threads(void);

/* matmul (Section 4.6.1, "AB"): C[m,n] (+)= sum_k A[m,k]*B[k,n] */
int sg_ref_matmul(int64_t M, int64_t N, int64_t K,
                  const float *A, int64_t a_sm, int64_t a_sk,
                  const float *B, int64_t b_sk, int64_t b_sn,
                  double *C, int64_t c_sm, int64_t c_sn,
                  double *S, int mode, int threads);
/* matmul with a fused pointwise consumer (Sections 2.1, 3.3): C[m,n] = act(sum_k A[m,k]*B[k,n] + bias[n]); act 0 identity,
 * 1 max(., 0); bias may be NULL; overwrite only; S = sum |a*b| + |bias| */
int sg_ref_matmul_bias_act(int64_t M, int64_t N, int64_t K,
                           const float *A, int64_t a_sm, int64_t a_sk,
                           const float *B, int64_t b_sk, int64_t b_sn,
                           const float *bias, int64_t bias_sn, int act,
                           double *C, int64_t c_sm, int64_t c_sn,
                           double *S, int threads);
/* listed elements (pm[i], pn[i]) of the same product -> out[i], sabs[i]; overwrite only */
int sg_ref_matmul_points(int64_t K,
                         const float *A, int64_t a_sm, int64_t a_sk,
                         const float *B, int64_t b_sk, int64_t b_sn,
                         int64_t npts, const int64_t *pm, const int64_t *pn,
                         double *out, double *sabs, int threads);

/* conv_1d_nwc_wcf (Section 3; Section 4.6.2 "(1-D)"): O[n,w,f] (+)= sum_{kw,c} I[n, w*sw+kw*dw, c]*K[kw,c,f] */
int sg_ref_conv1d_nwc_wcf(int64_t N, int64_t Wo, int64_t F, int64_t KW, int64_t C,
                          int64_t W_in, int64_t sw, int64_t dw,
                          const float *I, const int64_t *is /* n,w,c */,
                          const float *Kf, const int64_t *ks /* kw,c,f */,
                          double *O, const int64_t *os /* n,w,f */,
                          double *S, int mode, int threads);

/* conv_2d_nhwc_hwcf (Section 4.6.2 "(2-D)") */
int sg_ref_conv2d_nhwc_hwcf(int64_t N, int64_t Ho, int64_t Wo, int64_t F,
                            int64_t KH, int64_t KW, int64_t C, int64_t H_in, int64_t W_in,
                            int64_t sh, int64_t sw, int64_t dh, int64_t dw,
                            const float *I, const int64_t *is /* n,h,w,c */,
                            const float *Kf, const int64_t *ks /* kh,kw,c,f */,
                            double *O, const int64_t *os /* n,h,w,f */,
                            double *S, int mode, int threads);
/* listed outputs (pn,ph,pw,pf)[i] of the 2-D convolution -> out[i], sabs[i]; overwrite only */
int sg_ref_conv2d_points(int64_t KH, int64_t KW, int64_t C,
                         int64_t sh, int64_t sw, int64_t dh, int64_t dw,
                         const float *I, const int64_t *is, const float *Kf, const int64_t *ks,
                         int64_t npts, const int64_t *pn, const int64_t *ph, const int64_t *pw,
                         const int64_t *pf, double *out, double *sabs, int threads);

/* depthwise conv 2-D (Section 4.6.3): O[n,h,w,c] (+)= sum_{kh,kw} I[n,h*sh+kh*dh,w*sw+kw*dw,c]*K[kh,kw,c] */
int sg_ref_depthwise_conv2d_nhwc_hwc(int64_t N, int64_t Ho, int64_t Wo, int64_t C,
                                     int64_t KH, int64_t KW, int64_t H_in, int64_t W_in,
                                     int64_t sh, int64_t sw, int64_t dh, int64_t dw,
                                     const float *I, const int64_t *is /* n,h,w,c */,
                                     const float *Kf, const int64_t *ks /* kh,kw,c */,
                                     double *O, const int64_t *os /* n,h,w,c */,
                                     double *S, int mode, int threads);

/* memory-bound 2-D kernels (Section 4.4): element moves of `esize` bytes; sums in f64 */
int sg_ref_copy2d(int64_t R, int64_t C, int64_t esize, const void *src, int64_t ss0, int64_t ss1,
                  void *dst, int64_t ds0, int64_t ds1);
int sg_ref_transpose2d(int64_t R, int64_t C, int64_t esize, const void *src, int64_t ss0, int64_t ss1,
                       void *dst, int64_t ds0, int64_t ds1);
int sg_ref_colred2d(int64_t R, int64_t C, const float *A, int64_t as0, int64_t as1,
                    double *out, double *S, int mode, int threads);
int sg_ref_rowred2d(int64_t R, int64_t C, const float *A, int64_t as0, int64_t as1,
                    double *out, double *S, int mode, int threads);

#ifdef __cplusplus
}
#endif
#endif /* SG_REF_H_ */
