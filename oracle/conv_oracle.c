/*
 * CPU oracle for the forward-propagation (FPROP) direct 2-D convolution.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
 * paper's definition (Section 2, "Convolution") that the GPU kernels are
 * checked against.  It shares no code, header, table or helper with the CUDA
 * path and nothing in the product may call it.
 *
 * Definition (Section 2): Nb maps of Wi x Hi x Nc are convolved with No
 * filters of Sk x Sk x Nc, per channel, summed over channels, with a stride,
 * an optional padding offset of the origin, an apron of zeros around the map
 * and a final scale by alpha.  Written out:
 *
 *   out[o,y,x,n] = alpha * sum_{c,kh,kw} filt[c,kh,kw,o]
 *                                        * in0[c, y*stride-pad+kh, x*stride-pad+kw, n]
 *
 * with in0 = in inside [0,Hi) x [0,Wi) and 0 outside (the apron).  No filter
 * flip: Section 3 multiplies the unrolled patch by the filter matrix as is.
 *
 * Layout (Section 3, batch/filter innermost):
 *   in   [c][h][w][n]     ((c*Hi + h)*Wi + w)*Nb + n
 *   filt [c][kh][kw][o]   ((c*Sk + kh)*Sk + kw)*No + o
 *   out  [o][y][x][n]     ((o*Ho + y)*Wo + x)*Nb + n
 *
 * Output size: Ho = floor((Hi + 2*pad - Sk)/stride) + 1, same for Wo (the
 * reading under which every row of Table 1 is consistent).
 *
 * Arithmetic: every product and the running sum are fp64; alpha is applied
 * once to the finished sum in fp64; one rounding to fp32 on store.  The loop
 * order (n innermost, threads over (o,y)) is the only concession to speed;
 * there is no blocking, no im2col and no reordering of the definition.
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Field order is the boundary's descriptor order: Section 2's symbols. */
typedef struct oracle_conv_desc {
  int32_t Nb, Wi, Hi, Nc, No, Sk, stride, pad;
  float alpha;
} oracle_conv_desc;

static int out_dim(int in, int pad, int Sk, int stride) {
  int span = in + 2 * pad - Sk;
  if (span < 0) return 0;
  return span / stride + 1;
}

/* 0 on success, 1 on an invalid descriptor. */
int oracle_conv_out_dims(const oracle_conv_desc* d, int32_t* Ho, int32_t* Wo) {
  if (!d || d->Nb <= 0 || d->Wi <= 0 || d->Hi <= 0 || d->Nc <= 0 || d->No <= 0 ||
      d->Sk <= 0 || d->stride <= 0 || d->pad < 0)
    return 1;
  int ho = out_dim(d->Hi, d->pad, d->Sk, d->stride);
  int wo = out_dim(d->Wi, d->pad, d->Sk, d->stride);
  if (ho <= 0 || wo <= 0) return 1;
  if (Ho) *Ho = ho;
  if (Wo) *Wo = wo;
  return 0;
}

/* Section 2, complexity formula: C = 2 Nb Wo Ho (Nc Sk^2 + 1) No. */
uint64_t oracle_conv_flops(const oracle_conv_desc* d) {
  int32_t Ho, Wo;
  if (oracle_conv_out_dims(d, &Ho, &Wo)) return 0;
  return 2ull * (uint64_t)d->Nb * (uint64_t)Wo * (uint64_t)Ho *
         ((uint64_t)d->Nc * (uint64_t)d->Sk * (uint64_t)d->Sk + 1ull) * (uint64_t)d->No;
}

/*
 * Computes output rows y in [y_begin, y_end) of every filter (the full result
 * when y_begin = 0, y_end = Ho); rows outside the range are not written.
 * nthreads <= 0 means "all cores".  Returns 0, or 1 on a bad argument.
 */
int oracle_conv_fprop_rows(const oracle_conv_desc* d, const float* in, const float* filt,
                           float* out, int32_t y_begin, int32_t y_end, int32_t nthreads) {
  int32_t Ho, Wo;
  if (!in || !filt || !out || oracle_conv_out_dims(d, &Ho, &Wo)) return 1;
  if (y_begin < 0 || y_end > Ho || y_begin > y_end) return 1;
  const int Nb = d->Nb, Wi = d->Wi, Hi = d->Hi, Nc = d->Nc, No = d->No, Sk = d->Sk;
  const int stride = d->stride, pad = d->pad;
  const double alpha = (double)d->alpha;
  const int rows = y_end - y_begin;
  int bad_alloc = 0;
#ifdef _OPENMP
  if (nthreads > 0) omp_set_num_threads(nthreads);
#else
  (void)nthreads;
#endif
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)Nb);
    if (!s) {
#pragma omp atomic write
      bad_alloc = 1;
    }
#pragma omp for collapse(2) schedule(dynamic, 1)
    for (int o = 0; o < No; ++o) {
      for (int yr = 0; yr < rows; ++yr) {
        if (!s) continue;
        const int y = y_begin + yr;
        for (int x = 0; x < Wo; ++x) {
          for (int n = 0; n < Nb; ++n) s[n] = 0.0;
          for (int c = 0; c < Nc; ++c) {
            for (int kh = 0; kh < Sk; ++kh) {
              const int h = y * stride - pad + kh;
              if (h < 0 || h >= Hi) continue; /* apron row: contributes zeros */
              for (int kw = 0; kw < Sk; ++kw) {
                const int w = x * stride - pad + kw;
                if (w < 0 || w >= Wi) continue; /* apron column */
                const double f =
                    (double)filt[(((size_t)c * Sk + kh) * Sk + kw) * (size_t)No + o];
                const float* px = in + (((size_t)c * Hi + h) * Wi + w) * (size_t)Nb;
                for (int n = 0; n < Nb; ++n) s[n] += f * (double)px[n];
              }
            }
          }
          float* dst = out + (((size_t)o * Ho + y) * Wo + x) * (size_t)Nb;
          for (int n = 0; n < Nb; ++n) dst[n] = (float)(alpha * s[n]);
        }
      }
    }
    free(s);
  }
  return bad_alloc;
}

int oracle_conv_fprop(const oracle_conv_desc* d, const float* in, const float* filt,
                      float* out, int32_t nthreads) {
  int32_t Ho, Wo;
  if (oracle_conv_out_dims(d, &Ho, &Wo)) return 1;
  return oracle_conv_fprop_rows(d, in, filt, out, 0, Ho, nthreads);
}

/*
 * One output element, for spot checks at sizes where the full oracle would
 * take too long.  Returns the fp64 value alpha * sum (not yet rounded) and, in
 * *abs_sum, sum |filt * in| over the same terms (the scale of the a-priori
 * rounding bound of an fp32 dot product).
 */
double oracle_conv_fprop_point(const oracle_conv_desc* d, const float* in, const float* filt,
                               int32_t o, int32_t y, int32_t x, int32_t n, double* abs_sum) {
  const int Nb = d->Nb, Wi = d->Wi, Hi = d->Hi, Nc = d->Nc, No = d->No, Sk = d->Sk;
  double s = 0.0, a = 0.0;
  for (int c = 0; c < Nc; ++c)
    for (int kh = 0; kh < Sk; ++kh) {
      const int h = y * d->stride - d->pad + kh;
      if (h < 0 || h >= Hi) continue;
      for (int kw = 0; kw < Sk; ++kw) {
        const int w = x * d->stride - d->pad + kw;
        if (w < 0 || w >= Wi) continue;
        const double t = (double)filt[(((size_t)c * Sk + kh) * Sk + kw) * (size_t)No + o] *
                         (double)in[(((size_t)c * Hi + h) * Wi + w) * (size_t)Nb + n];
        s += t;
        a += t < 0 ? -t : t;
      }
    }
  if (abs_sum) *abs_sum = a;
  return (double)d->alpha * s;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * The same operation with per-axis filter size, stride and padding (Section 2 states one
 * square size, one stride and one padding; this is the plain generalisation of its sum,
 * used to check the library's relaxed-boundary entry point):
 *
 *   out[o,y,x,n] = alpha * sum_{c,kh,kw} filt[c,kh,kw,o]
 *                    * in0[c, y*stride_h - pad_h + kh, x*stride_w - pad_w + kw, n]
 *
 * kh < Skh, kw < Skw; filt is [Nc][Skh][Skw][No]; Ho = floor((Hi + 2 pad_h - Skh)/stride_h) + 1,
 * Wo likewise with the w quantities.  Same arithmetic as above.
 */
typedef struct oracle_conv_desc2 {
  int32_t Nb, Wi, Hi, Nc, No, Skw, Skh, stride_w, stride_h, pad_w, pad_h;
  float alpha;
} oracle_conv_desc2;

int oracle_conv2_out_dims(const oracle_conv_desc2* d, int32_t* Ho, int32_t* Wo) {
  if (!d || d->Nb <= 0 || d->Wi <= 0 || d->Hi <= 0 || d->Nc <= 0 || d->No <= 0 || d->Skw <= 0 ||
      d->Skh <= 0 || d->stride_w <= 0 || d->stride_h <= 0 || d->pad_w < 0 || d->pad_h < 0)
    return 1;
  int ho = out_dim(d->Hi, d->pad_h, d->Skh, d->stride_h);
  int wo = out_dim(d->Wi, d->pad_w, d->Skw, d->stride_w);
  if (ho <= 0 || wo <= 0) return 1;
  if (Ho) *Ho = ho;
  if (Wo) *Wo = wo;
  return 0;
}

int oracle_conv2_fprop(const oracle_conv_desc2* d, const float* in, const float* filt, float* out,
                       int32_t nthreads) {
  int32_t Ho, Wo;
  if (!in || !filt || !out || oracle_conv2_out_dims(d, &Ho, &Wo)) return 1;
  const int Nb = d->Nb, Wi = d->Wi, Hi = d->Hi, Nc = d->Nc, No = d->No;
  const int Skw = d->Skw, Skh = d->Skh;
  const double alpha = (double)d->alpha;
  int bad_alloc = 0;
#ifdef _OPENMP
  if (nthreads > 0) omp_set_num_threads(nthreads);
#else
  (void)nthreads;
#endif
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)Nb);
    if (!s) {
#pragma omp atomic write
      bad_alloc = 1;
    }
#pragma omp for collapse(2) schedule(dynamic, 1)
    for (int o = 0; o < No; ++o) {
      for (int y = 0; y < Ho; ++y) {
        if (!s) continue;
        for (int x = 0; x < Wo; ++x) {
          for (int n = 0; n < Nb; ++n) s[n] = 0.0;
          for (int c = 0; c < Nc; ++c) {
            for (int kh = 0; kh < Skh; ++kh) {
              const int h = y * d->stride_h - d->pad_h + kh;
              if (h < 0 || h >= Hi) continue;
              for (int kw = 0; kw < Skw; ++kw) {
                const int w = x * d->stride_w - d->pad_w + kw;
                if (w < 0 || w >= Wi) continue;
                const double f =
                    (double)filt[(((size_t)c * Skh + kh) * Skw + kw) * (size_t)No + o];
                const float* px = in + (((size_t)c * Hi + h) * Wi + w) * (size_t)Nb;
                for (int n = 0; n < Nb; ++n) s[n] += f * (double)px[n];
              }
            }
          }
          float* dst = out + (((size_t)o * Ho + y) * Wo + x) * (size_t)Nb;
          for (int n = 0; n < Nb; ++n) dst[n] = (float)(alpha * s[n]);
        }
      }
    }
    free(s);
  }
  return bad_alloc;
}
