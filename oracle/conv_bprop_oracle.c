/*
 * CPU oracle for the backward propagation (BPROP) of the direct 2-D convolution.
 *
 * TEST INFRASTRUCTURE ONLY.  Shares no code with the CUDA path; nothing in the
 * product may call it.
 *
 * The paper builds FPROP only and states (Abstract, Section 3.5 "Conclusion") that the same
 * techniques should carry over to BPROP without defining it.  BPROP is taken
 * here as what the word means for Section 2's operation
 *
 *   out[o,y,x,n] = alpha * sum_{c,kh,kw} filt[c,kh,kw,o]
 *                                        * in0[c, y*stride-pad+kh, x*stride-pad+kw, n]
 *
 * namely its two exact adjoints (the gradients of <dout, out> with respect to
 * the maps and to the filters), alpha included:
 *
 *   din  [c,h,w,n]   = alpha * sum_{o,y,x,kh,kw : y*stride-pad+kh = h, x*stride-pad+kw = w}
 *                                filt[c,kh,kw,o] * dout[o,y,x,n]
 *   dfilt[c,kh,kw,o] = alpha * sum_{y,x,n} in0[c, y*stride-pad+kh, x*stride-pad+kw, n]
 *                                          * dout[o,y,x,n]
 *
 * Terms whose input coordinate falls in the apron do not exist in din (the
 * apron is not a variable) and contribute zero to dfilt.
 *
 * Layouts are FPROP's: din like in ([c][h][w][n]), dfilt like filt
 * ([c][kh][kw][o]), dout like out ([o][y][x][n]).
 *
 * Arithmetic: products and running sums in fp64, alpha applied once to the
 * finished sum, one rounding to fp32 on store.  The sums are written as the
 * definitions above read: no blocking, no transformed filters, no reuse of the
 * FPROP routine.
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct oracle_conv_desc {
  int32_t Nb, Wi, Hi, Nc, No, Sk, stride, pad;
  float alpha;
} oracle_conv_desc;

int oracle_conv_out_dims(const oracle_conv_desc* d, int32_t* Ho, int32_t* Wo);

static void set_threads(int32_t nthreads) {
#ifdef _OPENMP
  if (nthreads > 0) omp_set_num_threads(nthreads);
#else
  (void)nthreads;
#endif
}

/*
 * Gradient with respect to the maps.  For every (c,h,w) the sum runs over the
 * filter taps (kh,kw) and keeps those for which an output pixel (y,x) exists
 * with y*stride - pad + kh = h and x*stride - pad + kw = w.
 * Returns 0, or 1 on a bad argument.
 */
int oracle_conv_bprop_data(const oracle_conv_desc* d, const float* dout, const float* filt,
                           float* din, int32_t nthreads) {
  int32_t Ho, Wo;
  if (!dout || !filt || !din || oracle_conv_out_dims(d, &Ho, &Wo)) return 1;
  const int Nb = d->Nb, Wi = d->Wi, Hi = d->Hi, Nc = d->Nc, No = d->No, Sk = d->Sk;
  const int stride = d->stride, pad = d->pad;
  const double alpha = (double)d->alpha;
  int bad_alloc = 0;
  set_threads(nthreads);
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)Nb);
    if (!s) {
#pragma omp atomic write
      bad_alloc = 1;
    }
#pragma omp for collapse(2) schedule(dynamic, 1)
    for (int c = 0; c < Nc; ++c) {
      for (int h = 0; h < Hi; ++h) {
        if (!s) continue;
        for (int w = 0; w < Wi; ++w) {
          for (int n = 0; n < Nb; ++n) s[n] = 0.0;
          for (int kh = 0; kh < Sk; ++kh) {
            const int ys = h + pad - kh; /* = y * stride */
            if (ys < 0 || ys % stride != 0) continue;
            const int y = ys / stride;
            if (y >= Ho) continue;
            for (int kw = 0; kw < Sk; ++kw) {
              const int xs = w + pad - kw;
              if (xs < 0 || xs % stride != 0) continue;
              const int x = xs / stride;
              if (x >= Wo) continue;
              const float* frow = filt + (((size_t)c * Sk + kh) * Sk + kw) * (size_t)No;
              for (int o = 0; o < No; ++o) {
                const double f = (double)frow[o];
                const float* g = dout + (((size_t)o * Ho + y) * Wo + x) * (size_t)Nb;
                for (int n = 0; n < Nb; ++n) s[n] += f * (double)g[n];
              }
            }
          }
          float* dst = din + (((size_t)c * Hi + h) * Wi + w) * (size_t)Nb;
          for (int n = 0; n < Nb; ++n) dst[n] = (float)(alpha * s[n]);
        }
      }
    }
    free(s);
  }
  return bad_alloc;
}

/* One element of din in fp64 (not rounded) and, in *abs_sum, the sum of |terms|. */
double oracle_conv_bprop_data_point(const oracle_conv_desc* d, const float* dout,
                                    const float* filt, int32_t c, int32_t h, int32_t w,
                                    int32_t n, double* abs_sum) {
  int32_t Ho, Wo;
  if (oracle_conv_out_dims(d, &Ho, &Wo)) return 0.0;
  const int Nb = d->Nb, No = d->No, Sk = d->Sk, stride = d->stride, pad = d->pad;
  double s = 0.0, a = 0.0;
  for (int kh = 0; kh < Sk; ++kh) {
    const int ys = h + pad - kh;
    if (ys < 0 || ys % stride != 0 || ys / stride >= Ho) continue;
    for (int kw = 0; kw < Sk; ++kw) {
      const int xs = w + pad - kw;
      if (xs < 0 || xs % stride != 0 || xs / stride >= Wo) continue;
      for (int o = 0; o < No; ++o) {
        const double t =
            (double)filt[(((size_t)c * Sk + kh) * Sk + kw) * (size_t)No + o] *
            (double)dout[(((size_t)o * Ho + ys / stride) * Wo + xs / stride) * (size_t)Nb + n];
        s += t;
        a += t < 0 ? -t : t;
      }
    }
  }
  if (abs_sum) *abs_sum = a;
  return (double)d->alpha * s;
}

/*
 * Gradient with respect to the filters.  Threads over (c,kh,kw); for each tap
 * the sum over the output pixels and images is accumulated per filter o.
 */
int oracle_conv_bprop_filter(const oracle_conv_desc* d, const float* in, const float* dout,
                             float* dfilt, int32_t nthreads) {
  int32_t Ho, Wo;
  if (!in || !dout || !dfilt || oracle_conv_out_dims(d, &Ho, &Wo)) return 1;
  const int Nb = d->Nb, Wi = d->Wi, Hi = d->Hi, Nc = d->Nc, No = d->No, Sk = d->Sk;
  const int stride = d->stride, pad = d->pad;
  const double alpha = (double)d->alpha;
  set_threads(nthreads);
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
  for (int c = 0; c < Nc; ++c) {
    for (int kh = 0; kh < Sk; ++kh) {
      for (int kw = 0; kw < Sk; ++kw) {
        float* dst = dfilt + (((size_t)c * Sk + kh) * Sk + kw) * (size_t)No;
        for (int o = 0; o < No; ++o) {
          double s = 0.0;
          for (int y = 0; y < Ho; ++y) {
            const int h = y * stride - pad + kh;
            if (h < 0 || h >= Hi) continue; /* apron row */
            for (int x = 0; x < Wo; ++x) {
              const int w = x * stride - pad + kw;
              if (w < 0 || w >= Wi) continue; /* apron column */
              const float* px = in + (((size_t)c * Hi + h) * Wi + w) * (size_t)Nb;
              const float* g = dout + (((size_t)o * Ho + y) * Wo + x) * (size_t)Nb;
              for (int n = 0; n < Nb; ++n) s += (double)px[n] * (double)g[n];
            }
          }
          dst[o] = (float)(alpha * s);
        }
      }
    }
  }
  return 0;
}

/* One element of dfilt in fp64 (not rounded) and the sum of |terms|. */
double oracle_conv_bprop_filter_point(const oracle_conv_desc* d, const float* in,
                                      const float* dout, int32_t c, int32_t kh, int32_t kw,
                                      int32_t o, double* abs_sum) {
  int32_t Ho, Wo;
  if (oracle_conv_out_dims(d, &Ho, &Wo)) return 0.0;
  const int Nb = d->Nb, Wi = d->Wi, Hi = d->Hi, stride = d->stride, pad = d->pad;
  double s = 0.0, a = 0.0;
  for (int y = 0; y < Ho; ++y) {
    const int h = y * stride - pad + kh;
    if (h < 0 || h >= Hi) continue;
    for (int x = 0; x < Wo; ++x) {
      const int w = x * stride - pad + kw;
      if (w < 0 || w >= Wi) continue;
      const float* px = in + (((size_t)c * Hi + h) * Wi + w) * (size_t)Nb;
      const float* g = dout + (((size_t)o * Ho + y) * Wo + x) * (size_t)Nb;
      for (int n = 0; n < Nb; ++n) {
        const double t = (double)px[n] * (double)g[n];
        s += t;
        a += t < 0 ? -t : t;
      }
    }
  }
  if (abs_sum) *abs_sum = a;
  return (double)d->alpha * s;
}

/*
 * The same two adjoints for the operation with per-axis filter size, stride and padding
 * (the relaxed-boundary generalisation; filt and dfilt are [Nc][Skh][Skw][No]):
 *
 *   din  [c,h,w,n]   = alpha * sum over (o,y,x,kh,kw) with y*stride_h-pad_h+kh = h and
 *                      x*stride_w-pad_w+kw = w of filt[c,kh,kw,o] * dout[o,y,x,n]
 *   dfilt[c,kh,kw,o] = alpha * sum_{y,x,n} in0[c, y*stride_h-pad_h+kh, x*stride_w-pad_w+kw, n]
 *                                          * dout[o,y,x,n]
 */
typedef struct oracle_conv_desc2 {
  int32_t Nb, Wi, Hi, Nc, No, Skw, Skh, stride_w, stride_h, pad_w, pad_h;
  float alpha;
} oracle_conv_desc2;

int oracle_conv2_out_dims(const oracle_conv_desc2* d, int32_t* Ho, int32_t* Wo);

int oracle_conv2_bprop_data(const oracle_conv_desc2* d, const float* dout, const float* filt,
                            float* din, int32_t nthreads) {
  int32_t Ho, Wo;
  if (!dout || !filt || !din || oracle_conv2_out_dims(d, &Ho, &Wo)) return 1;
  const int Nb = d->Nb, Wi = d->Wi, Hi = d->Hi, Nc = d->Nc, No = d->No;
  const int Skw = d->Skw, Skh = d->Skh;
  const double alpha = (double)d->alpha;
  int bad_alloc = 0;
  set_threads(nthreads);
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)Nb);
    if (!s) {
#pragma omp atomic write
      bad_alloc = 1;
    }
#pragma omp for collapse(2) schedule(dynamic, 1)
    for (int c = 0; c < Nc; ++c) {
      for (int h = 0; h < Hi; ++h) {
        if (!s) continue;
        for (int w = 0; w < Wi; ++w) {
          for (int n = 0; n < Nb; ++n) s[n] = 0.0;
          for (int kh = 0; kh < Skh; ++kh) {
            const int ys = h + d->pad_h - kh; /* = y * stride_h */
            if (ys < 0 || ys % d->stride_h != 0) continue;
            const int y = ys / d->stride_h;
            if (y >= Ho) continue;
            for (int kw = 0; kw < Skw; ++kw) {
              const int xs = w + d->pad_w - kw;
              if (xs < 0 || xs % d->stride_w != 0) continue;
              const int x = xs / d->stride_w;
              if (x >= Wo) continue;
              const float* frow = filt + (((size_t)c * Skh + kh) * Skw + kw) * (size_t)No;
              for (int o = 0; o < No; ++o) {
                const double f = (double)frow[o];
                const float* g = dout + (((size_t)o * Ho + y) * Wo + x) * (size_t)Nb;
                for (int n = 0; n < Nb; ++n) s[n] += f * (double)g[n];
              }
            }
          }
          float* dst = din + (((size_t)c * Hi + h) * Wi + w) * (size_t)Nb;
          for (int n = 0; n < Nb; ++n) dst[n] = (float)(alpha * s[n]);
        }
      }
    }
    free(s);
  }
  return bad_alloc;
}

int oracle_conv2_bprop_filter(const oracle_conv_desc2* d, const float* in, const float* dout,
                              float* dfilt, int32_t nthreads) {
  int32_t Ho, Wo;
  if (!in || !dout || !dfilt || oracle_conv2_out_dims(d, &Ho, &Wo)) return 1;
  const int Nb = d->Nb, Wi = d->Wi, Hi = d->Hi, Nc = d->Nc, No = d->No;
  const int Skw = d->Skw, Skh = d->Skh;
  const double alpha = (double)d->alpha;
  set_threads(nthreads);
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
  for (int c = 0; c < Nc; ++c) {
    for (int kh = 0; kh < Skh; ++kh) {
      for (int kw = 0; kw < Skw; ++kw) {
        float* dst = dfilt + (((size_t)c * Skh + kh) * Skw + kw) * (size_t)No;
        for (int o = 0; o < No; ++o) {
          double s = 0.0;
          for (int y = 0; y < Ho; ++y) {
            const int h = y * d->stride_h - d->pad_h + kh;
            if (h < 0 || h >= Hi) continue;
            for (int x = 0; x < Wo; ++x) {
              const int w = x * d->stride_w - d->pad_w + kw;
              if (w < 0 || w >= Wi) continue;
              const float* px = in + (((size_t)c * Hi + h) * Wi + w) * (size_t)Nb;
              const float* g = dout + (((size_t)o * Ho + y) * Wo + x) * (size_t)Nb;
              for (int n = 0; n < Nb; ++n) s += (double)px[n] * (double)g[n];
            }
          }
          dst[o] = (float)(alpha * s);
        }
      }
    }
  }
  return 0;
}
