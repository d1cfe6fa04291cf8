/*
 * The boundary is a C ABI: this program uses nothing but include/maxdnn.h, the CUDA runtime's
 * C API for memory, and libc.  It runs one small FPROP and both gradients, checks them against
 * sums written out below (the definition of the operation, Section 2, in double precision),
 * and prints "C ABI OK".  Built and run by tests/test_c_abi_gpu.py.
 */
#include <cuda_runtime_api.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>

#include "maxdnn.h"

static float frand(unsigned* s) {
  *s = *s * 1664525u + 1013904223u;
  return (float)((*s >> 8) & 0xFFFF) / 32768.0f - 1.0f;
}

#define CK(x)                                                        \
  do {                                                               \
    if ((x) != 0) {                                                  \
      fprintf(stderr, "failed at line %d: %s\n", __LINE__, #x);      \
      return 1;                                                      \
    }                                                                \
  } while (0)

int main(void) {
  maxdnn_conv_desc d = {32, 10, 8, 8, 32, 3, 1, 1, 0.5f};   /* Nb Wi Hi Nc No Sk stride pad alpha */
  int32_t Ho, Wo;
  CK(maxdnn_conv_out_dims(&d, &Ho, &Wo));
  const size_t n_in = maxdnn_conv_in_elems(&d), n_f = maxdnn_conv_filt_elems(&d),
               n_out = maxdnn_conv_out_elems(&d);
  float *h_in = malloc(n_in * 4), *h_f = malloc(n_f * 4), *h_g = malloc(n_out * 4);
  float *h_out = malloc(n_out * 4), *h_din = malloc(n_in * 4), *h_df = malloc(n_f * 4);
  unsigned seed = 12345u;
  for (size_t i = 0; i < n_in; ++i) h_in[i] = frand(&seed);
  for (size_t i = 0; i < n_f; ++i) h_f[i] = frand(&seed);
  for (size_t i = 0; i < n_out; ++i) h_g[i] = frand(&seed);

  float *d_in, *d_f, *d_g, *d_out, *d_din, *d_df;
  void *ws1 = NULL, *ws2 = NULL;
  size_t b1 = 0, b2 = 0;
  CK(maxdnn_conv_bprop_data_workspace(&d, MAXDNN_KERNEL_FP32, &b1));
  CK(maxdnn_conv_bprop_filter_workspace(&d, MAXDNN_KERNEL_FP32, &b2));
  CK(cudaMalloc((void**)&d_in, n_in * 4)); CK(cudaMalloc((void**)&d_f, n_f * 4));
  CK(cudaMalloc((void**)&d_g, n_out * 4)); CK(cudaMalloc((void**)&d_out, n_out * 4));
  CK(cudaMalloc((void**)&d_din, n_in * 4)); CK(cudaMalloc((void**)&d_df, n_f * 4));
  CK(cudaMalloc(&ws1, b1 ? b1 : 16)); CK(cudaMalloc(&ws2, b2 ? b2 : 16));
  CK(cudaMemcpy(d_in, h_in, n_in * 4, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_f, h_f, n_f * 4, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_g, h_g, n_out * 4, cudaMemcpyHostToDevice));

  CK(maxdnn_conv_fprop(&d, d_in, d_f, d_out, NULL));
  CK(maxdnn_conv_bprop_data(&d, MAXDNN_KERNEL_FP32, d_g, d_f, d_din, ws1, b1, NULL));
  CK(maxdnn_conv_bprop_filter(&d, MAXDNN_KERNEL_FP32, d_in, d_g, d_df, ws2, b2, NULL));
  CK(maxdnn_last_device_status(NULL));
  CK(cudaMemcpy(h_out, d_out, n_out * 4, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(h_din, d_din, n_in * 4, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(h_df, d_df, n_f * 4, cudaMemcpyDeviceToHost));

  /* the three sums, term by term */
  double* r_out = calloc(n_out, 8);
  double* r_din = calloc(n_in, 8);
  double* r_df = calloc(n_f, 8);
  for (int o = 0; o < d.No; ++o)
    for (int y = 0; y < Ho; ++y)
      for (int x = 0; x < Wo; ++x)
        for (int n = 0; n < d.Nb; ++n) {
          const size_t io = (((size_t)o * Ho + y) * Wo + x) * d.Nb + n;
          for (int c = 0; c < d.Nc; ++c)
            for (int kh = 0; kh < d.Sk; ++kh)
              for (int kw = 0; kw < d.Sk; ++kw) {
                const int h = y * d.stride - d.pad + kh, w = x * d.stride - d.pad + kw;
                if (h < 0 || h >= d.Hi || w < 0 || w >= d.Wi) continue;
                const size_t ii = (((size_t)c * d.Hi + h) * d.Wi + w) * d.Nb + n;
                const size_t jf = (((size_t)c * d.Sk + kh) * d.Sk + kw) * d.No + o;
                r_out[io] += (double)d.alpha * h_f[jf] * h_in[ii];
                r_din[ii] += (double)d.alpha * h_f[jf] * h_g[io];
                r_df[jf] += (double)d.alpha * h_in[ii] * h_g[io];
              }
        }
  double e[3] = {0, 0, 0}, m[3] = {0, 0, 0};
  for (size_t i = 0; i < n_out; ++i) { e[0] = fmax(e[0], fabs(h_out[i] - r_out[i])); m[0] = fmax(m[0], fabs(r_out[i])); }
  for (size_t i = 0; i < n_in; ++i) { e[1] = fmax(e[1], fabs(h_din[i] - r_din[i])); m[1] = fmax(m[1], fabs(r_din[i])); }
  for (size_t i = 0; i < n_f; ++i) { e[2] = fmax(e[2], fabs(h_df[i] - r_df[i])); m[2] = fmax(m[2], fabs(r_df[i])); }
  printf("fprop %.2e  bprop_data %.2e  bprop_filter %.2e  (launches %llu)\n", e[0] / m[0], e[1] / m[1],
         e[2] / m[2], (unsigned long long)maxdnn_launch_count());
  if (!(e[0] / m[0] <= 1e-5 && e[1] / m[1] <= 1e-5 && e[2] / m[2] <= 1e-5)) return 2;
  puts("C ABI OK");
  return 0;
}
