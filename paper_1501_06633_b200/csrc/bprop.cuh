// Backward-propagation kernels (the adjoints of the operation of Section 2; the paper
// names BPROP in its Abstract and Section 3.5 ("Conclusion") as where its techniques should carry over).
//
//  - flip_transpose_kernel: filt[c][kh][kw][o] -> ft[o][Skh-1-kh][Skw-1-kw][c], the filter
//    bank with which the gradient with respect to the maps is an FPROP of the output
//    gradient (stride 1).
//  - wgrad_kernel: gradient with respect to the filters in exact fp32.  The same
//    technique as the forward kernel — bulk tensor copies into a ring of shared-memory
//    stages, a register-blocked multiply-accumulate inner loop of packed FFMA2 — with
//    the reduction running over output pixels and images:
//        dfilt[k][o] = alpha * sum_r patch[k][r] * dout[o][r],  r = (y, x, n).
//    Both operands arrive with r contiguous (32 images = one 128-byte row per gradient
//    row / filter), so a thread reads 16 bytes = 4 values of r from each of its 8 + 8
//    rows and the two halves of a packed multiply-add accumulate even and odd r, added
//    at the end.
//  - wgrad_reduce_kernel: adds the partial sums of the reduction splits in a fixed order.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "plan.h"
#include "ptx_util.cuh"

namespace maxdnn {

template <typename T>
__global__ void __launch_bounds__(256)
flip_transpose_kernel(const T* __restrict__ filt, T* __restrict__ ft, int Nc, int taps, int No) {
  __shared__ T tile[32][33];
  const int tap = blockIdx.z;              // kh * Sk + kw
  const int tap_t = taps - 1 - tap;        // (Sk-1-kh) * Sk + (Sk-1-kw)
  const int o0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int c = c0 + i, o = o0 + threadIdx.x;
    if (c < Nc && o < No) tile[i][threadIdx.x] = filt[((size_t)c * taps + tap) * No + o];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int o = o0 + i, c = c0 + threadIdx.x;
    if (c < Nc && o < No) ft[((size_t)o * taps + tap_t) * Nc + c] = tile[threadIdx.x][i];
  }
}

// Strided map gradient: the sub-filter of one class, flipped and transposed:
//   ft[o][j'][i'][c] = filt[c][rho_h + s_h (Jh-1-j')][rho_w + s_w (Jw-1-i')][o]
template <typename T>
__global__ void __launch_bounds__(256)
subfilter_flip_transpose_kernel(const T* __restrict__ filt, T* __restrict__ ft, int Nc, int Skh,
                                int Skw, int No, int s_h, int s_w, int rho_h, int rho_w, int Jh,
                                int Jw) {
  __shared__ T tile[32][33];
  const int jp = blockIdx.z / Jw, ip = blockIdx.z % Jw;     // position in the transformed bank
  const int kh = rho_h + s_h * (Jh - 1 - jp), kw = rho_w + s_w * (Jw - 1 - ip);
  const int o0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int c = c0 + i, o = o0 + threadIdx.x;
    if (c < Nc && o < No) tile[i][threadIdx.x] = filt[(((size_t)c * Skh + kh) * Skw + kw) * No + o];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int o = o0 + i, c = c0 + threadIdx.x;
    if (c < Nc && o < No) ft[(((size_t)o * Jh + jp) * Jw + ip) * Nc + c] = tile[threadIdx.x][i];
  }
}

// din[c][h_first + s_h a][w_first + s_w b][n] = sub[c][a][b][n]: the class's gradient onto its grid.
__global__ void __launch_bounds__(256)
dgrad_scatter_kernel(const float4* __restrict__ sub, float4* __restrict__ din, int Nc, int n_h,
                     int n_w, int nb4, int Hi, int Wi, int s_h, int s_w, int h_first,
                     int w_first) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t total = (size_t)Nc * n_h * n_w * nb4;
  if (i >= total) return;
  size_t r = i;
  const int n = (int)(r % nb4); r /= nb4;
  const int b = (int)(r % n_w); r /= n_w;
  const int a = (int)(r % n_h);
  const int c = (int)(r / n_h);
  din[(((size_t)c * Hi + h_first + s_h * a) * Wi + w_first + s_w * b) * nb4 + n] = sub[i];
}

// Split of fp32 values for the three-product TF32 scheme: hi = the value rounded to the
// nearest TF32 number (10 mantissa bits; a TF32 tensor core reads an fp32 word and ignores
// the low 13 bits, so hi passes through it unchanged), lo = value - hi (exact in fp32),
// itself rounded to TF32.  Rounding to nearest instead of clearing the low bits makes lo,
// the dropped lo x lo product and the rounding of lo zero-mean, so their sums over K terms
// grow like sqrt(K); with cleared bits they all carry the operand's sign and, on
// same-signed inputs, add up linearly (measured: 9e-5 of the largest output at K = 9216).
// dst holds three copies of the tensor back to back along its outermost (channel) axis:
// part p is hi where bit p of `lo_mask` is clear, lo where it is set.
__device__ __forceinline__ float round_to_tf32(float v) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
  return __uint_as_float(r);
}

__global__ void __launch_bounds__(256)
tf32_split3_kernel(const float4* __restrict__ src, float4* __restrict__ dst, size_t n4,
                   uint32_t lo_mask) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const float4 a = src[i];
  float4 hi, lo;
  hi.x = round_to_tf32(a.x); hi.y = round_to_tf32(a.y);
  hi.z = round_to_tf32(a.z); hi.w = round_to_tf32(a.w);
  lo.x = round_to_tf32(a.x - hi.x); lo.y = round_to_tf32(a.y - hi.y);
  lo.z = round_to_tf32(a.z - hi.z); lo.w = round_to_tf32(a.w - hi.w);
#pragma unroll
  for (int p = 0; p < 3; ++p) dst[(size_t)p * n4 + i] = ((lo_mask >> p) & 1u) ? lo : hi;
}

// The split for the filter gradient, whose reduction runs over images: row r of dst is
// [hi | lo] of row r of src, each part n4 float4 long (the kernel reads the parts it needs
// for each of the three products: hi x hi, lo x hi, hi x lo).
__global__ void __launch_bounds__(256)
tf32_split2_rows_kernel(const float4* __restrict__ src, float4* __restrict__ dst, size_t rows,
                        int n4) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * (size_t)n4) return;
  const size_t row = i / (size_t)n4;
  const int j = (int)(i - row * (size_t)n4);
  const float4 a = src[i];
  float4 hi, lo;
  hi.x = round_to_tf32(a.x); hi.y = round_to_tf32(a.y);
  hi.z = round_to_tf32(a.z); hi.w = round_to_tf32(a.w);
  lo.x = round_to_tf32(a.x - hi.x); lo.y = round_to_tf32(a.y - hi.y);
  lo.z = round_to_tf32(a.z - hi.z); lo.w = round_to_tf32(a.w - hi.w);
  dst[(row * 2) * (size_t)n4 + j] = hi;
  dst[(row * 2 + 1) * (size_t)n4 + j] = lo;
}

// Staging copies for shapes the bulk tensor copies cannot address (row pitches that are
// not multiples of 16 bytes): dst[row][j] = src[row][j] for j < n, 0 for n <= j < n_pad
// (pad_inner), and the reverse for results (unpad_inner drops the padding columns).
template <typename T>
__global__ void __launch_bounds__(256)
pad_inner_kernel(const T* __restrict__ src, T* __restrict__ dst, size_t rows, int n, int n_pad) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * (size_t)n_pad) return;
  const size_t row = i / (size_t)n_pad;
  const int j = (int)(i - row * (size_t)n_pad);
  dst[i] = j < n ? src[row * (size_t)n + j] : T(0);
}

__global__ void __launch_bounds__(256)
unpad_inner_kernel(const float* __restrict__ src, float* __restrict__ dst, size_t rows, int n,
                   int n_pad) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * (size_t)n) return;
  const size_t row = i / (size_t)n;
  const int j = (int)(i - row * (size_t)n);
  dst[i] = src[row * (size_t)n_pad + j];
}

constexpr int kWgThreads = 256;               // 8 warps: 16 x 16 threads, 8 x 8 results each (stride 16)
constexpr uint32_t kWgOperandBytes = 128 * 128;   // 128 rows x 32 floats
constexpr int kWgSub = 2;                         // reduction steps per ring stage

struct WgradArgs {
  WgradGeom g;
  float* dfilt;        // result when g.splits == 1
  float* partial;      // [splits][Nc Sk^2][No] otherwise
  WaitCtx wc;          // status block and this launch's epoch (see ptx_util.cuh)
};

// Which (tile, split, reduction step) comes next; the copy-issuing lane and the
// arithmetic warps walk the same sequence.
struct WgradCursor {
  int item;            // index over (tile, split); >= n_items: done
  int r, r_end;        // reduction steps of this item: [r, r_end)
  int y, x, nc;        // r = (y * Wo + x) * n_chunks + nc
  int ob, cb, khb, split;

  __device__ __forceinline__ void start(const WgradGeom& g, int it) {
    item = it;
    if (it >= g.n_items) return;
    // Items are ordered split-major: the CTAs that run at the same time work on the same
    // range of output pixels for different tiles, so each slice of the two operands is
    // fetched from HBM once and served to the other tiles' CTAs by L2.
    const int tiles = g.n_items / g.splits;
    split = it / tiles;
    int t = it - split * tiles;
    ob = t % g.o_blocks; t /= g.o_blocks;
    cb = t % g.c_blocks;
    khb = t / g.c_blocks;
    r = split * g.steps_per_split;
    r_end = r + g.steps_per_split < g.r_steps ? r + g.steps_per_split : g.r_steps;
    nc = r % g.n_chunks;
    const int px = r / g.n_chunks;
    x = px % g.Wo;
    y = px / g.Wo;
  }
  __device__ __forceinline__ bool done(const WgradGeom& g) const { return item >= g.n_items; }
  // Next reduction step; moves to this CTA's (or CTA pair's) next item, `item_stride`
  // further, when the current one is exhausted.
  __device__ __forceinline__ void advance(const WgradGeom& g, int item_stride) {
    if (++r < r_end) {
      if (++nc == g.n_chunks) {
        nc = 0;
        if (++x == g.Wo) { x = 0; ++y; }
      }
    } else {
      start(g, item + item_stride);
    }
  }
};

__global__ void __launch_bounds__(kWgThreads, 1)
wgrad_kernel(const __grid_constant__ CUtensorMap map_dout, const __grid_constant__ CUtensorMap map_in,
             const __grid_constant__ WgradArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const WgradGeom& g = args.g;
  // Stage s: [filters' output gradient: 128 rows x 128 B][patch rows: 128 x 128 B], both
  // written by the copy engine with the 128-byte swizzle (16-byte chunk index XOR row
  // index mod 8), which needs 1024-byte aligned buffers.
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  // A ring stage holds kWgSub consecutive reduction steps (fewer at the end of an item): the
  // consumers pay one barrier round trip and one producer turn per stage.
  const int stages = g.stages / kWgSub;
  const uint32_t stage_bytes = (uint32_t)kWgSub * 2u * kWgOperandBytes;
  const uint32_t full_bar = base + (uint32_t)stages * stage_bytes;
  const uint32_t empty_bar = full_bar + 8u * stages;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar + 8u * s, 1);
      mbar_init(empty_bar + 8u * s, kWgThreads / 32);
    }
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  __syncthreads();

  // ------------------------------------------------ copy issue (warp 0, lane 0)
  WgradCursor pc;
  int p_stage = 0;
  uint32_t p_phase = 0;
  bool p_ok = true;
  const uint32_t tx_bytes = (uint32_t)(g.box_o + g.rows) * 128u;
  // The eight warps take turns at issuing the copies, one reduction step each (a fixed
  // issuing warp slows its scheduler, and the whole CTA runs at that scheduler's pace):
  // every thread keeps the cursor and advances it once per step; lane 0 of the warp whose
  // turn it is waits for the ring slot (free since two steps) and issues the two copies.
  auto produce = [&](bool mine) {
    if (pc.done(g)) return;
    const int n_sub = (pc.r + 1 < pc.r_end) ? kWgSub : 1;   // a stage never spans two items
    bool go = mine && p_ok;
    const uint32_t fb = full_bar + 8u * p_stage;
    const uint32_t dst = base + (uint32_t)p_stage * stage_bytes;
    if (go) {
      if (!mbar_wait(empty_bar + 8u * p_stage, p_phase ^ 1u, args.wc, kDevTimeoutEmpty)) {
        p_ok = false;
        go = false;
      } else {
        mbar_arrive_expect_tx(fb, (uint32_t)n_sub * tx_bytes);
      }
    }
    for (int sub = 0; sub < n_sub; ++sub) {
      if (go) {
        const uint32_t d2 = dst + (uint32_t)sub * 2u * kWgOperandBytes;
        tma_load_4d(d2, &map_dout, fb, pc.nc * 32, pc.x, pc.y, pc.ob * 128);
        tma_load_4d(d2 + kWgOperandBytes, &map_in, fb, pc.nc * 32, pc.x * g.stride_w - g.pad_w,
                    pc.y * g.stride_h - g.pad_h + pc.khb * g.bh, pc.cb * g.bc);
      }
      pc.advance(g, (int)gridDim.x);
    }
    if (++p_stage == stages) { p_stage = 0; p_phase ^= 1u; }
  };
  int turn = 0;
  if (warp == 0 && lane == 0) {
    prefetch_tensormap(&map_dout);
    prefetch_tensormap(&map_in);
  }
  pc.start(g, blockIdx.x);
  for (int s = 0; s + 2 < stages; ++s) produce(warp == 0 && lane == 0);
  __syncwarp();

  // ------------------------------------------------ arithmetic (all 8 warps)
  const int wo = warp >> 1, wn = warp & 1;
  const int to = wo * 4 + (lane >> 3);    // filters to + 16 j of the tile, j = 0..7
  const int tk = wn * 8 + (lane & 7);     // gradient rows tk + 16 i, i = 0..7
  // All threads walk the eight 16-byte chunks (4 values of r) in the same logical order
  // q.  The copy engine stored chunk q of a row at position q ^ (row mod 8).  A warp
  // reads, per load instruction, 8 patch rows (tk mod 8 all different) or 4 filter rows
  // (to mod 8 all different): different positions, hence different banks, and the
  // lanes that share a row share its 16 bytes — one shared-memory wavefront per load.
  // (Rows 8 to + j per thread would put a warp's 4 filter rows in the same banks: that
  // version spent 68 % of the shared-memory cycles and ran 20 % slower.)
  const uint32_t t7 = (uint32_t)tk & 7u, o7 = (uint32_t)to & 7u;
  const uint32_t p_base = kWgOperandBytes + (uint32_t)tk * 128u;
  const uint32_t g_base = (uint32_t)to * 128u;

  WgradCursor cc;
  cc.start(g, blockIdx.x);
  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;

  while (ok && !cc.done(g)) {
    float2 acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = make_float2(0.f, 0.f);
    const int item = cc.item;
    const int ob = cc.ob, cb = cc.cb, khb = cc.khb, split = cc.split;
    const int n_steps = cc.r_end - cc.r;

    for (int s = 0; s < n_steps; s += kWgSub) {
      produce(warp == turn && lane == 0);
      turn = (turn + 1) & 7;
      __syncwarp();
      if (!mbar_wait(full_bar + 8u * stage, phase, args.wc, kDevTimeoutFull)) {
        ok = false;
        break;
      }
      const int n_sub = (s + 1 < n_steps) ? kWgSub : 1;
#pragma unroll 1
      for (int sub = 0; sub < n_sub; ++sub) {
      const uint8_t* ss = base_ptr + (size_t)stage * stage_bytes + (size_t)sub * 2u * kWgOperandBytes;
      // Sixteen blocks per step: (16-byte chunk q, half of it): first the even pair of r for
      // all 64 results, then the odd pair, so consecutive multiply-adds never depend on each
      // other.  Operands come by 8-byte loads (beside a stream of packed multiply-adds an
      // 8-byte load is nearly free, a 16-byte load is not), and those of block b + 1 are
      // fetched into the second register buffer before block b's multiply-adds are issued
      // (+2.5 %; fetching the next step's first block ahead of the barrier as well made the
      // kernel spill and lose 7 %).
      float2 G[2][8], P[2][8];
      auto fetch = [&](int b, float2 (&Gb)[8], float2 (&Pb)[8]) {
        const int q = b >> 1, half = b & 1;
        const uint8_t* sg = ss + g_base + (((uint32_t)q ^ o7) << 4) + half * 8;
        const uint8_t* sp = ss + p_base + (((uint32_t)q ^ t7) << 4) + half * 8;
#pragma unroll
        for (int j = 0; j < 8; ++j) Gb[j] = lds64(sg + j * 2048);
#pragma unroll
        for (int i = 0; i < 8; ++i) Pb[i] = lds64(sp + i * 2048);
      };
      fetch(0, G[0], P[0]);
#pragma unroll
      for (int b = 0; b < 16; ++b) {
        if (b + 1 < 16) fetch(b + 1, G[(b + 1) & 1], P[(b + 1) & 1]);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
          for (int ii = 0; ii < 8; ++ii) {
            const int i = (j & 1) ? 7 - ii : ii;
            acc[i][j] = __ffma2_rn(P[b & 1][i], G[b & 1][j], acc[i][j]);
          }
        }
      }
      }   // sub
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar + 8u * stage);
      if (++stage == stages) { stage = 0; phase ^= 1u; }
    }
    if (!ok) break;
    // move the cursor past this item
    cc.start(g, item + (int)gridDim.x);

    // ---------------------------------------------- store this item's 128 x 128 block
    const bool direct = (g.splits == 1);
    const size_t K = (size_t)g.Nc * g.Skh * g.Skw;
    float* dst_base = direct ? args.dfilt : args.partial + (size_t)split * K * g.No;
    const float scale = direct ? g.alpha : 1.0f;
    const int o = ob * 128 + to;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = tk + 16 * i;                  // (c_l * bh + h_l) * bw + w_l
      if (row >= g.rows) continue;
      const int w_l = row % g.bw;
      const int t = row / g.bw;
      const int h_l = t % g.bh;
      const int c = cb * g.bc + t / g.bh;
      const int kh = khb * g.bh + h_l;
      if (c >= g.Nc || kh >= g.Skh) continue;
      float* dst = dst_base + (((size_t)c * g.Skh + kh) * g.Skw + w_l) * g.No + o;
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (o + 16 * j < g.No) dst[16 * j] = (acc[i][j].x + acc[i][j].y) * scale;
    }
  }

  // Exit path of the issuing lane after a wait ran out: let copies in flight land.
  if (lane == 0 && (!ok || !p_ok)) {
    for (int s = 0; s < stages; ++s) {
      const uint32_t par = (s < p_stage) ? p_phase : (p_phase ^ 1u);
      mbar_wait_grace(full_bar + 8u * s, par);
    }
  }
}

// dfilt[i] = alpha * (partial[0][i] + partial[1][i] + ... ), four elements per thread.
__global__ void __launch_bounds__(256)
wgrad_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dfilt, size_t n4,
                    int splits, float alpha) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const float4* p = reinterpret_cast<const float4*>(partial);
  float4 s = p[i];
  for (int k = 1; k < splits; ++k) {
    const float4 v = p[(size_t)k * n4 + i];
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  reinterpret_cast<float4*>(dfilt)[i] = make_float4(s.x * alpha, s.y * alpha, s.z * alpha, s.w * alpha);
}

}  // namespace maxdnn
