// Exact-fp32 FPROP convolution kernel for sm_100a.
//
// One persistent CTA per SM walks a list of tiles.  A tile is the GEMM block of
// Section 3.2: tile_m filters x (tile_px adjacent output pixels x tile_n images),
// 128 columns wide.  Warp 8 is the producer: one elected lane walks the K-step
// table (Section 3.2's precomputed offsets) and issues, per step, one bulk tensor
// copy of filter-matrix rows and tile_px copies of patch rows into a ring of
// shared-memory stages; the copy engine zero-fills the apron, so the consumers
// never test a bound.  Warps 0-7 are consumers: each thread owns an MR x 8
// register block (Section 3.1's 8 x 8 register blocking) and runs a flat loop
// of shared loads and packed fp32 multiply-adds, operands double-buffered in
// registers (Section 3.1, "double buffering of shared memory loads").
#pragma once
#include "plan.h"
#include "ptx_util.cuh"

namespace maxdnn {

constexpr int kFfmaConsumerWarps = 8;
// Eight consumer warps plus the producer warp.
constexpr int ffma_threads(int) { return (kFfmaConsumerWarps + 1) * 32; }

struct FfmaArgs {
  ConvGeom g;
  float* out;
  uint32_t* status;
  KStepTable table;
};

template <int MR>
struct Frag {
  float2 a[MR / 2];
  float4 b[2];
};

template <int MR>
__device__ __forceinline__ void load_frag(Frag<MR>& f, const float* a_row, const float* b0,
                                          const float* b1) {
  if constexpr (MR % 4 == 0) {
#pragma unroll
    for (int q = 0; q < MR / 4; ++q) {
      const float4 v = *reinterpret_cast<const float4*>(a_row + q * 64);
      f.a[2 * q] = make_float2(v.x, v.y);
      f.a[2 * q + 1] = make_float2(v.z, v.w);
    }
  } else {
#pragma unroll
    for (int p = 0; p < MR / 2; ++p) f.a[p] = *reinterpret_cast<const float2*>(a_row + p * 32);
  }
  f.b[0] = *reinterpret_cast<const float4*>(b0);
  f.b[1] = *reinterpret_cast<const float4*>(b1);
}

// acc pairs: P[i][j] = {acc(2i,2j), acc(2i+1,2j+1)}, Q[i][j] = {acc(2i,2j+1), acc(2i+1,2j)}.
// Both products of a 2 x 2 sub-block come from one packed multiply-add each: the
// filter pair times the patch pair, and the filter pair times the swapped patch pair.
template <int MR>
__device__ __forceinline__ void fma_block(const Frag<MR>& f, float2 (&P)[MR / 2][4],
                                          float2 (&Q)[MR / 2][4]) {
  float2 bn[4], bs[4];
  bn[0] = make_float2(f.b[0].x, f.b[0].y);
  bn[1] = make_float2(f.b[0].z, f.b[0].w);
  bn[2] = make_float2(f.b[1].x, f.b[1].y);
  bn[3] = make_float2(f.b[1].z, f.b[1].w);
#pragma unroll
  for (int j = 0; j < 4; ++j) bs[j] = make_float2(bn[j].y, bn[j].x);
#pragma unroll
  for (int i = 0; i < MR / 2; ++i) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      P[i][j] = __ffma2_rn(f.a[i], bn[j], P[i][j]);
      Q[i][j] = __ffma2_rn(f.a[i], bs[j], Q[i][j]);
    }
  }
}

// One row of the flat loop: operand loads for the row after next are issued
// before the multiply-adds of the current row (register double buffering).
#define MAXDNN_ROW_PTRS(R) a_ptr + (R) * Mt, b0_ptr + (R) * b_pitch, b1_ptr + (R) * b_pitch

template <int MR, bool FIXED>
__global__ void __launch_bounds__(ffma_threads(MR), 1)
ffma_conv_kernel(const __grid_constant__ CUtensorMap map_filt,
                 const __grid_constant__ CUtensorMap map_in,
                 const __grid_constant__ FfmaArgs args) {
  constexpr int Mt = 16 * MR;
  extern __shared__ uint8_t smem_raw[];
  const ConvGeom& g = args.g;

  // Carve shared memory: [stages x filter box][stages x patch boxes][barriers].
  const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int stages = g.stages;
  const uint32_t a_off = 0;
  const uint32_t b_off = (uint32_t)stages * g.a_stage_bytes;
  const uint32_t bar_off = b_off + (uint32_t)stages * g.b_stage_bytes;
  const uint32_t full_bar = base + bar_off;          // stages x 8 bytes
  const uint32_t empty_bar = full_bar + 8u * stages; // stages x 8 bytes

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar + 8u * s, 1);
      mbar_init(empty_bar + 8u * s, kFfmaConsumerWarps);
    }
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  __syncthreads();

  const int n_ksteps = g.n_ksteps;
  const int rows = g.rows;

  if (warp >= kFfmaConsumerWarps) {
    // ------------------------------------------------------------ producer
    if (warp == kFfmaConsumerWarps && lane == 0) {
      prefetch_tensormap(&map_filt);
      prefetch_tensormap(&map_in);
      const uint32_t tx_bytes = (uint32_t)(g.a_box_bytes + g.b_boxes * g.b_box_bytes);
      const int w_step = g.stride;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < g.n_tiles && ok; tile += gridDim.x) {
        int r = tile;
        const int ob = r % g.o_blocks; r /= g.o_blocks;
        const int nch = r % g.n_chunks; r /= g.n_chunks;
        const int xr = r % g.x_runs;
        const int y = r / g.x_runs;
        const int o0 = ob * Mt;
        const int n0 = nch * g.tile_n;
        const int h0 = y * g.stride - g.pad;
        const int w0 = xr * g.tile_px * g.stride - g.pad;
        for (int s = 0; s < n_ksteps; ++s) {
          if (!mbar_wait_backoff(empty_bar + 8u * stage, phase ^ 1u, args.status,
                                 kDevTimeoutEmpty)) {
            ok = false;
            break;
          }
          const maxdnn_kstep ks = args.table.s[s];
          const uint32_t fb = full_bar + 8u * stage;
          mbar_arrive_expect_tx(fb, tx_bytes);
          tma_load_4d(base + a_off + (uint32_t)stage * g.a_stage_bytes, &map_filt, fb, o0, ks.kw0,
                      ks.kh, ks.c0);
          uint32_t dst = base + b_off + (uint32_t)stage * g.b_stage_bytes;
          int w = w0 + ks.kw0;
          for (int t = 0; t < g.b_boxes; ++t) {
            tma_load_4d(dst, &map_in, fb, n0, w, h0 + ks.kh, ks.c0);
            dst += g.b_slot_bytes;
            w += w_step;
          }
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Leaving early: let every copy already issued land before the CTA's
        // shared memory is released.
        for (int s = 0; s < stages; ++s) {
          const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
          mbar_wait(full_bar + 8u * s, par, nullptr, kDevTimeoutDrain);
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  const int wo = warp >> 1, wn = warp & 1;
  const int to = wo * 4 + (lane >> 3);   // 0..15 along the filter axis
  const int tn = wn * 8 + (lane & 7);    // 0..15 along the column axis
  const int a_elem = (MR % 4 == 0) ? 4 * to : 2 * to;

  // This thread's two groups of four columns -> (pixel, image) and smem offset.
  const int used_cols = g.tile_px * g.tile_n;
  int col_px[2], col_n[2];
  uint32_t b_elem[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int col = 4 * tn + 64 * h;
    const bool live = col < used_cols;
    col_px[h] = live ? col / g.tile_n : -1;
    col_n[h] = live ? col % g.tile_n : 0;
    if (FIXED)
      b_elem[h] = (uint32_t)col;
    else
      b_elem[h] = live ? (uint32_t)(col_px[h] * (g.b_slot_bytes >> 2) + col_n[h]) : 0u;
  }
  const int b_pitch = FIXED ? kTileCols : g.tile_n;   // floats between patch rows

  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;

  for (int tile = blockIdx.x; tile < g.n_tiles && ok; tile += gridDim.x) {
    float2 P[MR / 2][4], Q[MR / 2][4];
#pragma unroll
    for (int i = 0; i < MR / 2; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        P[i][j] = make_float2(0.f, 0.f);
        Q[i][j] = make_float2(0.f, 0.f);
      }

    Frag<MR> f0, f1;
    ok = mbar_wait(full_bar + 8u * stage, phase, args.status, kDevTimeoutFull);
    if (!ok) break;
    const float* a_ptr =
        reinterpret_cast<const float*>(base_ptr + a_off + (size_t)stage * g.a_stage_bytes) + a_elem;
    const float* bs_ptr =
        reinterpret_cast<const float*>(base_ptr + b_off + (size_t)stage * g.b_stage_bytes);
    const float* b0_ptr = bs_ptr + b_elem[0];
    const float* b1_ptr = bs_ptr + b_elem[1];
    load_frag<MR>(f0, MAXDNN_ROW_PTRS(0));

    for (int s = 0; s < n_ksteps; ++s) {
      // f0 holds row 0 of this stage.  Four rows per iteration while the row
      // after the block is still inside the stage.
      int r = 0;
#pragma unroll 1
      for (; r + 4 < rows; r += 4) {
        load_frag<MR>(f1, MAXDNN_ROW_PTRS(1));
        fma_block<MR>(f0, P, Q);
        load_frag<MR>(f0, MAXDNN_ROW_PTRS(2));
        fma_block<MR>(f1, P, Q);
        load_frag<MR>(f1, MAXDNN_ROW_PTRS(3));
        fma_block<MR>(f0, P, Q);
        load_frag<MR>(f0, MAXDNN_ROW_PTRS(4));
        fma_block<MR>(f1, P, Q);
        a_ptr += 4 * Mt; b0_ptr += 4 * b_pitch; b1_ptr += 4 * b_pitch;
      }
#pragma unroll 1
      for (; rows - r > 2; r += 2) {   // 3 or 4 rows left: two of them here
        load_frag<MR>(f1, MAXDNN_ROW_PTRS(1));
        fma_block<MR>(f0, P, Q);
        load_frag<MR>(f0, MAXDNN_ROW_PTRS(2));
        fma_block<MR>(f1, P, Q);
        a_ptr += 2 * Mt; b0_ptr += 2 * b_pitch; b1_ptr += 2 * b_pitch;
      }
      const bool two_left = (rows - r == 2);
      if (two_left) {
        load_frag<MR>(f1, MAXDNN_ROW_PTRS(1));
        fma_block<MR>(f0, P, Q);
      }
      // The last row of this stage is in f1 (two_left) or f0.  Prefetch row 0 of
      // the next stage into the other buffer before computing it.
      const int cur_stage = stage;
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      const bool more = s + 1 < n_ksteps;
      if (more) {
        ok = mbar_wait(full_bar + 8u * stage, phase, args.status, kDevTimeoutFull);
        if (!ok) break;
        a_ptr = reinterpret_cast<const float*>(base_ptr + a_off + (size_t)stage * g.a_stage_bytes) +
                a_elem;
        bs_ptr = reinterpret_cast<const float*>(base_ptr + b_off + (size_t)stage * g.b_stage_bytes);
        b0_ptr = bs_ptr + b_elem[0];
        b1_ptr = bs_ptr + b_elem[1];
      }
      if (two_left) {
        if (more) load_frag<MR>(f0, MAXDNN_ROW_PTRS(0));
        fma_block<MR>(f1, P, Q);
      } else {
        if (more) load_frag<MR>(f1, MAXDNN_ROW_PTRS(0));
        fma_block<MR>(f0, P, Q);
        f0 = f1;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar + 8u * cur_stage);
    }
    if (!ok) break;

    // ---------------------------------------------------------- epilogue
    // alpha scaling and store; for a fixed filter a quarter-warp writes one full
    // 128-byte line of `out`, so stores are coalesced straight from registers.
    {
      int r = tile;
      const int ob = r % g.o_blocks; r /= g.o_blocks;
      const int nch = r % g.n_chunks; r /= g.n_chunks;
      const int xr = r % g.x_runs;
      const int y = r / g.x_runs;
      const int o0 = ob * Mt;
      const int n0 = nch * g.tile_n;
      const int x0 = xr * g.tile_px;
      const float alpha = g.alpha;
#pragma unroll
      for (int i = 0; i < MR; ++i) {
        const int o_local = (MR % 4 == 0) ? ((i >> 2) * 64 + 4 * to + (i & 3))
                                          : ((i >> 1) * 32 + 2 * to + (i & 1));
        const int o = o0 + o_local;
        if (o >= g.No) continue;
        const int i2 = i >> 1, ia = i & 1;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int x = x0 + col_px[h];
          const int n = n0 + col_n[h];
          if (col_px[h] < 0 || x >= g.Wo || n >= g.Nb) continue;
          float4 v;
          // columns 4h .. 4h+3 of this row: j = 2*j2 + jb with j2 = 2h, 2h+1
          v.x = ia == 0 ? P[i2][2 * h].x : Q[i2][2 * h].y;
          v.y = ia == 0 ? Q[i2][2 * h].x : P[i2][2 * h].y;
          v.z = ia == 0 ? P[i2][2 * h + 1].x : Q[i2][2 * h + 1].y;
          v.w = ia == 0 ? Q[i2][2 * h + 1].x : P[i2][2 * h + 1].y;
          v.x *= alpha; v.y *= alpha; v.z *= alpha; v.w *= alpha;
          float* dst = args.out + (((size_t)o * g.Ho + y) * g.Wo + x) * (size_t)g.Nb + n;
          __stcs(reinterpret_cast<float4*>(dst), v);
        }
      }
    }
  }
}
#undef MAXDNN_ROW_PTRS

}  // namespace maxdnn
