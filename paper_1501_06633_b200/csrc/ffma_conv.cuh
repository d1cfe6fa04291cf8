// Exact-fp32 FPROP convolution kernel for sm_100a.
//
// One persistent CTA per SM walks a list of tiles.  A tile is the GEMM block of
// Section 3.2: tile_m filters x (tile_px adjacent output pixels x tile_n images).
// The producer — one lane — walks the K-step table (Section 3.2's precomputed
// offsets) and issues, per step, one bulk tensor copy of filter-matrix rows and one
// (or tile_px) copies of patch rows into a ring of shared-memory stages; the copy
// engine zero-fills the apron, so the consumers never test a bound.  Eight consumer
// warps: each thread owns an MR x NR register block (Section 3.1's register
// blocking) and runs a flat loop of shared loads and packed fp32 multiply-adds,
// operands double-buffered in registers (Section 3.1, "double buffering of shared
// memory loads").
//
// The producer is a ninth warp when the register block leaves room for it
// (registers are allocated per four warps, so nine warps cap a thread at 168).
// Larger blocks (MR*NR >= 96) run with eight warps and 255 registers; there the
// consumer warps take turns at issuing the copies, one K step each.
#pragma once
#include "plan.h"
#include "ptx_util.cuh"

namespace maxdnn {

constexpr int kFfmaConsumerWarps = 8;
__host__ __device__ constexpr bool ffma_inline_producer(int mr, int nr) { return mr * nr >= kFfmaInlineMinAcc; }
__host__ __device__ constexpr int ffma_threads(int mr, int nr, bool ragged = false) {
  // ragged: four copy warps (two for patches, two for filters) that move the rows themselves
  return (kFfmaConsumerWarps + (ragged ? 4 : ffma_inline_producer(mr, nr) ? 0 : 1)) * 32;
}

// Multiply-add order per register-block shape (see fma_block), from timings on B200.
__host__ __device__ constexpr int ffma_order(int mr, int nr) {
  return (mr == 16 && nr == 8) ? 0 : (mr == 6 && nr == 8) ? 2 : 1;
}

// Rows of K per iteration of the main loop, by register block and rows per K step
// (long_steps: 96 rows and more).  The 8 x 8 and 6 x 8 blocks gain 5-8 % from long iterations
// (16 rows for steps of 32 to 64 rows, 32 rows for the ~100-row steps; 12 to 30 rows measure
// alike, 46 rows overflow the instruction cache: -10 %); the 4 x 8 block gains 3.5 % from 32
// rows on ~100-row steps and loses 2-3 % from long iterations on 32-row steps; the blocks of
// 128 accumulators lose 1.5 % with 8 rows, the 4 x 16 block 2-3 %: those keep 4.
__host__ __device__ constexpr int ffma_long_block(int mr, int nr, bool long_steps) {
  if (mr == 4 && nr == 8) return long_steps ? 32 : 4;
  return ((mr == 8 || mr == 6) && nr == 8) ? (long_steps ? 32 : 16) : 4;
}

struct FfmaArgs {
  ConvGeom g;
  float* out;
  WaitCtx wc;          // status block and this launch's epoch (see ptx_util.cuh)
  // Test hook for the bounded waits: if non-zero, CTA 0 initialises its "full" barriers
  // to expect one arrival more than they will ever get, so the consumers' first wait
  // runs out and the kernel reports kDevTimeoutFull instead of hanging.
  uint32_t test_missing_arrival;
  // Non-zero: every CTA adds its elapsed SM cycles and nanoseconds (first instruction to
  // last store) to words 2 and 3 (split-tail kernel: 4 and 5) of the status block with atomicMax — the elapsed
  // processor clocks of Section 3.3's efficiency formula, measured inside the kernel.
  uint32_t clock_stamp;
  // Split tail (g.sk_tiles > 0): one slot of tile_m x tile_cols partial sums per CTA, and
  // one flag word per CTA that receives this launch's epoch when the slot is complete.
  float* sk_partial;
  uint32_t* sk_flags;
  KStepTable table;
  // Ragged kernel only (Nb or No not a multiple of 4, which the bulk tensor copies cannot
  // address): the tensors themselves, read by the copy warps with 4-byte asynchronous copies.
  const float* in;
  const float* filt;
};

// ---------------------------------------------------------------------------------------
// Work items.  A CTA walks whole tiles first (static round-robin over [tile_begin,
// sk_first)), then its share of the SPLIT TAIL: the last sk_tiles tiles, fewer than the
// grid has CTAs, would leave SMs idle for a whole tile's time, so their K steps — sk_tiles x
// n_ksteps of them, numbered tile by tile — are dealt out evenly, CTA i taking the
// contiguous range [i U / G, (i + 1) U / G).  A range is shorter than one tile, so it covers
// the end of one tile and / or the beginning of the next.  The CTA whose range holds a
// tile's LAST K step finishes that tile: it adds the partial sums that the lower-numbered
// CTAs holding the tile's earlier steps wrote to their slots, in CTA order (a fixed order:
// results are bitwise reproducible), then scales and stores.  Every CTA does its
// contributing piece before its finishing piece, so a finisher waits only for CTAs with
// lower numbers, which never wait for it.
// ---------------------------------------------------------------------------------------
// The item arithmetic itself (ffma_item_at, sk_range) lives in plan.h so that the host can
// list a CTA's items too.
__device__ __forceinline__ bool ffma_item(const ConvGeom& g, int k, FfmaItem& it) {
  return ffma_item_at(g, (int)gridDim.x, (int)blockIdx.x, k, it);
}

template <int MR, int NR>
struct Frag {
  float2 a[MR / 2];
  float4 b[NR / 4];
};

// Thread (to, tn) of the 16 x 16 consumer grid reads, from row `a_row` of the staged
// filter box, MR values (float4 groups 64 filters apart, or float2 groups 32 apart)
// and, from the staged patch row, NR values (float4 groups 64 columns apart).
// W64: every group of four is fetched by two 8-byte loads instead of one 16-byte load.
template <int MR, int NR, bool FIXED, bool W64>
__device__ __forceinline__ void load_frag(Frag<MR, NR>& f, const float* a_row,
                                          const float* const (&b_row)[NR / 4], int b_off) {
  if constexpr (MR % 4 == 0) {
#pragma unroll
    for (int q = 0; q < MR / 4; ++q) {
      if constexpr (W64) {
        f.a[2 * q] = lds64(a_row + q * 64);
        f.a[2 * q + 1] = lds64(a_row + q * 64 + 2);
      } else {
        const float4 v = *reinterpret_cast<const float4*>(a_row + q * 64);
        f.a[2 * q] = make_float2(v.x, v.y);
        f.a[2 * q + 1] = make_float2(v.z, v.w);
      }
    }
  } else {
#pragma unroll
    for (int p = 0; p < MR / 2; ++p) f.a[p] = *reinterpret_cast<const float2*>(a_row + p * 32);
  }
#pragma unroll
  for (int h = 0; h < NR / 4; ++h) {
    const float* src = FIXED ? b_row[0] + b_off + 64 * h : b_row[h] + b_off;
    if constexpr (W64) {
      const float2 lo = lds64(src), hi = lds64(src + 2);
      f.b[h] = make_float4(lo.x, lo.y, hi.x, hi.y);
    } else {
      f.b[h] = *reinterpret_cast<const float4*>(src);
    }
  }
}

// acc pairs: P[i][j] = {acc(2i,2j), acc(2i+1,2j+1)}, Q[i][j] = {acc(2i,2j+1), acc(2i+1,2j)}.
// Both products of a 2 x 2 sub-block come from one packed multiply-add each: the
// filter pair times the patch pair, and the filter pair times the swapped patch pair.
template <int MR, int NR>
__device__ __forceinline__ void fma_block(const Frag<MR, NR>& f, float2 (&P)[MR / 2][NR / 2],
                                          float2 (&Q)[MR / 2][NR / 2]) {
  float2 bn[NR / 2], bs[NR / 2];
#pragma unroll
  for (int h = 0; h < NR / 4; ++h) {
    bn[2 * h] = make_float2(f.b[h].x, f.b[h].y);
    bn[2 * h + 1] = make_float2(f.b[h].z, f.b[h].w);
  }
#pragma unroll
  for (int j = 0; j < NR / 2; ++j) bs[j] = make_float2(bn[j].y, bn[j].x);
  // The order of the multiply-adds decides how often consecutive instructions share an
  // operand register (and how they collide in the register banks); measured per block
  // shape, 3-6 % apart.  All orders walk the column pairs in the outer loop.
  constexpr int kOrder = ffma_order(MR, NR);
#pragma unroll
  for (int j = 0; j < NR / 2; ++j) {
#pragma unroll
    for (int ii = 0; ii < MR / 2; ++ii) {
      // kOrder 0: filter pairs ascending; 1, 2: serpentine (back down on odd columns)
      const int i = (kOrder != 0 && (j & 1)) ? (MR / 2 - 1 - ii) : ii;
      if (kOrder == 2 && (j & 1)) {   // 2: swapped-pair product first on the way back
        Q[i][j] = __ffma2_rn(f.a[i], bs[j], Q[i][j]);
        P[i][j] = __ffma2_rn(f.a[i], bn[j], P[i][j]);
      } else {
        P[i][j] = __ffma2_rn(f.a[i], bn[j], P[i][j]);
        Q[i][j] = __ffma2_rn(f.a[i], bs[j], Q[i][j]);
      }
    }
  }
}

// Producer state: which K step of which tile is loaded next, into which ring stage.  The
// whole-tile kernel (SPLIT = false) walks tiles tile_begin + CTA, + grid, ... below tile_end,
// all K steps of each; the split-tail kernel walks this CTA's work items.
template <bool SPLIT>
struct FfmaProducer {
  int item, step, step_end, stage;   // item: tile number (whole tiles) or item number (split)
  uint32_t phase;                    // step_end <= step: no work left
  int o0, n0, h0, w0;

  __device__ __forceinline__ void set_item(const ConvGeom& g, int mt) {
    int r;
    if constexpr (SPLIT) {
      FfmaItem it;
      if (!ffma_item(g, item, it)) { step = 0; step_end = -1; return; }
      step = it.s0; step_end = it.s1;
      r = it.tile;
    } else {
      if (item >= g.tile_end) { step = 0; step_end = -1; return; }
      step = 0; step_end = g.n_ksteps;
      r = item;
    }
    const int ob = r % g.o_blocks; r /= g.o_blocks;
    const int nch = r % g.n_chunks; r /= g.n_chunks;
    const int xr = r % g.x_runs;
    const int y = r / g.x_runs;
    o0 = ob * mt;
    n0 = nch * g.tile_n;
    h0 = y * g.stride_h - g.pad_h;
    w0 = xr * g.tile_px * g.stride_w - g.pad_w;
  }

  __device__ __forceinline__ void init(const ConvGeom& g, int mt) {
    item = SPLIT ? 0 : g.tile_begin + (int)blockIdx.x;
    stage = 0; phase = 0;
    o0 = n0 = h0 = w0 = 0;
    set_item(g, mt);
  }

  __device__ __forceinline__ bool has_work(const ConvGeom&) const { return step < step_end; }

  // Waits for the ring slot, issues the copies of one K step, advances.
  template <bool BACKOFF>
  __device__ __forceinline__ bool issue(const FfmaArgs& args, const CUtensorMap* map_filt,
                                        const CUtensorMap* map_in, uint32_t a_base, uint32_t b_base,
                                        uint32_t full_bar, uint32_t empty_bar, int mt) {
    const ConvGeom& g = args.g;
    const uint32_t eb = empty_bar + 8u * stage;
    const bool ok = BACKOFF ? mbar_wait_backoff(eb, phase ^ 1u, args.wc, kDevTimeoutEmpty)
                            : mbar_wait(eb, phase ^ 1u, args.wc, kDevTimeoutEmpty);
    if (!ok) return false;
    const maxdnn_kstep ks = args.table.s[step];
    const uint32_t fb = full_bar + 8u * stage;
    mbar_arrive_expect_tx(fb, (uint32_t)(g.a_box_bytes + g.b_boxes * g.b_box_bytes));
    // boxes are (o | n, kw | w, c, kh | h): filter rows outermost, so that the rows of a short
    // last step are the leading rows of its box
    tma_load_4d(a_base + (uint32_t)stage * g.a_stage_bytes, map_filt, fb, o0, ks.kw0, ks.c0, ks.kh);
    uint32_t dst = b_base + (uint32_t)stage * g.b_stage_bytes;
    int w = w0 + ks.kw0;
    for (int t = 0; t < g.b_boxes; ++t) {
      tma_load_4d(dst, map_in, fb, n0, w, ks.c0, h0 + ks.kh);
      dst += g.b_slot_bytes;
      w += g.stride_w;
    }
    advance(g, mt);
    return true;
  }

  // The state after one more K step has been issued (by this thread or by another one that
  // keeps an identical copy of the state).
  __device__ __forceinline__ void advance(const ConvGeom& g, int mt) {
    if (++stage == g.stages) { stage = 0; phase ^= 1u; }
    if (++step == step_end) {
      item += SPLIT ? 1 : (int)gridDim.x;
      set_item(g, mt);
    }
  }

  // After a failed wait: let every copy already issued land before the CTA's shared
  // memory is released.
  __device__ __forceinline__ void drain(const ConvGeom& g, uint32_t full_bar) {
    for (int s = 0; s < g.stages; ++s) {
      const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
      mbar_wait_grace(full_bar + 8u * s, par);
    }
  }
};

// Bounded wait for a peer CTA's "slot complete" flag (split tail).
__device__ __noinline__ bool wait_peer_flag(const uint32_t* flag, uint32_t epoch, const WaitCtx& wc) {
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      uint32_t v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
      if (v == epoch) return true;
      __nanosleep(100);
    }
    if (globaltimer_ns() - t0 > kWaitBudgetNs) break;
    if (launch_gave_up(wc)) break;
  }
  record_give_up(wc, kDevTimeoutPeer);
  return false;
}



// ---------------------------------------------------------------------------------------
// Ragged shapes.  A row of Nb images (or No filters) that is not a multiple of 16 bytes
// cannot be the pitch of a bulk tensor copy.  The ragged kernel therefore stages the same
// boxes with ordinary loads and shared-memory stores of 4 or 8 bytes (zeros for what lies
// outside the tensors — the apron, the tails of Nb and No, surplus rows of a K step), made
// by four copy warps: two for the patch rows, two for the filter rows, each arriving on the
// stage's "full" barrier when its rows are written (4 arrivals per stage).  The
// staged layout is the one-box-per-pixel layout of the bulk path, so the consumers are
// unchanged; the epilogue stores element by element with bounds.
// ---------------------------------------------------------------------------------------
// VEC floats (4 or 8 bytes) of one lane: loaded from global memory (zeros if !valid; the
// source is not read then) and stored to shared memory.
template <int VEC> struct RaggedVal { float v[VEC]; };
template <int VEC>
__device__ __forceinline__ RaggedVal<VEC> ragged_ldg(const float* src, bool valid) {
  RaggedVal<VEC> r;
  if constexpr (VEC == 2) {
    float2 t = make_float2(0.f, 0.f);
    if (valid) t = __ldg(reinterpret_cast<const float2*>(src));
    r.v[0] = t.x; r.v[1] = t.y;
  } else {
    r.v[0] = valid ? __ldg(src) : 0.f;
  }
  return r;
}
template <int VEC>
__device__ __forceinline__ void ragged_sts(uint32_t dst, const RaggedVal<VEC>& r) {
  if constexpr (VEC == 2)
    asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(dst), "f"(r.v[0]), "f"(r.v[1]) : "memory");
  else
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst), "f"(r.v[0]) : "memory");
}

// One copy warp's whole life: every K step of every tile of this CTA.  PATCH: the patch
// rows [pixel][kh][c][kw] of tile_n images each; else the filter rows [kh][c][kw] of MT
// filters.  Two warps share each kind, each taking half of a box's channels.  The copy
// warps compete with eight warps of packed multiply-adds for issue slots (those leave about
// a tenth), so the loop over a box's channels is bare: one load, one shared-memory store and
// two pointer increments per 32 x VEC floats, eight loads in flight per lane; everything
// that depends on the pixel, the filter row or column is computed outside it.
// (Asynchronous copies of 4 or 8 bytes were tried first and were no faster: the limit is
// the instruction count of the copy warps, not the copy mechanism.)
template <int MT, bool PATCH, int VEC>
__device__ __forceinline__ void ragged_copy_loop(const FfmaArgs& args, int part, int parts,
                                                 uint32_t stage_base, uint32_t stage_bytes,
                                                 uint32_t full_bar, uint32_t empty_bar,
                                                 const CUtensorMap* map_filt, uint32_t a_base) {
  constexpr int kInFlight = 8;
  const ConvGeom& g = args.g;
  const int lane = threadIdx.x & 31;
  const float* const tensor = PATCH ? args.in : args.filt;
  const int len = PATCH ? g.tile_n : MT;                       // floats per staged row
  const uint32_t row_bytes = 4u * (uint32_t)len;
  const uint32_t c_pitch = row_bytes * (uint32_t)g.kwc;        // next channel in the stage
  const size_t plane = PATCH ? (size_t)g.Hi * g.Wi * g.Nb : (size_t)g.Skh * g.Skw * g.No;
  const int ci_lo = part * g.kc / parts, ci_hi = (part + 1) * g.kc / parts;   // this warp's channels
  int stage = 0;
  uint32_t phase = 0;
  for (int tile = g.tile_begin + (int)blockIdx.x; tile < g.tile_end; tile += (int)gridDim.x) {
    int r = tile;
    const int ob = r % g.o_blocks; r /= g.o_blocks;
    const int nch = r % g.n_chunks; r /= g.n_chunks;
    const int xr = r % g.x_runs;
    const int y = r / g.x_runs;
    const int i0 = PATCH ? nch * g.tile_n : ob * MT;              // first image / filter
    const int n_valid = min(len, (PATCH ? g.Nb : g.No) - i0);
    const int x0 = xr * g.tile_px;
    for (int s = 0; s < g.n_ksteps; ++s) {
      if (!mbar_wait_backoff(empty_bar + 8u * stage, phase ^ 1u, args.wc, kDevTimeoutEmpty)) return;
      const maxdnn_kstep ks = args.table.s[s];
      const uint32_t dst0 = stage_base + (uint32_t)stage * stage_bytes;
      const int c_valid = g.Nc - ks.c0;                            // channels of the box inside the tensor
      if (map_filt != nullptr && lane == 0) {
        // filter rows that the bulk tensor copy can address (No a multiple of 4): one copy,
        // counted on the same barrier (this arrival is the barrier's fifth)
        const uint32_t fb = full_bar + 8u * stage;
        mbar_arrive_expect_tx(fb, (uint32_t)g.a_box_bytes);
        tma_load_4d(a_base + (uint32_t)stage * g.a_stage_bytes, map_filt, fb, ob * MT, ks.kw0, ks.c0, ks.kh);
      }
      for (int t = 0; t < (PATCH ? g.tile_px : 1); ++t) {
        for (int khi = 0; khi < g.box_kh; ++khi) {
          for (int kwi = 0; kwi < g.kwc; ++kwi) {
            // the row of channel c0 for this (pixel, filter row, filter column), and whether
            // it lies inside the tensor
            bool ok;
            size_t off;
            if constexpr (PATCH) {
              const int h = y * g.stride_h - g.pad_h + ks.kh + khi;
              const int w = (x0 + t) * g.stride_w - g.pad_w + ks.kw0 + kwi;
              ok = ks.kh + khi < g.Skh && h >= 0 && h < g.Hi && w >= 0 && w < g.Wi;
              off = ok ? (((size_t)ks.c0 * g.Hi + h) * g.Wi + w) * (size_t)g.Nb : 0;
            } else {
              const int kh = ks.kh + khi, kw = ks.kw0 + kwi;
              ok = kh < g.Skh && kw < g.Skw;
              off = ok ? (((size_t)ks.c0 * g.Skh + kh) * g.Skw + kw) * (size_t)g.No : 0;
            }
            const uint32_t d_row = dst0 + (PATCH ? (uint32_t)t * g.b_slot_bytes : 0u) +
                                   (uint32_t)(khi * g.kc * g.kwc + kwi) * row_bytes;
            for (int e = lane * VEC; e < len; e += 32 * VEC) {
              const bool e_ok = ok && e < n_valid;
              const float* src = tensor + (e_ok ? off + i0 + e + (size_t)ci_lo * plane : 0);
              uint32_t dst = d_row + 4u * (uint32_t)e + (uint32_t)ci_lo * c_pitch;
              for (int ci = ci_lo; ci < ci_hi; ci += kInFlight) {
                RaggedVal<VEC> val[kInFlight];
#pragma unroll
                for (int j = 0; j < kInFlight; ++j)
                  val[j] = ragged_ldg<VEC>(src + (e_ok ? j * plane : 0), e_ok && ci + j < c_valid);
#pragma unroll
                for (int j = 0; j < kInFlight; ++j)
                  if (ci + j < ci_hi) ragged_sts<VEC>(dst + (uint32_t)j * c_pitch, val[j]);
                if (e_ok) src += kInFlight * plane;
                dst += (uint32_t)kInFlight * c_pitch;
              }
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar + 8u * stage);
      if (++stage == g.stages) { stage = 0; phase ^= 1u; }
    }
  }
}

// 8-byte pieces where every row start and every row length allows it, else 4-byte ones.
// With ragged filters (No not a multiple of 4) warps 0, 1 copy patches and 2, 3 filters;
// else all four copy patches and lane 0 of the first also issues the filter boxes as bulk
// tensor copies.
template <int MT>
__device__ __noinline__ void ragged_copy_warp(const FfmaArgs& args, int role, const CUtensorMap* map_filt,
                                              uint32_t a_base, uint32_t b_base, uint32_t full_bar,
                                              uint32_t empty_bar) {
  const ConvGeom& g = args.g;
  const bool filt_bulk = (g.No & 3) == 0;
  const bool patch_role = filt_bulk || role < 2;
  const int parts = filt_bulk ? 4 : 2, part = filt_bulk ? role : (role & 1);
  const CUtensorMap* mf = (filt_bulk && role == 0) ? map_filt : nullptr;
  if (patch_role) {
    const bool pairs = ((g.Nb | g.tile_n) & 1) == 0 && (reinterpret_cast<uintptr_t>(args.in) & 7) == 0;
    if (pairs) ragged_copy_loop<MT, true, 2>(args, part, parts, b_base, g.b_stage_bytes, full_bar, empty_bar, mf, a_base);
    else ragged_copy_loop<MT, true, 1>(args, part, parts, b_base, g.b_stage_bytes, full_bar, empty_bar, mf, a_base);
  } else {
    const bool pairs = (g.No & 1) == 0 && (reinterpret_cast<uintptr_t>(args.filt) & 7) == 0;
    if (pairs) ragged_copy_loop<MT, false, 2>(args, part, parts, a_base, g.a_stage_bytes, full_bar, empty_bar, nullptr, 0);
    else ragged_copy_loop<MT, false, 1>(args, part, parts, a_base, g.a_stage_bytes, full_bar, empty_bar, nullptr, 0);
  }
}

#define MAXDNN_ROW(R) a_ptr + (R) * Mt, b_ptr, (R) * b_pitch

// SPLIT = false: whole tiles [tile_begin, tile_end).  SPLIT = true: this CTA's pieces of the
// split tail (launched after the whole-tile kernel on the same stream; work items as if
// tile_begin were the first split tile).  Operands come by 8-byte loads for the blocks of
// 16 columns and by 16-byte loads for the others (which is faster was measured per block).
// RAGGED: the copy warps of ragged_copy_warp instead of bulk tensor copies, bounds-checked
// element stores (whole tiles, one box per pixel only).
// LB: rows of K per iteration of the main loop (4, or more for the small register blocks:
// see ffma_long_block).
template <int MR, int NR, bool FIXED, bool SPLIT, bool RAGGED = false, int LB = 4>
__global__ void __launch_bounds__(ffma_threads(MR, NR, RAGGED), 1)
ffma_conv_kernel(const __grid_constant__ CUtensorMap map_filt,
                 const __grid_constant__ CUtensorMap map_in,
                 const __grid_constant__ FfmaArgs args) {
  constexpr int Mt = 16 * MR;           // filters per tile
  constexpr int Nt = 16 * NR;           // columns per tile
  constexpr int NH = NR / 4;            // float4 column groups per thread
  constexpr bool INLINE = ffma_inline_producer(MR, NR) && !RAGGED;
  constexpr bool W64 = NR == 16;
  constexpr int kLongBlock = LB;   // rows per iteration of the first loop over a step's rows
  static_assert(LB >= 4 && LB % 2 == 0, "rows per iteration");
  static_assert(!RAGGED || (!FIXED && !SPLIT), "ragged instances");
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
  const uint32_t sk_bar = empty_bar + 8u * stages;   // split tail: "every warp stored its partial sums"

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  long long stamp_cycles = 0;
  uint64_t stamp_ns = 0;
  if (args.clock_stamp != 0 && threadIdx.x == 0) {
    stamp_cycles = clock64();
    stamp_ns = globaltimer_ns();
  }

  if (threadIdx.x == 0) {
    const uint32_t extra = (args.test_missing_arrival != 0 && blockIdx.x == 0) ? 1u : 0u;
    for (int s = 0; s < stages; ++s) {
      // ragged: four copy warps, and the lane that issues bulk filter copies where it can
      mbar_init(full_bar + 8u * s, (RAGGED ? 4 + ((g.No & 3) == 0 ? 1 : 0) : 1) + extra);
      mbar_init(empty_bar + 8u * s, kFfmaConsumerWarps);
    }
    if constexpr (SPLIT) mbar_init(sk_bar, kFfmaConsumerWarps);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  __syncthreads();

  const int rows_full = g.rows;

  if constexpr (RAGGED) {
    if (warp >= kFfmaConsumerWarps) {
      if (threadIdx.x == kFfmaConsumerWarps * 32 && (g.No & 3) == 0) prefetch_tensormap(&map_filt);
      ragged_copy_warp<Mt>(args, warp - kFfmaConsumerWarps, &map_filt, base + a_off, base + b_off,
                           full_bar, empty_bar);
      return;
    }
  } else if constexpr (!INLINE) {
    if (warp == kFfmaConsumerWarps) {
      // ---------------------------------------------------- producer warp
      if (lane == 0) {
        prefetch_tensormap(&map_filt);
        prefetch_tensormap(&map_in);
        FfmaProducer<SPLIT> p;
        p.init(g, Mt);
        bool ok = true;
        while (ok && p.has_work(g))
          ok = p.template issue<true>(args, &map_filt, &map_in, base + a_off, base + b_off, full_bar,
                                      empty_bar, Mt);
        if (!ok) p.drain(g, full_bar);
      }
      return;
    }
  }

  // -------------------------------------------------------------- consumers
  // Producer state of the INLINE variants (registers: kept in shared memory it cost the
  // large blocks 3 %, the loads sitting in the consumers' instruction stream).
  FfmaProducer<SPLIT> prod;
  bool prod_ok = true;
  // The consumer warps take turns at the producer's job, one K step each, so that its
  // instructions are spread over the four schedulers instead of slowing one of them (all
  // the others end up waiting for that one).  Every thread keeps the producer's state and
  // advances it once per K step; only lane 0 of the warp whose turn it is issues the copies.
  int turn = 0;
  if constexpr (INLINE) {
    prod.init(g, Mt);
    if (warp == 0 && lane == 0) {
      prefetch_tensormap(&map_filt);
      prefetch_tensormap(&map_in);
    }
    for (int s = 0; s + 2 < stages && prod.has_work(g); ++s) {
      if (warp == 0) {
        if (lane == 0 && prod_ok)
          prod_ok = prod.template issue<false>(args, &map_filt, &map_in, base + a_off, base + b_off,
                                               full_bar, empty_bar, Mt);
        else
          prod.advance(g, Mt);
        __syncwarp();
      } else {
        prod.advance(g, Mt);
      }
    }
  }

  const int wo = warp >> 1, wn = warp & 1;
  const int to = wo * 4 + (lane >> 3);   // 0..15 along the filter axis
  const int tn = wn * 8 + (lane & 7);    // 0..15 along the column axis
  const int a_elem = (MR % 4 == 0) ? 4 * to : 2 * to;

  // Offset (in floats, inside a stage) of this thread's groups of four columns.  Group h is
  // column 4 tn + 64 h of the tile = (pixel, image) (col / tile_n, col % tile_n); with one box
  // per stage the columns of a row are contiguous, else a pixel's box starts b_slot_bytes
  // after its neighbour's.  (The epilogue recomputes pixel and image from the column.)
  const int used_cols = g.tile_px * g.tile_n;
  uint32_t b_elem[NH];
  // (pixel, image) of each group: kept in registers by the small blocks, recomputed in the
  // epilogue by the large ones, which have no registers to spare
  int col_px[INLINE ? 1 : NH], col_n[INLINE ? 1 : NH];
#pragma unroll
  for (int h = 0; h < NH; ++h) {
    const int col = 4 * tn + 64 * h;
    if constexpr (!INLINE) {
      col_px[h] = col < used_cols ? col / g.tile_n : -1;
      col_n[h] = col < used_cols ? col % g.tile_n : 0;
    }
    if (FIXED)
      b_elem[h] = (uint32_t)col;
    else
      b_elem[h] = col < used_cols
                      ? (uint32_t)((col / g.tile_n) * (g.b_slot_bytes >> 2) + col % g.tile_n) : 0u;
  }
  const int b_pitch = FIXED ? Nt : g.tile_n;   // floats between patch rows

  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;

  // One work item: K steps [s0, s1) of `tile` into fresh accumulators, then what its kind
  // asks for.  The instance with SPLIT = false is the whole-tile one (all K steps, plain
  // epilogue): none of the split tail's code or state is part of it, so the loop that walks
  // whole tiles is compiled exactly as a kernel without a split tail would be.
  auto run_item = [&](const int tile, const int s0, const int s1, const int kind) {
    float2 P[MR / 2][NR / 2], Q[MR / 2][NR / 2];
#pragma unroll
    for (int i = 0; i < MR / 2; ++i)
#pragma unroll
      for (int j = 0; j < NR / 2; ++j) {
        P[i][j] = make_float2(0.f, 0.f);
        Q[i][j] = make_float2(0.f, 0.f);
      }

    Frag<MR, NR> f0, f1;
    ok = mbar_wait(full_bar + 8u * stage, phase, args.wc, kDevTimeoutFull);
    if (!ok) return;
    const float* a_ptr;
    const float* b_ptr[NH];
    auto point_at_stage = [&](int st) {
      a_ptr = reinterpret_cast<const float*>(base_ptr + a_off + (size_t)st * g.a_stage_bytes) + a_elem;
      const float* bs = reinterpret_cast<const float*>(base_ptr + b_off + (size_t)st * g.b_stage_bytes);
#pragma unroll
      for (int h = 0; h < NH; ++h) b_ptr[h] = bs + b_elem[h];
    };
    point_at_stage(stage);
    load_frag<MR, NR, FIXED, W64>(f0, MAXDNN_ROW(0));

    for (int s = s0; s < s1; ++s) {
      if constexpr (INLINE) {
        // Refill the slot this CTA finished two steps ago (every warp has released it
        // by now, so the wait does not hold the issuing warp back) with the K step that is
        // (stages - 2) ahead of the one being consumed.
        if (prod.has_work(g)) {
          if (warp == turn) {
            if (lane == 0 && prod_ok)
              prod_ok = prod.template issue<false>(args, &map_filt, &map_in, base + a_off,
                                                   base + b_off, full_bar, empty_bar, Mt);
            else
              prod.advance(g, Mt);
            __syncwarp();
          } else {
            prod.advance(g, Mt);
          }
        }
        turn = (turn + 1) & 7;
      }
      // f0 holds row 0 of this stage.  Four rows per iteration while the row
      // after the block is still inside the stage.
      const int rows = s < g.short_from ? rows_full : g.rows_short;
      int r = 0;
      if constexpr (kLongBlock > 4) {
        // The small register blocks spend a larger share of their instructions on the
        // loop itself: they take kLongBlock rows per iteration first.
#pragma unroll 1
        for (; r + kLongBlock < rows; r += kLongBlock) {
#pragma unroll
          for (int u = 0; u < kLongBlock; u += 2) {
            load_frag<MR, NR, FIXED, W64>(f1, MAXDNN_ROW(u + 1));
            fma_block<MR, NR>(f0, P, Q);
            load_frag<MR, NR, FIXED, W64>(f0, MAXDNN_ROW(u + 2));
            fma_block<MR, NR>(f1, P, Q);
          }
          a_ptr += kLongBlock * Mt;
#pragma unroll
          for (int h = 0; h < NH; ++h) b_ptr[h] += kLongBlock * b_pitch;
        }
      }
#pragma unroll 1
      for (; r + 4 < rows; r += 4) {
        load_frag<MR, NR, FIXED, W64>(f1, MAXDNN_ROW(1));
        fma_block<MR, NR>(f0, P, Q);
        load_frag<MR, NR, FIXED, W64>(f0, MAXDNN_ROW(2));
        fma_block<MR, NR>(f1, P, Q);
        load_frag<MR, NR, FIXED, W64>(f1, MAXDNN_ROW(3));
        fma_block<MR, NR>(f0, P, Q);
        load_frag<MR, NR, FIXED, W64>(f0, MAXDNN_ROW(4));
        fma_block<MR, NR>(f1, P, Q);
        a_ptr += 4 * Mt;
#pragma unroll
        for (int h = 0; h < NH; ++h) b_ptr[h] += 4 * b_pitch;
      }
#pragma unroll 1
      for (; rows - r > 2; r += 2) {   // 3 or 4 rows left: two of them here
        load_frag<MR, NR, FIXED, W64>(f1, MAXDNN_ROW(1));
        fma_block<MR, NR>(f0, P, Q);
        load_frag<MR, NR, FIXED, W64>(f0, MAXDNN_ROW(2));
        fma_block<MR, NR>(f1, P, Q);
        a_ptr += 2 * Mt;
#pragma unroll
        for (int h = 0; h < NH; ++h) b_ptr[h] += 2 * b_pitch;
      }
      const bool two_left = (rows - r == 2);
      if (two_left) {
        load_frag<MR, NR, FIXED, W64>(f1, MAXDNN_ROW(1));
        fma_block<MR, NR>(f0, P, Q);
      }
      // The last row of this stage is in f1 (two_left) or f0.  Prefetch row 0 of
      // the next stage into the other buffer before computing it.
      const int cur_stage = stage;
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      const bool more = s + 1 < s1;
      if (more) {
        ok = mbar_wait(full_bar + 8u * stage, phase, args.wc, kDevTimeoutFull);
        if (!ok) break;
        point_at_stage(stage);
      }
      if (two_left) {
        if (more) load_frag<MR, NR, FIXED, W64>(f0, MAXDNN_ROW(0));
        fma_block<MR, NR>(f1, P, Q);
      } else {
        if (more) load_frag<MR, NR, FIXED, W64>(f1, MAXDNN_ROW(0));
        fma_block<MR, NR>(f0, P, Q);
        f0 = f1;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar + 8u * cur_stage);
    }
    if (!ok) return;

    if constexpr (SPLIT) {
      // ----------------------------------------------- split tail: partial sums
      // A slot holds a thread's accumulators as float4 {P.x, P.y, Q.x, Q.y}, element
      // [pair index][thread], so that a warp's store of one pair index is one 512-byte run.
      constexpr int kPairs = (MR / 2) * (NR / 2);
      if (kind == kItemContribute) {
        float4* slot = reinterpret_cast<float4*>(args.sk_partial) +
                       (size_t)blockIdx.x * (kPairs * 256) + threadIdx.x;
#pragma unroll
        for (int i = 0; i < MR / 2; ++i)
#pragma unroll
          for (int j = 0; j < NR / 2; ++j)
            __stcg(slot + (i * (NR / 2) + j) * 256,
                   make_float4(P[i][j].x, P[i][j].y, Q[i][j].x, Q[i][j].y));
        __threadfence();
        __syncwarp();
        if (lane == 0) mbar_arrive(sk_bar);
        if (threadIdx.x == 0) {
          // every consumer warp has stored and fenced: publish the slot under this launch's epoch
          if (mbar_wait(sk_bar, 0, args.wc, kDevTimeoutPeer))
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(args.sk_flags + blockIdx.x),
                         "r"(args.wc.epoch) : "memory");
        }
        return;
      }
      if (kind == kItemFinish) {
        // the CTAs below this one whose ranges hold the tile's earlier K steps, in order
        const int grid = (int)gridDim.x;
        const int first_unit = (tile - g.sk_first) * g.n_ksteps;
        int j = (int)(((long long)first_unit * grid) / g.sk_units);
        int u0, u1;
        sk_range(g, j, grid, &u0, &u1);
        while (j > 0 && u0 > first_unit) { --j; sk_range(g, j, grid, &u0, &u1); }
        while (u1 <= first_unit) { ++j; sk_range(g, j, grid, &u0, &u1); }
        for (; j < (int)blockIdx.x && ok; ++j) {
          sk_range(g, j, grid, &u0, &u1);
          if (u1 <= u0) continue;                      // a CTA without a share
          bool ready = true;
          if (lane == 0) ready = wait_peer_flag(args.sk_flags + j, args.wc.epoch, args.wc);
          ready = __shfl_sync(0xffffffffu, ready ? 1 : 0, 0) != 0;
          __syncwarp();          // lane 0's acquire orders the other lanes' reads of the slot
          if (!ready) { ok = false; break; }
          const float4* slot = reinterpret_cast<const float4*>(args.sk_partial) +
                               (size_t)j * (kPairs * 256) + threadIdx.x;
#pragma unroll
          for (int i = 0; i < MR / 2; ++i)
#pragma unroll
            for (int jj = 0; jj < NR / 2; ++jj) {
              const float4 v = __ldcg(slot + (i * (NR / 2) + jj) * 256);
              P[i][jj].x += v.x; P[i][jj].y += v.y; Q[i][jj].x += v.z; Q[i][jj].y += v.w;
              // at most four loads in flight: the accumulators leave no room for more
              if ((jj & 3) == 3) asm volatile("" ::: "memory");
            }
        }
        if (!ok) return;
      }
    }

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
        for (int h = 0; h < NH; ++h) {
          int x, n;
          if constexpr (INLINE) {
            const int col = 4 * tn + 64 * h;
            if (col >= used_cols) continue;
            x = x0 + col / g.tile_n;
            n = n0 + col % g.tile_n;
          } else {
            if (col_px[h] < 0) continue;
            x = x0 + col_px[h];
            n = n0 + col_n[h];
          }
          if (x >= g.Wo || n >= g.Nb) continue;
          float4 v;
          // columns 4h .. 4h+3 of this row: j = 2*j2 + jb with j2 = 2h, 2h+1
          v.x = ia == 0 ? P[i2][2 * h].x : Q[i2][2 * h].y;
          v.y = ia == 0 ? Q[i2][2 * h].x : P[i2][2 * h].y;
          v.z = ia == 0 ? P[i2][2 * h + 1].x : Q[i2][2 * h + 1].y;
          v.w = ia == 0 ? Q[i2][2 * h + 1].x : P[i2][2 * h + 1].y;
          v.x *= alpha; v.y *= alpha; v.z *= alpha; v.w *= alpha;
          float* dst = args.out + (((size_t)o * g.Ho + y) * g.Wo + x) * (size_t)g.Nb + n;
          if constexpr (RAGGED) {       // rows of Nb floats start anywhere: element stores
            __stcs(dst, v.x);
            if (n + 1 < g.Nb) __stcs(dst + 1, v.y);
            if (n + 2 < g.Nb) __stcs(dst + 2, v.z);
            if (n + 3 < g.Nb) __stcs(dst + 3, v.w);
          } else {
            __stcs(reinterpret_cast<float4*>(dst), v);
          }
        }
      }
    }
  };

  if constexpr (SPLIT) {
    FfmaItem item;
    for (int k = 0; ok && ffma_item(g, k, item); ++k)
      run_item(item.tile, item.s0, item.s1, item.kind);
  } else {
    const int n_ksteps = g.n_ksteps;
    for (int tile = g.tile_begin + blockIdx.x; tile < g.tile_end && ok; tile += gridDim.x)
      run_item(tile, 0, n_ksteps, (int)kItemWhole);
  }

  if constexpr (INLINE) {
    if (lane == 0 && !(ok && prod_ok)) prod.drain(g, full_bar);
  }
  if (args.clock_stamp != 0 && threadIdx.x == 0 && args.wc.status) {
    atomicMax(args.wc.status + (SPLIT ? 4 : 2), (uint32_t)(clock64() - stamp_cycles));
    atomicMax(args.wc.status + (SPLIT ? 5 : 3), (uint32_t)(globaltimer_ns() - stamp_ns));
  }
}
#undef MAXDNN_ROW

}  // namespace maxdnn
