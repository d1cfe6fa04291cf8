// Filter gradient on the tensor cores (tcgen05 MMA, fp32 accumulators in TMEM), TF32 or
// BF16 operands — ONE kernel template for one-SM and two-SM tiles and for the reduction kept
// in one accumulator or added up in chunks: the GEMM
//     D[o][k] = sum_r dout[o][r] * patch[k][r],   r = (y, x, n),   dfilt[k][o] = alpha D[o][k]
// with both operands K-major — the reduction index is the contiguous one: a reduction
// step is the 128 bytes of images (32 fp32 / 64 bf16) of one output pixel, which a bulk
// tensor copy lands as rows of 128 bytes with the 128-byte swizzle, the canonical K-major
// operand layout.  A = 128 filters x 128 B, B = up to 256 gradient rows x 128 B (bc
// channels x bh filter rows x Sk filter columns: one box of a bh x Sk window of input
// pixels), four MMAs of 32 bytes of K per step.
//
// Warp 0: copies (one elected lane).  Warp 1: MMA issue and TMEM.  Warps 2..: epilogue
// (TMEM -> registers -> global; a thread holds one filter, so each stored row of 32
// filters is one 128-byte line), which drains one accumulator while the MMA warp fills
// the other; where a gradient row goes in dfilt comes from a table in shared memory
// built once per CTA (the index arithmetic per element would otherwise cost more than
// the reduction of a split).  The reduction is split over CTAs as in the fp32 kernel;
// partial sums are added in a fixed order by wgrad_reduce_kernel.  Every wait is bounded.
//
// PAIR (tcgen05 cta_group::2): a cluster of two CTAs works on a tile of 256 filters x up to
// 256 gradient rows.  CTA r stages its 128 filters of the output gradient and the gradient
// rows of HALF of the tile's channels; the leader issues MMAs of M = 256 that read each half
// of the row operand from the CTA that holds it.  Per SM and per MMA 8 KB instead of 12 KB
// are staged — the one-SM tile is bound by that fill rate — and the ring holds six stages of
// 32 KB.  Synchronisation as in the two-SM forward kernel: both CTAs' copies complete on the
// leader's "full" barrier, on which only the leader arrives (expecting both CTAs' bytes);
// the leader's commits reach the "empty" / "accumulator complete" barriers of both CTAs; both
// CTAs' epilogue warps arrive on the leader's "accumulator drained" barrier.
//
// CHUNK (TF32 only; behind maxdnn_conv_bprop_filter_tf32x3): the tensor core truncates its
// fp32 accumulator at every MMA, so the MMA warp starts a fresh TMEM accumulator every
// chunk_steps reduction steps and EIGHT epilogue warps (two per TMEM lane quarter, for the
// tile's gradient rows 0-127 and 128-255) add the chunks in registers with round-to-nearest
// adds; after an item's last chunk the totals are stored through the row table.  The three
// TF32 products of that entry point are one reduction over three times the images: three
// passes over tensors stored [hi | lo] along the image axis, which the copy warp addresses.
#pragma once
#include "bprop.cuh"
#include "umma_util.cuh"

namespace maxdnn {

// warps: copies, MMA, then 4 (plain) or 8 (chunked) epilogue warps
__host__ __device__ constexpr int wgrad_umma_threads(bool chunk) { return (2 + (chunk ? 8 : 4)) * 32; }
constexpr uint32_t kWgUmmaABytes = 128 * 128;      // 128 filters x 128 B
constexpr uint32_t kWgUmmaBBytes = 256 * 128;      // up to 256 gradient rows x 128 B (two-SM: half per CTA)

struct WgradUmmaArgs {
  WgradGeom g;            // rows <= 256; n_chunks counts groups of `atom` images
  uint32_t idesc;
  uint32_t atom;          // images per reduction step: 32 (tf32) or 64 (bf16)
  uint32_t chunk_steps;   // chunked kernel only: reduction steps per TMEM accumulator
  uint32_t x3_per_part;   // chunked kernel only: reduction steps (groups of 32 images) per product part
  float* dfilt;
  float* partial;
  WaitCtx wc;          // status block and this launch's epoch (see ptx_util.cuh)
};

// What the epilogue roles need from the kernel's set-up.
struct WgradCtx {
  const int2* row_tab;    // accumulator column -> {dfilt row offset in the tile; channel << 16 | filter row}
  uint32_t accf_bar, acce_bar, leader_acce, tmem_base, rank;
  int unit, n_units;      // this CTA's (pair's) first item and the item stride
};

// Where the tile of `cc` starts in dfilt (or in this split's partial sums) for filter `o`.
__device__ __forceinline__ float* wgrad_tile_dst(const WgradUmmaArgs& args, const WgradCursor& cc, int o) {
  const WgradGeom& g = args.g;
  const size_t K = (size_t)g.Nc * g.Skh * g.Skw;
  return (g.splits == 1 ? args.dfilt : args.partial + (size_t)cc.split * K * g.No) +
         ((size_t)(cc.cb * g.bc) * g.Skh + (size_t)cc.khb * g.bh) * g.Skw * g.No + o;
}

// Epilogue of the plain kernel (warps 2-5): 32 accumulator columns at a time to global memory.
template <bool PAIR>
__device__ __forceinline__ void wgrad_epilogue_plain(const WgradUmmaArgs& args, const WgradCtx& cx,
                                                     int warp, int lane) {
  const WgradGeom& g = args.g;
  const int q = warp & 3;                      // TMEM lane quarter this warp may read
  const int n_live = PAIR ? g.n_mma : g.rows;  // accumulator columns in use
  WgradCursor cc;
  cc.start(g, cx.unit);
  uint32_t it = 0;
  bool ok = true;
  const float scale = g.splits == 1 ? g.alpha : 1.0f;
  while (ok && !cc.done(g)) {
    const uint32_t acc = it & 1u;
    if (!mbar_wait(cx.accf_bar + 8u * acc, (it >> 1) & 1u, args.wc, kDevTimeoutAccum)) {
      ok = false;
      break;
    }
    tcgen05_fence_after();
    const int o = cc.ob * (PAIR ? 256 : 128) + (int)cx.rank * 128 + q * 32 + lane;
    const int c_lim = g.Nc - cc.cb * g.bc;          // channels / filter rows of this tile
    const int h_lim = g.Skh - cc.khb * g.bh;         // that exist
    float* dst = wgrad_tile_dst(args, cc, o);
    const uint32_t t_row = cx.tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256u;
    for (int col = 0; col < n_live; col += 32) {
      uint32_t v[32];
      tmem_ld_32x32(t_row + (uint32_t)col, v);
      tmem_wait_ld();
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const int2 e = cx.row_tab[col + j];
        if (col + j < n_live && (e.y >> 16) < c_lim && (e.y & 0xffff) < h_lim && o < g.No)
          dst[(size_t)e.x * g.No] = __uint_as_float(v[j]) * scale;
      }
    }
    tcgen05_fence_before();
    __syncwarp();
    if (lane == 0) {
      if constexpr (PAIR) mbar_arrive_cluster(cx.leader_acce + 8u * acc);
      else mbar_arrive(cx.acce_bar + 8u * acc);
    }
    cc.start(g, cc.item + cx.n_units);
    ++it;
  }
}

// Epilogue of the chunked kernel (warps 2-9), out of line (128 totals per thread).
template <bool PAIR>
__device__ __noinline__ void wgrad_epilogue_chunk(const WgradUmmaArgs& args, const WgradCtx cx,
                                                  int warp, int lane) {
  const WgradGeom& g = args.g;
  const int q = warp & 3;                      // TMEM lane quarter this warp may read
  const int half = (warp - 2) >> 2;            // accumulator columns [128 half, 128 half + 128)
  const int n_live = PAIR ? g.n_mma : g.rows;
  const int chunk_steps = (int)args.chunk_steps;
  WgradCursor cc;
  cc.start(g, cx.unit);
  uint32_t chunk = 0;
  bool ok = true;
  const float scale = g.splits == 1 ? g.alpha : 1.0f;
  while (ok && !cc.done(g)) {
    const int n_steps = cc.r_end - cc.r;
    const int n_chunks = (n_steps + chunk_steps - 1) / chunk_steps;
    float tot[128];
    for (int c = 0; c < n_chunks && ok; ++c, ++chunk) {
      const uint32_t acc = chunk & 1u;
      if (!mbar_wait(cx.accf_bar + 8u * acc, (chunk >> 1) & 1u, args.wc, kDevTimeoutAccum)) {
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const uint32_t t_row = cx.tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256u + (uint32_t)(half * 128);
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (half * 128 + 16 * k >= n_live) continue;          // warp-uniform
        uint32_t v[16];
        tmem_ld_32x16(t_row + (uint32_t)(16 * k), v);
        tmem_wait_ld();
        if (c == 0) {
#pragma unroll
          for (int j = 0; j < 16; ++j) tot[16 * k + j] = __uint_as_float(v[j]);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) tot[16 * k + j] += __uint_as_float(v[j]);   // round to nearest
        }
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) {
        if constexpr (PAIR) mbar_arrive_cluster(cx.leader_acce + 8u * acc);
        else mbar_arrive(cx.acce_bar + 8u * acc);
      }
    }
    if (!ok) break;
    const int o = cc.ob * (PAIR ? 256 : 128) + (int)cx.rank * 128 + q * 32 + lane;
    const int c_lim = g.Nc - cc.cb * g.bc;
    const int h_lim = g.Skh - cc.khb * g.bh;
    float* dst = wgrad_tile_dst(args, cc, o);
#pragma unroll
    for (int j = 0; j < 128; ++j) {
      const int col = half * 128 + j;
      const int2 e = cx.row_tab[col];
      if (col < n_live && (e.y >> 16) < c_lim && (e.y & 0xffff) < h_lim && o < g.No)
        dst[(size_t)e.x * g.No] = tot[j] * scale;
    }
    cc.start(g, cc.item + cx.n_units);
  }
}

template <bool BF16, bool PAIR, bool CHUNK>
__global__ void __launch_bounds__(wgrad_umma_threads(CHUNK), 1)
wgrad_umma_kernel(const __grid_constant__ CUtensorMap map_dout,
                  const __grid_constant__ CUtensorMap map_in,
                  const __grid_constant__ WgradUmmaArgs args) {
  static_assert(!(CHUNK && BF16), "the chunked sum exists for TF32 operands only");
  constexpr int kEpiWarps = CHUNK ? 8 : 4;
  constexpr int kThreads = wgrad_umma_threads(CHUNK);
  extern __shared__ uint8_t smem_raw[];
  const WgradGeom& g = args.g;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int stages = g.stages;
  const uint32_t stage_bytes = kWgUmmaABytes + (PAIR ? kWgUmmaBBytes / 2 : kWgUmmaBBytes);
  const uint32_t bar_off = (uint32_t)stages * stage_bytes;
  const uint32_t full_bar = base + bar_off;             // two-SM: the leader's are used
  const uint32_t empty_bar = full_bar + 8u * stages;
  const uint32_t accf_bar = empty_bar + 8u * stages;    // 2: accumulator complete
  const uint32_t acce_bar = accf_bar + 16u;             // 2: accumulator drained (two-SM: the leader's)
  const uint32_t done_bar = acce_bar + 16u;
  const uint32_t tmem_slot = done_bar + 8u;
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(base_ptr + bar_off + 16u * stages + 40u);
  int2* row_tab = reinterpret_cast<int2*>(base_ptr + bar_off + 1024u);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar + 8u * s, 1);     // the (leader's) copy warp (two-SM: expects both CTAs' bytes)
      mbar_init(empty_bar + 8u * s, 1);    // the (leader's) commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar + 8u * a, 1);
      mbar_init(acce_bar + 8u * a, kEpiWarps * (PAIR ? 2 : 1));   // the epilogue warps (of both CTAs)
    }
    mbar_init(done_bar, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) tmem_alloc_all<PAIR>(tmem_slot);
  // accumulator column -> {dfilt row offset relative to the tile's first row; channel << 16 |
  // filter row}; two-SM: the second half of the columns are the peer's channels
  {
    const int hcols = PAIR ? g.n_mma >> 1 : 256;
    const int rows_cta = PAIR ? g.rows_h : 256;
    for (int col = threadIdx.x; col < 256; col += kThreads) {
      const int half = col >= hcols ? 1 : 0;
      const int row = col - half * hcols;
      if (row < rows_cta) {
        const int w_l = row % g.bw;
        const int t = row / g.bw;
        const int h_l = t % g.bh;
        const int c_l = half * g.bc_h + t / g.bh;
        row_tab[col] = make_int2((c_l * g.Skh + h_l) * g.Skw + w_l, (c_l << 16) | h_l);
      } else {
        row_tab[col] = make_int2(0, 0x7fff << 16);             // no such row: never stored
      }
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if constexpr (PAIR) {
    cluster_arrive();
    cluster_wait();
  }
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  const uint32_t leader_full = PAIR ? map_to_cta(full_bar, 0) : full_bar;
  const uint32_t leader_acce = PAIR ? map_to_cta(acce_bar, 0) : acce_bar;

  if (warp == 0) {
    // ------------------------------------------------------------- copies
    if (lane == 0) {
      prefetch_tensormap(&map_dout);
      prefetch_tensormap(&map_in);
    }
    const uint32_t tx_bytes = (PAIR ? 2u : 1u) * (uint32_t)(g.box_o + (PAIR ? g.rows_h : g.rows)) * 128u;
    const uint64_t pol_last = l2_policy_evict_last();
    WgradCursor pc;
    pc.start(g, unit);
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    while (ok && !pc.done(g)) {
      if (!mbar_wait(empty_bar + 8u * stage, phase ^ 1u, args.wc, kDevTimeoutEmpty)) {
        ok = false;
        break;
      }
      const uint32_t fb = leader_full + 8u * stage;
      const uint32_t dst = base + (uint32_t)stage * stage_bytes;
      int n_g = pc.nc * (int)args.atom, n_x = n_g;       // first image of the step in dout / in
      if constexpr (CHUNK) {
        // the three products one after another along the image axis: hi x hi, hi x lo, lo x hi
        // of tensors stored [hi | lo]
        const int per = (int)args.x3_per_part;
        const int part = pc.nc / per;
        const int within = pc.nc - part * per;
        n_g = ((part == 2 ? per : 0) + within) * (int)args.atom;
        n_x = ((part == 1 ? per : 0) + within) * (int)args.atom;
      }
      const int o0 = pc.ob * (PAIR ? 256 : 128) + (int)rank * 128;
      const int c0 = pc.cb * g.bc + (PAIR ? (int)rank * g.bc_h : 0);
      const int w0 = pc.x * g.stride_w - g.pad_w, h0 = pc.y * g.stride_h - g.pad_h + pc.khb * g.bh;
      if (elect_one()) {
        if (rank == 0) mbar_arrive_expect_tx(full_bar + 8u * stage, tx_bytes);
        if constexpr (PAIR) {
          tma_load_4d_pair(dst, &map_dout, fb, n_g, pc.x, pc.y, o0, pol_last);
          tma_load_4d_pair(dst + kWgUmmaABytes, &map_in, fb, n_x, w0, h0, c0, pol_last);
        } else {
          tma_load_4d_hint(dst, &map_dout, fb, n_g, pc.x, pc.y, o0, pol_last);
          tma_load_4d_hint(dst + kWgUmmaABytes, &map_in, fb, n_x, w0, h0, c0, pol_last);
        }
      }
      __syncwarp();
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      pc.advance(g, n_units);
    }
    if (!ok) {
      // Leaving early: give copies already issued time to land.
      if constexpr (PAIR) {
        // (their barrier lives in the leader CTA and cannot be polled from the peer)
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) {}
      } else {
        for (int s = 0; s < stages; ++s) {
          const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
          mbar_wait_grace(full_bar + 8u * s, par);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issue (two-SM: leader only)
    if (rank == 0) {
      WgradCursor cc;
      cc.start(g, unit);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t chunk = 0;     // accumulators started so far: this one is chunk & 1
      bool ok = true;
      // K-major operands, 128-byte swizzle: rows of 128 B, groups of 8 rows 1024 B apart;
      // the next 32 bytes of K are the next 32 bytes of every row (start address + 32).
      const uint64_t desc_hi = make_smem_desc(0, 0, 1024, 2u);
      while (ok && !cc.done(g)) {
        const int n_steps = cc.r_end - cc.r;
        const int chunk_steps = CHUNK ? (int)args.chunk_steps : n_steps;   // plain: one per item
        for (int s0 = 0; s0 < n_steps && ok; s0 += chunk_steps, ++chunk) {
          // the epilogue has drained this accumulator (used two chunks ago)
          const uint32_t acc = chunk & 1u;
          if (!mbar_wait(acce_bar + 8u * acc, ((chunk >> 1) & 1u) ^ 1u, args.wc, kDevTimeoutAccFree)) {
            ok = false;
            break;
          }
          tcgen05_fence_after();
          const uint32_t d_tmem = tmem_base + acc * 256u;
          const int s1 = s0 + chunk_steps < n_steps ? s0 + chunk_steps : n_steps;
          uint32_t accumulate = 0;
          for (int s = s0; s < s1; ++s) {
            if (!mbar_wait(full_bar + 8u * stage, phase, args.wc, kDevTimeoutFull)) {
              ok = false;
              break;
            }
            tcgen05_fence_after();
            const uint32_t a_addr = base + (uint32_t)stage * stage_bytes;
            const uint64_t adesc0 = desc_hi | (uint64_t)((a_addr & 0x3FFFFu) >> 4);
            const uint64_t bdesc0 = desc_hi | (uint64_t)(((a_addr + kWgUmmaABytes) & 0x3FFFFu) >> 4);
            if (elect_one()) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                if constexpr (PAIR)
                  tcgen05_mma_pair<BF16>(d_tmem, adesc0 + (uint64_t)(2 * j), bdesc0 + (uint64_t)(2 * j),
                                         args.idesc, accumulate | (uint32_t)(j > 0));
                else
                  tcgen05_mma<BF16>(d_tmem, adesc0 + (uint64_t)(2 * j), bdesc0 + (uint64_t)(2 * j),
                                    args.idesc, accumulate | (uint32_t)(j > 0));
              }
              if constexpr (PAIR) tcgen05_commit_pair(empty_bar + 8u * stage);   // frees the stage in both CTAs
              else tcgen05_commit(empty_bar + 8u * stage);
            }
            accumulate = 1;
            __syncwarp();
            if (++stage == stages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          if (elect_one()) {
            if constexpr (PAIR) tcgen05_commit_pair(accf_bar + 8u * acc);
            else tcgen05_commit(accf_bar + 8u * acc);
          }
          __syncwarp();
        }
        if (!ok) break;
        cc.start(g, cc.item + n_units);
      }
      if (elect_one()) {
        if constexpr (PAIR) tcgen05_commit_pair(done_bar, 1);
        else tcgen05_commit(done_bar);
      }
      mbar_wait(done_bar, 0, args.wc, kDevTimeoutDrain);
    }
  } else {
    // ------------------------------------------------------------ epilogue (two-SM: both CTAs)
    WgradCtx cx;
    cx.row_tab = row_tab; cx.accf_bar = accf_bar; cx.acce_bar = acce_bar; cx.leader_acce = leader_acce;
    cx.tmem_base = tmem_base; cx.rank = rank; cx.unit = unit; cx.n_units = n_units;
    if constexpr (CHUNK) wgrad_epilogue_chunk<PAIR>(args, cx, warp, lane);
    else wgrad_epilogue_plain<PAIR>(args, cx, warp, lane);
  }

  // Two-SM: neither CTA leaves (or frees TMEM) while its peer may still arrive on its
  // barriers, have copies in flight that report to it, or run MMAs that read its shared memory.
  tcgen05_fence_before();
  __syncthreads();
  if constexpr (PAIR) {
    cluster_arrive();
    cluster_wait();
  }
  if (warp == 1) {
    tcgen05_fence_after();
    tmem_dealloc_all<PAIR>(tmem_base);
  }
}

}  // namespace maxdnn
