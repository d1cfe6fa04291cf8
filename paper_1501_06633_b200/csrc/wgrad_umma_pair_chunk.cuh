// Two-SM form of the chunked TF32 filter-gradient kernel (see wgrad_umma_chunk.cuh for the
// chunks and the three products, wgrad_umma_pair.cuh for the two-SM tile): the leader's MMA
// warp starts a fresh accumulator in both CTAs' TMEM every chunk_steps reduction steps, the
// eight epilogue warps of each CTA add the chunks of their 128 filters in registers.
#pragma once
#include "wgrad_umma_chunk.cuh"
#include "wgrad_umma_pair.cuh"

namespace maxdnn {

// Epilogue warps (2-9 of each CTA) of the two-SM chunked filter-gradient kernel, out of line
// like wgrad_chunk_epilogue_role; a CTA drains its own 128 filters.
__device__ __noinline__ void wgrad_pair_chunk_epilogue_role(const WgradUmmaArgs& args, const int2* row_tab,
                                                            uint32_t accf_bar, uint32_t leader_acce,
                                                            uint32_t tmem_base, int warp, int lane,
                                                            uint32_t rank, int pair, int n_pairs) {
  const WgradGeom& g = args.g;
  const int q = warp & 3;
  const int half = (warp - 2) >> 2;            // accumulator columns [128 half, 128 half + 128)
  const int chunk_steps = (int)args.chunk_steps;
  WgradCursor cc;
  cc.start(g, pair);
  uint32_t chunk = 0;
  bool ok = true;
  const bool direct = (g.splits == 1);
  const size_t K = (size_t)g.Nc * g.Skh * g.Skw;
  const float scale = direct ? g.alpha : 1.0f;
  while (ok && !cc.done(g)) {
    const int n_steps = cc.r_end - cc.r;
    const int n_chunks = (n_steps + chunk_steps - 1) / chunk_steps;
    float tot[128];
    for (int c = 0; c < n_chunks && ok; ++c, ++chunk) {
      const uint32_t acc = chunk & 1u;
      if (!mbar_wait(accf_bar + 8u * acc, (chunk >> 1) & 1u, args.wc, kDevTimeoutAccum)) {
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256u + (uint32_t)(half * 128);
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (half * 128 + 16 * k >= g.n_mma) continue;          // warp-uniform
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
      if (lane == 0) mbar_arrive_cluster(leader_acce + 8u * acc);
    }
    if (!ok) break;
    const int o = cc.ob * 256 + (int)rank * 128 + q * 32 + lane;
    const int c_lim = g.Nc - cc.cb * g.bc;
    const int h_lim = g.Skh - cc.khb * g.bh;
    float* dst = (direct ? args.dfilt : args.partial + (size_t)cc.split * K * g.No) +
                 ((size_t)(cc.cb * g.bc) * g.Skh + (size_t)cc.khb * g.bh) * g.Skw * g.No + o;
#pragma unroll
    for (int j = 0; j < 128; ++j) {
      const int col = half * 128 + j;
      const int2 e = row_tab[col];
      if (col < g.n_mma && (e.y >> 16) < c_lim && (e.y & 0xffff) < h_lim && o < g.No)
        dst[(size_t)e.x * g.No] = tot[j] * scale;
    }
    cc.start(g, cc.item + n_pairs);
  }
}

__global__ void __launch_bounds__(kWgChunkThreads, 1)
wgrad_umma_pair_chunk_kernel(const __grid_constant__ CUtensorMap map_dout,
                             const __grid_constant__ CUtensorMap map_in,
                             const __grid_constant__ WgradUmmaArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const WgradGeom& g = args.g;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int stages = g.stages;
  const uint32_t half_b_bytes = 128u * 128u;                 // up to 128 gradient rows per CTA
  const uint32_t stage_bytes = kWgUmmaABytes + half_b_bytes;
  const uint32_t bar_off = (uint32_t)stages * stage_bytes;
  const uint32_t full_bar = base + bar_off;                  // the leader's are used
  const uint32_t empty_bar = full_bar + 8u * stages;
  const uint32_t accf_bar = empty_bar + 8u * stages;         // 2
  const uint32_t acce_bar = accf_bar + 16u;                  // 2; the leader's are used
  const uint32_t done_bar = acce_bar + 16u;
  const uint32_t tmem_slot = done_bar + 8u;
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(base_ptr + bar_off + 16u * stages + 40u);
  int2* row_tab = reinterpret_cast<int2*>(base_ptr + bar_off + 1024u);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;
  const int hcols = g.n_mma >> 1;                            // accumulator columns per half

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar + 8u * s, 1);     // the leader's copy warp (expects both CTAs' bytes)
      mbar_init(empty_bar + 8u * s, 1);    // the leader's commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar + 8u * a, 1);     // the leader's commit
      mbar_init(acce_bar + 8u * a, 16);    // eight epilogue warps in each of the two CTAs
    }
    mbar_init(done_bar, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot),
                 "r"(kWgUmmaTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  // accumulator column -> {dfilt row offset relative to the tile's first row; channel << 16 | filter row}
  for (int col = threadIdx.x; col < 256; col += kWgChunkThreads) {
    const int half = col >= hcols ? 1 : 0;
    const int row = col - half * hcols;
    if (row < g.rows_h) {
      const int w_l = row % g.bw;
      const int t = row / g.bw;
      const int h_l = t % g.bh;
      const int c_l = half * g.bc_h + t / g.bh;
      row_tab[col] = make_int2((c_l * g.Skh + h_l) * g.Skw + w_l, (c_l << 16) | h_l);
    } else {
      row_tab[col] = make_int2(0, 0x7fff << 16);             // no such row: never stored
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  const uint32_t leader_full = map_to_cta(full_bar, 0);
  const uint32_t leader_acce = map_to_cta(acce_bar, 0);

  if (warp == 0) {
    // ------------------------------------------------------------- copies
    if (lane == 0) {
      prefetch_tensormap(&map_dout);
      prefetch_tensormap(&map_in);
    }
    const uint32_t tx_bytes = 2u * (uint32_t)(g.box_o + g.rows_h) * 128u;   // both CTAs' boxes
    const uint64_t pol_last = l2_policy_evict_last();
    WgradCursor pc;
    pc.start(g, pair);
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
      // the three products one after another along the image axis (see wgrad_umma_chunk_kernel)
      const int per = (int)args.x3_per_part;
      const int part = pc.nc / per;
      const int within = pc.nc - part * per;
      const int n_g = ((part == 2 ? per : 0) + within) * (int)args.atom;
      const int n_x = ((part == 1 ? per : 0) + within) * (int)args.atom;
      if (elect_one()) {
        if (rank == 0) mbar_arrive_expect_tx(full_bar + 8u * stage, tx_bytes);
        tma_load_4d_pair(dst, &map_dout, fb, n_g, pc.x, pc.y, pc.ob * 256 + (int)rank * 128, pol_last);
        tma_load_4d_pair(dst + kWgUmmaABytes, &map_in, fb, n_x, pc.x * g.stride_w - g.pad_w,
                         pc.y * g.stride_h - g.pad_h + pc.khb * g.bh,
                         pc.cb * g.bc + (int)rank * g.bc_h, pol_last);
      }
      __syncwarp();
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      pc.advance(g, n_pairs);
    }
    if (!ok) {
      // Leaving early: give copies already issued time to land (their barrier lives in
      // the leader CTA and cannot be polled from the peer).
      const uint64_t t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ull) {}
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issue (leader only)
    if (rank == 0) {
      WgradCursor cc;
      cc.start(g, pair);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t chunk = 0;     // chunks started so far: accumulator chunk & 1
      const int chunk_steps = (int)args.chunk_steps;
      bool ok = true;
      const uint64_t desc_hi = make_smem_desc(0, 0, 1024, 2u);
      while (ok && !cc.done(g)) {
        const int n_steps = cc.r_end - cc.r;
        for (int s0 = 0; s0 < n_steps && ok; s0 += chunk_steps, ++chunk) {
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
                tcgen05_mma_pair<false>(d_tmem, adesc0 + (uint64_t)(2 * j), bdesc0 + (uint64_t)(2 * j),
                                        args.idesc, accumulate | (uint32_t)(j > 0));
              }
              tcgen05_commit_pair(empty_bar + 8u * stage);       // frees the stage in both CTAs
            }
            accumulate = 1;
            __syncwarp();
            if (++stage == stages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          if (elect_one()) tcgen05_commit_pair(accf_bar + 8u * acc);
          __syncwarp();
        }
        if (!ok) break;
        cc.start(g, cc.item + n_pairs);
      }
      if (elect_one()) tcgen05_commit_pair(done_bar, 1);
      mbar_wait(done_bar, 0, args.wc, kDevTimeoutDrain);
    }
  } else {
    // ------------------------------------------------------------ epilogue (both CTAs)
    wgrad_pair_chunk_epilogue_role(args, row_tab, accf_bar, leader_acce, tmem_base, warp, lane, rank,
                                   pair, n_pairs);
  }

  // Neither CTA leaves (or frees TMEM) while its peer may still arrive on its barriers,
  // have copies in flight that report to it, or run MMAs that read its shared memory.
  tcgen05_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(kWgUmmaTmemCols)
                 : "memory");
  }
}

}  // namespace maxdnn
