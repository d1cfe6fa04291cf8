// Two-SM variant of the chunked TF32 FPROP kernel (see umma_chunk_conv.cuh for why K is
// summed in chunks, and umma_pair_conv.cuh for the two-SM tile): 256 filters per CTA pair,
// the leader's MMA warp starts a fresh accumulator (in both CTAs' TMEM) every chunk_steps
// K steps, and the eight epilogue warps of EACH CTA add the chunks of their 128 filters in
// registers.  Warp 0: patch copies, warp 1: MMA issue (leader), warp 2: filter copies,
// warps 3-10: epilogue.
#pragma once
#include "umma_chunk_conv.cuh"
#include "umma_pair_conv.cuh"

namespace maxdnn {

// Epilogue warps (3-10 of each CTA) of the two-SM chunked kernel, out of line like
// chunk_epilogue_role.  A CTA drains its own 128 filters (its TMEM) of every chunk; the
// two warps of a lane quarter take the tile's columns 0-127 and 128-255.
__device__ __noinline__ void pair_chunk_epilogue_role(const CUtensorMap& map_out, const UmmaArgs& args,
                                                      uint32_t base, uint8_t* base_ptr, uint32_t st_off,
                                                      uint32_t accf_bar, uint32_t leader_acce,
                                                      uint32_t tmem_base, int warp, int lane,
                                                      uint32_t rank, int pair, int n_pairs) {
  const ConvGeom& g = args.g;
  const int n_ksteps = g.n_ksteps;
  const int n_cols = g.tile_px * g.tile_n;   // MMA N (both halves)
  const int half_cols = n_cols >> 1;         // columns whose patches each CTA stages
  const int q = warp & 3;
  const int half = (warp - 3) >> 2;
  const int ew = warp - 3;                   // 0..7: one staging tile each
  const uint32_t stg = base + st_off + (uint32_t)ew * kStageTileBytes;
  uint8_t* stg_ptr = base_ptr + st_off + (size_t)ew * kStageTileBytes;
  const float alpha = g.alpha;
  const uint64_t pol_first = l2_policy_evict_first();
  const int chunk_steps = (int)args.chunk_steps;
  const int chunks_per_tile = (n_ksteps + chunk_steps - 1) / chunk_steps;
  bool ok = true;
  uint32_t chunk = 0;
  for (int tile = pair; tile < g.n_tiles && ok; tile += n_pairs) {
    int r = tile;
    const int ob = r % g.o_blocks; r /= g.o_blocks;
    const int nch = r % g.n_chunks; r /= g.n_chunks;
    const int xr = r % g.x_runs;
    const int y = r / g.x_runs;
    const int o0 = ob * 2 * kUmmaM + (int)rank * kUmmaM + q * 32;
    const int n0 = nch * g.tile_n;
    const int x0 = xr * g.tile_px;
    // image and pixel of a group of 32 columns: columns [0, half_cols) were staged by
    // the leader, the rest by its peer
    auto col_n = [&](int col) {
      const int hr = col >= half_cols ? 1 : 0;
      const int cl = col - hr * half_cols;
      const int pl = cl / g.cta_n;
      return n0 + (g.split_n ? hr * g.cta_n : 0) + (cl - pl * g.cta_n);
    };
    auto col_x = [&](int col) {
      const int hr = col >= half_cols ? 1 : 0;
      const int cl = col - hr * half_cols;
      return x0 + (g.split_n ? 0 : hr * g.cta_px) + cl / g.cta_n;
    };
    uint32_t live = 0;       // warp-uniform bit mask over this warp's four groups
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int col = half * 128 + 32 * k;
      if ((col < n_cols) && (col_x(col) < g.Wo) && (col_n(col) < g.Nb) && (o0 < g.No)) live |= 1u << k;
    }
    float tot[128];
    for (int c = 0; c < chunks_per_tile && ok; ++c, ++chunk) {
      const uint32_t acc = chunk & 1u;
      if (!mbar_wait(accf_bar + 8u * acc, (chunk >> 1) & 1u, args.wc, kDevTimeoutAccum)) {
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * kAccCols +
                             (uint32_t)(half * 128);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (!((live >> k) & 1u)) continue;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t v[16];
          tmem_ld_32x16(t_row + (uint32_t)(32 * k + 16 * hh), v);
          tmem_wait_ld();
          if (c == 0) {
#pragma unroll
            for (int j = 0; j < 16; ++j) tot[32 * k + 16 * hh + j] = __uint_as_float(v[j]);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) tot[32 * k + 16 * hh + j] += __uint_as_float(v[j]);   // round to nearest
          }
        }
      }
      // this accumulator may be overwritten by the chunk after next: tell the leader's MMA warp
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_acce + 8u * acc);
    }
    if (!ok) break;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (!((live >> k) & 1u)) continue;
      if (lane == 0) bulk_wait_read<0>();      // the staging tile has been read by the previous store
      __syncwarp();
      uint8_t* row = stg_ptr + (size_t)lane * 128;
#pragma unroll
      for (int cc = 0; cc < 8; ++cc) {
        float4 o4;
        o4.x = tot[32 * k + 4 * cc + 0] * alpha;
        o4.y = tot[32 * k + 4 * cc + 1] * alpha;
        o4.z = tot[32 * k + 4 * cc + 2] * alpha;
        o4.w = tot[32 * k + 4 * cc + 3] * alpha;
        *reinterpret_cast<float4*>(row + ((cc ^ (lane & 7)) << 4)) = o4;
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        const int col = half * 128 + 32 * k;
        tma_store_4d_hint(&map_out, stg, col_n(col), col_x(col), y, o0, pol_first);
        bulk_commit();
      }
    }
  }
  if (lane == 0) bulk_wait_all();
}

// Geometry fields used here: tile_m = 256 (filters per pair tile), tile_px = pixels per
// pair tile (even), b_box_w = pixels of ONE CTA's strip, b_stage_bytes = ONE CTA's patch
// bytes per stage; args.tap_b_bytes / lbo_* describe the per-CTA staged layout.
__global__ void __launch_bounds__(kUmmaChunkThreads, 1)
umma_pair_chunk_conv_kernel(const __grid_constant__ CUtensorMap map_filt,
                            const __grid_constant__ CUtensorMap map_in,
                            const __grid_constant__ CUtensorMap map_out,
                            const __grid_constant__ UmmaArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const ConvGeom& g = args.g;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzle atoms: 1024-byte aligned
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int stages = g.stages;
  const uint32_t a_off = 0;
  const uint32_t b_off = (uint32_t)stages * g.a_stage_bytes;
  const uint32_t st_off = b_off + (uint32_t)stages * g.b_stage_bytes;     // 8 staging tiles
  const uint32_t bar_off = st_off + 8u * kStageTileBytes;
  const uint32_t full_bar = base + bar_off;
  const uint32_t empty_bar = full_bar + 8u * stages;
  const uint32_t accf_bar = empty_bar + 8u * stages;   // 2: accumulator complete
  const uint32_t acce_bar = accf_bar + 16u;            // 2: accumulator drained (leader's is used)
  const uint32_t done_bar = acce_bar + 16u;            // exit path
  const uint32_t tmem_slot = done_bar + 8u;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(base_ptr + bar_off +
                                                                          16u * stages + 40u);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();     // 0 = leader
  const int pair = blockIdx.x >> 1;
  const int n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    const uint32_t extra = (args.test_missing_arrival != 0 && blockIdx.x == 0) ? 1u : 0u;   // test hook
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar + 8u * s, 2 + extra);   // the leader's two producer warps (they expect both CTAs' bytes)
      mbar_init(empty_bar + 8u * s, 1);  // the leader's commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar + 8u * a, 1);   // the leader's commit
      mbar_init(acce_bar + 8u * a, 16);  // eight epilogue warps in each of the two CTAs
    }
    mbar_init(done_bar, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  // Both CTAs' barriers exist before anything arrives on them from the peer.
  cluster_arrive();
  cluster_wait();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  const int n_ksteps = g.n_ksteps;
  const int mma_per_step = g.kc / (int)args.umma_k;
  const uint32_t leader_full = map_to_cta(full_bar, 0);
  const uint32_t leader_acce = map_to_cta(acce_bar, 0);

  if (warp == 0 || warp == 2) {
    // ----------------------------------------------------------- producers
    const bool patch_role = (warp == 0);
    {
      if (lane == 0) {
        prefetch_tensormap(&map_filt);
        prefetch_tensormap(&map_in);
      }
      // Only the leader arrives on its "full" barrier, expecting the bytes of BOTH CTAs'
      // copies of its kind; the peer's copies merely complete on that barrier.  A copy of
      // the peer that lands before the leader's arrival leaves the byte count negative
      // for a moment, which a phase tolerates: it cannot end before the arrival.
      const uint32_t tx_bytes =
          2u * (patch_role ? (uint32_t)(g.b_boxes * g.b_box_bytes) : (uint32_t)g.a_stage_bytes);
      const int m_atoms = kUmmaM / (int)args.atom;
      const uint32_t a_atom_bytes = args.lbo_a_bytes;
      const uint64_t pol_last = l2_policy_evict_last();
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < g.n_tiles && ok; tile += n_pairs) {
        int r = tile;
        const int ob = r % g.o_blocks; r /= g.o_blocks;
        const int nch = r % g.n_chunks; r /= g.n_chunks;
        const int xr = r % g.x_runs;
        const int y = r / g.x_runs;
        const int o0 = ob * 2 * kUmmaM + (int)rank * kUmmaM;          // this CTA's 128 filters
        // this CTA's half of the tile's columns: half of the images or half of the pixels
        const int na0 = (nch * g.tile_n + (g.split_n ? (int)rank * g.cta_n : 0)) / (int)args.atom;
        const int h0 = y * g.stride_h - g.pad_h;
        const int w0 = (xr * g.tile_px + (g.split_n ? 0 : (int)rank * g.cta_px)) * g.stride_w - g.pad_w;
        maxdnn_kstep ks = args.table.s[0];
        for (int s = 0; s < n_ksteps; ++s) {
          const maxdnn_kstep ks_next = args.table.s[s + 1 < n_ksteps ? s + 1 : 0];
          if (!mbar_wait(empty_bar + 8u * stage, phase ^ 1u, args.wc, kDevTimeoutEmpty)) {
            ok = false;
            break;
          }
          const uint32_t fb = leader_full + 8u * stage;    // both CTAs report to the leader
          const uint32_t a_dst = base + a_off + (uint32_t)stage * g.a_stage_bytes;
          const uint32_t b_dst = base + b_off + (uint32_t)stage * g.b_stage_bytes;
          if (elect_one()) {
            if (rank == 0) mbar_arrive_expect_tx(full_bar + 8u * stage, tx_bytes);
            if (patch_role) {
              uint32_t dst = b_dst;
              int w = w0 + ks.kw0;
              for (int t = 0; t < g.b_boxes; ++t) {
                tma_load_5d_pair(dst, &map_in, fb, 0, ks.c0, na0, w, h0 + ks.kh, pol_last);
                dst += g.b_slot_bytes;
                w += g.stride_w;
              }
            } else {
              uint32_t dst = a_dst;
              for (int m = 0; m < m_atoms; ++m) {
                tma_load_4d_pair(dst, &map_filt, fb, o0 + m * (int)args.atom, ks.c0, ks.kw0, ks.kh,
                                 pol_last);
                dst += a_atom_bytes;
              }
            }
          }
          __syncwarp();
          ks = ks_next;
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Leaving early: give copies already issued time to land (their barrier lives
        // in the leader CTA and cannot be polled from here).
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) {}
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer (leader CTA only)
    if (rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      uint32_t chunk = 0;     // chunks started so far: accumulator chunk & 1
      const int chunk_steps = (int)args.chunk_steps;
      const uint64_t desc_hi_a = make_smem_desc(0, args.lbo_a_bytes, args.sbo_bytes, 1u);
      const uint64_t desc_hi_b = make_smem_desc(0, args.lbo_b_bytes, args.sbo_bytes, 1u);
      for (int tile = pair; tile < g.n_tiles && ok; tile += n_pairs) {
        // chunk loop around the plain kernel's step loop (see umma_chunk_conv_kernel)
        for (int s0 = 0; s0 < n_ksteps && ok; s0 += chunk_steps, ++chunk) {
          const uint32_t acc = chunk & 1u;
          if (!mbar_wait(acce_bar + 8u * acc, ((chunk >> 1) & 1u) ^ 1u, args.wc,
                         kDevTimeoutAccFree)) {
            ok = false;
            break;
          }
          tcgen05_fence_after();
          const uint32_t d_tmem = tmem_base + acc * kAccCols;
          const int s1 = s0 + chunk_steps < n_ksteps ? s0 + chunk_steps : n_ksteps;
          uint32_t accumulate = 0;
          for (int s = s0; s < s1; ++s) {
            if (!mbar_wait(full_bar + 8u * stage, phase, args.wc, kDevTimeoutFull)) {
              ok = false;
              break;
            }
            tcgen05_fence_after();
            const uint32_t a_addr = base + a_off + (uint32_t)stage * g.a_stage_bytes;
            const uint32_t b_addr = base + b_off + (uint32_t)stage * g.b_stage_bytes;
            const uint64_t a_base_desc = desc_hi_a | (uint64_t)((a_addr & 0x3FFFFu) >> 4);
            const uint64_t b_base_desc = desc_hi_b | (uint64_t)((b_addr & 0x3FFFFu) >> 4);
            const uint64_t kstep = (uint64_t)(args.kstep_bytes >> 4);
            const uint64_t tap_a = (uint64_t)(args.tap_a_bytes >> 4);
            const uint64_t tap_b = (uint64_t)(args.tap_b_bytes >> 4);
            if (elect_one()) {
              uint32_t acc_flag = accumulate;
              for (int kw = 0; kw < g.kwc; ++kw) {
                uint64_t adesc = a_base_desc + (uint64_t)kw * tap_a;
                uint64_t bdesc = b_base_desc + (uint64_t)kw * tap_b;
#pragma unroll 4
                for (int j = 0; j < mma_per_step; ++j) {
                  tcgen05_mma_pair<false>(d_tmem, adesc, bdesc, args.idesc, acc_flag);
                  acc_flag = 1;
                  adesc += kstep;
                  bdesc += kstep;
                }
              }
              tcgen05_commit_pair(empty_bar + 8u * stage);   // frees the stage in both CTAs
            }
            accumulate = 1;
            __syncwarp();
            if (++stage == stages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          if (elect_one()) tcgen05_commit_pair(accf_bar + 8u * acc);   // chunk complete, both CTAs
        }
      }
      // Exit path: every MMA issued so far has finished before TMEM is released.
      if (elect_one()) tcgen05_commit_pair(done_bar, 1);
      mbar_wait(done_bar, 0, args.wc, kDevTimeoutDrain);
    }
  } else {
    // ------------------------------------------------------------ epilogue
    pair_chunk_epilogue_role(map_out, args, base, base_ptr, st_off, accf_bar, leader_acce, tmem_base,
                             warp, lane, rank, pair, n_pairs);
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
                 "r"((uint32_t)kTmemCols)
                 : "memory");
  }
}

}  // namespace maxdnn
