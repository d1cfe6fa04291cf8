// Two-SM variant of the tensor-core FPROP kernel (tcgen05 MMA with cta_group::2).
//
// A cluster of two CTAs (one SM each) works on one tile of 256 filters x
// (tile_px pixels x tile_n images) <= 256 columns.  CTA r of the pair stages filters
// [128 r, 128 r + 128) of the tile and HALF of the patch columns (half of the tile's
// images when it holds two 128-byte groups of them, else half of its pixels); the
// leader CTA (rank 0) issues one MMA of M = 256 for both, which reads each half of the
// patch operand from the shared memory of the CTA that holds it.  Per SM and per FLOP
// this halves the patch bytes staged and read by the MMAs, and the number of MMA
// instructions and K steps — the shared-memory fill rate (about 64 bytes per clock and
// SM) is what bounds the one-SM kernel.  Each CTA keeps its 128 filter rows of the accumulators in its own
// TMEM and runs its own epilogue.
//
// Synchronisation across the pair uses mbarriers only: both CTAs' copies complete on the
// LEADER's "full" barrier (no multicast copy is used anywhere), on which only the
// leader's producers arrive, expecting the bytes of both CTAs — an arrival on the peer's
// barrier per step costs about a microsecond and serialises the ring; the leader's commits
// arrive on the "empty" / "accumulator complete" barriers of both CTAs; the epilogue
// warps of both CTAs arrive on the leader's "accumulator drained" barrier.  Every wait
// has the same iteration limit and status word as in the one-SM kernel.
#pragma once
#include "umma_conv.cuh"

namespace maxdnn {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}

// Address of the same shared-memory location in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t out;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(smem_addr), "r"(rank));
  return out;
}

__device__ __forceinline__ void cluster_arrive() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Arrivals on a barrier that may live in the peer CTA (cluster-space address).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(
                   cluster_bar),
               "r"(bytes)
               : "memory");
}

// Commit of the leader's MMAs: arrives on the barrier at this offset in the CTAs of
// `mask` (bit r = CTA rank r); 3 = both.
__device__ __forceinline__ void tcgen05_commit_pair(uint32_t bar, uint16_t mask = 3) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 "
      "[%0], %1;" ::"r"(bar),
      "h"(mask)
      : "memory");
}

// Tiled bulk tensor loads whose completion barrier may live in the peer CTA of the pair
// (the destination is always this CTA's shared memory; nothing is multicast).
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                                 int c0, int c1, int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      ".L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_5d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                                 int c0, int c1, int c2, int c3, int c4,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      ".L2::cache_hint [%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4),
      "l"(policy)
      : "memory");
}

template <bool BF16>
__device__ __forceinline__ void tcgen05_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                                 uint32_t idesc, uint32_t accumulate) {
  if constexpr (BF16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}

// Geometry fields used here: tile_m = 256 (filters per pair tile), tile_px = pixels per
// pair tile (even), b_box_w = pixels of ONE CTA's strip, b_stage_bytes = ONE CTA's patch
// bytes per stage; args.tap_b_bytes / lbo_* describe the per-CTA staged layout.
template <bool BF16>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_pair_conv_kernel(const __grid_constant__ CUtensorMap map_filt,
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
      mbar_init(acce_bar + 8u * a, 8);   // four epilogue warps in each of the two CTAs
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
  const int n_cols = g.tile_px * g.tile_n;   // MMA N (both halves)
  const int half_cols = n_cols >> 1;         // columns whose patches each CTA stages
  const uint32_t leader_full = map_to_cta(full_bar, 0);
  const uint32_t leader_acce = map_to_cta(acce_bar, 0);

  if (warp == 0 || warp == 6) {
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
      int it = 0;
      const uint64_t desc_hi_a = make_smem_desc(0, args.lbo_a_bytes, args.sbo_bytes, BF16 ? 2u : 1u);
      const uint64_t desc_hi_b = make_smem_desc(0, args.lbo_b_bytes, args.sbo_bytes, BF16 ? 2u : 1u);
      for (int tile = pair; tile < g.n_tiles && ok; tile += n_pairs, ++it) {
        const int acc = it & 1;
        const uint32_t acc_par = ((uint32_t)(it >> 1) & 1u) ^ 1u;
        if (!mbar_wait(acce_bar + 8u * acc, acc_par, args.wc, kDevTimeoutAccFree)) {
          ok = false;
          break;
        }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * kAccCols;
        uint32_t accumulate = 0;
        for (int s = 0; s < n_ksteps; ++s) {
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
                tcgen05_mma_pair<BF16>(d_tmem, adesc, bdesc, args.idesc, acc_flag);
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
        if (elect_one()) tcgen05_commit_pair(accf_bar + 8u * acc);   // accumulator complete, both CTAs
      }
      // Exit path: every MMA issued so far has finished before TMEM is released.
      if (elect_one()) tcgen05_commit_pair(done_bar, 1);
      mbar_wait(done_bar, 0, args.wc, kDevTimeoutDrain);
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;                  // TMEM lane quarter this warp may read
    const int ew = warp - 2;                 // 0..3: staging tiles 2*ew, 2*ew+1
    const uint32_t stg0 = base + st_off + (uint32_t)(2 * ew) * kStageTileBytes;
    uint8_t* stg0_ptr = base_ptr + st_off + (size_t)(2 * ew) * kStageTileBytes;
    const float alpha = g.alpha;
    const uint64_t pol_first = l2_policy_evict_first();
    bool ok = true;
    int it = 0;
    int buf = 0;
    for (int tile = pair; tile < g.n_tiles && ok; tile += n_pairs, ++it) {
      const int acc = it & 1;
      const uint32_t acc_par = (uint32_t)(it >> 1) & 1u;
      int r = tile;
      const int ob = r % g.o_blocks; r /= g.o_blocks;
      const int nch = r % g.n_chunks; r /= g.n_chunks;
      const int xr = r % g.x_runs;
      const int y = r / g.x_runs;
      const int o0 = ob * 2 * kUmmaM + (int)rank * kUmmaM + q * 32;
      const int n0 = nch * g.tile_n;
      const int x0 = xr * g.tile_px;
      if (!mbar_wait(accf_bar + 8u * acc, acc_par, args.wc, kDevTimeoutAccum)) {
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kAccCols;
      for (int col = 0; col < n_cols; col += 32) {
        // columns [0, half) were staged by the leader, [half, 2 half) by its peer
        const int hr = col >= half_cols ? 1 : 0;
        const int cl = col - hr * half_cols;
        const int pl = cl / g.cta_n;
        const int n = n0 + (g.split_n ? hr * g.cta_n : 0) + (cl - pl * g.cta_n);
        const int x = x0 + (g.split_n ? 0 : hr * g.cta_px) + pl;
        const bool live = (x < g.Wo) && (n < g.Nb) && (o0 < g.No);   // warp-uniform
        if (!live) continue;
        uint32_t v[32];
        tmem_ld_32x32(t_row + (uint32_t)col, v);
        tmem_wait_ld();
        if (lane == 0) bulk_wait_read<1>();
        __syncwarp();
        uint8_t* row = stg0_ptr + (size_t)buf * kStageTileBytes + (size_t)lane * 128;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          float4 o4;
          o4.x = __uint_as_float(v[4 * c + 0]) * alpha;
          o4.y = __uint_as_float(v[4 * c + 1]) * alpha;
          o4.z = __uint_as_float(v[4 * c + 2]) * alpha;
          o4.w = __uint_as_float(v[4 * c + 3]) * alpha;
          *reinterpret_cast<float4*>(row + ((c ^ (lane & 7)) << 4)) = o4;
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_4d_hint(&map_out, stg0 + (uint32_t)buf * kStageTileBytes, n, x, y, o0, pol_first);
          bulk_commit();
        }
        buf ^= 1;
      }
      // all TMEM reads of this accumulator are complete: tell the leader's MMA warp
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_acce + 8u * acc);
    }
    if (lane == 0) bulk_wait_all();
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
