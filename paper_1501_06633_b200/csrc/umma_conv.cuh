// Tensor-core FPROP convolution kernel for sm_100a (tcgen05 MMA, TMEM accumulators): ONE
// kernel template for one-SM and two-SM tiles, TF32 and BF16 operands, and for the sum over K
// kept in one accumulator or added up in chunks.
//
// GEMM view (Section 3): Out[o, (x, n)] = sum_k F[k, o] * Patch[k, (x, n)].  Both
// operands are contiguous along their non-K dimension (filters along o, patches
// along n), so both are staged "MN-major": one bulk tensor copy writes, per group of
// 32 (fp32) or 64 (bf16) filters / images, kc rows of 128 bytes with the 128-byte
// swizzle, which is exactly the shared-memory layout the MMA descriptors read.
//
// Roles.  Warp 0 walks the K-step table and issues the copies of the patch boxes, warp 2
// those of the filter boxes (one elected lane each; apron zero-filled by the copy engine).
// Warp 1: one lane issues the MMAs into one of two TMEM accumulators and commits to the
// ring's "empty" barriers.  Warps 3..: epilogue — TMEM -> registers, alpha, swizzled
// staging tile in shared memory, bulk tensor store of 32 filters x 32 images (full
// 128-byte lines) — while the MMA warp already fills the other accumulator.  Every wait is
// bounded and ends in a status code; TMEM is always freed.
//
// PAIR (two-SM tiles, tcgen05 cta_group::2).  A cluster of two CTAs works on one tile of 256
// filters x (tile_px pixels x tile_n images) <= 256 columns.  CTA r of the pair stages
// filters [128 r, 128 r + 128) of the tile and HALF of the patch columns (half of the
// tile's images when it holds two 128-byte groups of them, else half of its pixels); the
// leader CTA (rank 0) issues one MMA of M = 256 for both, which reads each half of the patch
// operand from the shared memory of the CTA that holds it.  Per SM and per FLOP this halves
// the patch bytes staged and read by the MMAs, and the number of MMA instructions and K
// steps — the shared-memory fill rate (about 64 bytes per clock and SM) is what bounds the
// one-SM tile.  Each CTA keeps its 128 filter rows of the accumulators in its own TMEM and
// runs its own epilogue.  Synchronisation across the pair uses mbarriers only: both CTAs'
// copies complete on the LEADER's "full" barrier (no multicast copy is used anywhere), on
// which only the leader's producers arrive, expecting the bytes of both CTAs — an arrival
// on the peer's barrier per step costs about a microsecond and serialises the ring; the
// leader's commits arrive on the "empty" / "accumulator complete" barriers of both CTAs; the
// epilogue warps of both CTAs arrive on the leader's "accumulator drained" barrier.
//
// CHUNK (TF32 only; behind the three-product entry points).  The tensor core truncates its
// fp32 accumulator at every MMA; over a long sum of same-signed terms that one-sided error
// grows linearly (about 1e-8 K of the result).  Here the MMA warp starts a fresh TMEM
// accumulator every `chunk_steps` K steps, and EIGHT epilogue warps — two per TMEM lane
// quarter, each holding 128 of the tile's columns of its 32 filters in registers — add the
// finished chunks with round-to-nearest fp32 adds, so the truncation only ever acts on a
// chunk's short partial sum.  The MMA warp's loop over a chunk's K steps is the plain loop
// with the chunk loop around it: a K step can be as short as four MMAs, and a chunk test
// inside the step loop cost 17 % on such layers.  (The plain kernel is the same code with
// one chunk per tile.)
#pragma once
#include "umma_util.cuh"

namespace maxdnn {

// warps: patch copies, MMA, filter copies, then 4 (plain) or 8 (chunked) epilogue warps
__host__ __device__ constexpr int umma_threads(bool chunk) { return (3 + (chunk ? 8 : 4)) * 32; }

// What the roles of one CTA share: where things are in shared memory and which tile comes next.
struct UmmaCtx {
  uint32_t base;            // shared-memory window address of the (1024-byte aligned) carve
  uint8_t* base_ptr;        // the same place as a generic pointer
  uint32_t a_off, b_off, st_off;
  uint32_t full_bar, empty_bar, accf_bar, acce_bar, done_bar;
  uint32_t leader_full, leader_acce;   // the leader CTA's barriers (= the CTA's own if not PAIR)
  uint32_t tmem_base;
  uint32_t rank;            // 0 = leader (always 0 if not PAIR)
  int unit, n_units;        // this CTA's (pair's) first tile and the tile stride
};

// (pixel, image) of column `col` of a tile whose first pixel / image are x0 / n0.  Two-SM
// tiles: columns [0, half) were staged by the leader, [half, 2 half) by its peer.
__device__ __forceinline__ void umma_col_to_xn(const ConvGeom& g, int half_cols, int col, int x0, int n0,
                                               int* x, int* n) {
  const int hr = col >= half_cols ? 1 : 0;
  const int cl = col - hr * half_cols;
  const int pl = cl / g.cta_n;
  *n = n0 + (g.split_n ? hr * g.cta_n : 0) + (cl - pl * g.cta_n);
  *x = x0 + (g.split_n ? 0 : hr * g.cta_px) + pl;
}

// Epilogue of the plain kernel (warps 3-6): per group of 32 columns one TMEM load, alpha, a
// swizzled 4 KB staging tile (two per warp, alternating) and one bulk tensor store.
template <bool PAIR>
__device__ __forceinline__ void umma_epilogue_plain(const CUtensorMap& map_out, const UmmaArgs& args,
                                                    const UmmaCtx& cx, int warp, int lane) {
  const ConvGeom& g = args.g;
  const int n_cols = g.tile_px * g.tile_n;                 // MMA N
  const int half_cols = PAIR ? n_cols >> 1 : n_cols;
  const int q = warp & 3;                  // TMEM lane quarter this warp may read
  const int ew = warp - 3;                 // 0..3: staging tiles 2*ew, 2*ew+1
  const uint32_t stg0 = cx.base + cx.st_off + (uint32_t)(2 * ew) * kStageTileBytes;
  uint8_t* stg0_ptr = cx.base_ptr + cx.st_off + (size_t)(2 * ew) * kStageTileBytes;
  const float alpha = g.alpha;
  const uint64_t pol_first = l2_policy_evict_first();
  bool ok = true;
  int it = 0;
  int buf = 0;
  for (int tile = cx.unit; tile < g.n_tiles && ok; tile += cx.n_units, ++it) {
    const int acc = it & 1;
    const uint32_t acc_par = (uint32_t)(it >> 1) & 1u;
    int r = tile;
    const int ob = r % g.o_blocks; r /= g.o_blocks;
    const int nch = r % g.n_chunks; r /= g.n_chunks;
    const int xr = r % g.x_runs;
    const int y = r / g.x_runs;
    const int o0 = ob * (PAIR ? 2 : 1) * kUmmaM + (int)cx.rank * kUmmaM + q * 32;
    const int n0 = nch * g.tile_n;
    const int x0 = xr * g.tile_px;
    if (!mbar_wait(cx.accf_bar + 8u * acc, acc_par, args.wc, kDevTimeoutAccum)) {
      ok = false;
      break;
    }
    tcgen05_fence_after();
    const uint32_t t_row = cx.tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kAccCols;
    for (int col = 0; col < n_cols; col += 32) {
      int x, n;
      umma_col_to_xn(g, half_cols, col, x0, n0, &x, &n);
      const bool live = (x < g.Wo) && (n < g.Nb) && (o0 < g.No);   // warp-uniform
      if (!live) continue;
      uint32_t v[32];
      tmem_ld_32x32(t_row + (uint32_t)col, v);
      tmem_wait_ld();
      // the staging tile about to be overwritten must have been read by its store
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
    // all TMEM reads of this accumulator are complete: hand it back to the (leader's) MMA warp
    tcgen05_fence_before();
    __syncwarp();
    if (lane == 0) {
      if constexpr (PAIR) mbar_arrive_cluster(cx.leader_acce + 8u * acc);
      else mbar_arrive(cx.acce_bar + 8u * acc);
    }
  }
  if (lane == 0) bulk_wait_all();
}

// Epilogue of the chunked kernel (warps 3-10), kept out of line: its 128 totals per thread
// fill the register file, and inlined they made the compiler spill values that the copy and
// MMA warps read in their short per-step loops.  A warp may read the TMEM lanes 32 (warp % 4)
// ...; the two warps of a quarter take the tile's columns 0-127 and 128-255.
template <bool PAIR>
__device__ __noinline__ void umma_epilogue_chunk(const CUtensorMap& map_out, const UmmaArgs& args,
                                                 const UmmaCtx cx, int warp, int lane) {
  const ConvGeom& g = args.g;
  const int n_ksteps = g.n_ksteps;
  const int n_cols = g.tile_px * g.tile_n;
  const int half_cols = PAIR ? n_cols >> 1 : n_cols;
  const int q = warp & 3;
  const int half = (warp - 3) >> 2;
  const int ew = warp - 3;                 // 0..7: one staging tile each
  const uint32_t stg = cx.base + cx.st_off + (uint32_t)ew * kStageTileBytes;
  uint8_t* stg_ptr = cx.base_ptr + cx.st_off + (size_t)ew * kStageTileBytes;
  const float alpha = g.alpha;
  const uint64_t pol_first = l2_policy_evict_first();
  const int chunk_steps = (int)args.chunk_steps;
  const int chunks_per_tile = (n_ksteps + chunk_steps - 1) / chunk_steps;
  bool ok = true;
  uint32_t chunk = 0;
  for (int tile = cx.unit; tile < g.n_tiles && ok; tile += cx.n_units) {
    int r = tile;
    const int ob = r % g.o_blocks; r /= g.o_blocks;
    const int nch = r % g.n_chunks; r /= g.n_chunks;
    const int xr = r % g.x_runs;
    const int y = r / g.x_runs;
    const int o0 = ob * (PAIR ? 2 : 1) * kUmmaM + (int)cx.rank * kUmmaM + q * 32;
    const int n0 = nch * g.tile_n;
    const int x0 = xr * g.tile_px;
    // which of this warp's four groups of 32 columns hold results (warp-uniform bit mask)
    uint32_t live = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int col = half * 128 + 32 * k;
      int x, n;
      umma_col_to_xn(g, half_cols, col, x0, n0, &x, &n);
      if ((col < n_cols) && (x < g.Wo) && (n < g.Nb) && (o0 < g.No)) live |= 1u << k;
    }
    float tot[128];
    for (int c = 0; c < chunks_per_tile && ok; ++c, ++chunk) {
      const uint32_t acc = chunk & 1u;
      if (!mbar_wait(cx.accf_bar + 8u * acc, (chunk >> 1) & 1u, args.wc, kDevTimeoutAccum)) {
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const uint32_t t_row = cx.tmem_base + ((uint32_t)(q * 32) << 16) + acc * kAccCols +
                             (uint32_t)(half * 128);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (!((live >> k) & 1u)) continue;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {      // 16 columns per load: the totals leave few registers
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
      // this accumulator may be overwritten by the chunk after next
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) {
        if constexpr (PAIR) mbar_arrive_cluster(cx.leader_acce + 8u * acc);
        else mbar_arrive(cx.acce_bar + 8u * acc);
      }
    }
    if (!ok) break;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (!((live >> k) & 1u)) continue;
      // the staging tile must have been read by the previous store
      if (lane == 0) bulk_wait_read<0>();
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
        int x, n;
        umma_col_to_xn(g, half_cols, half * 128 + 32 * k, x0, n0, &x, &n);
        tma_store_4d_hint(&map_out, stg, n, x, y, o0, pol_first);
        bulk_commit();
      }
    }
  }
  if (lane == 0) bulk_wait_all();
}

// Geometry fields as the two-SM tiles read them: tile_m = 256 (filters per pair tile),
// tile_px = pixels per pair tile, b_box_w = pixels of ONE CTA's strip, b_stage_bytes = ONE
// CTA's patch bytes per stage; args.tap_b_bytes / lbo_* describe the per-CTA staged layout.
template <bool BF16, bool PAIR, bool CHUNK>
__global__ void __launch_bounds__(umma_threads(CHUNK), 1)
umma_conv_kernel(const __grid_constant__ CUtensorMap map_filt,
                 const __grid_constant__ CUtensorMap map_in,
                 const __grid_constant__ CUtensorMap map_out,
                 const __grid_constant__ UmmaArgs args) {
  static_assert(!(CHUNK && BF16), "the chunked sum exists for TF32 operands only");
  constexpr int kEpiWarps = CHUNK ? 8 : 4;
  extern __shared__ uint8_t smem_raw[];
  const ConvGeom& g = args.g;
  UmmaCtx cx;
  cx.base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzle atoms: 1024-byte aligned
  cx.base_ptr = smem_raw + (cx.base - smem_u32(smem_raw));
  const int stages = g.stages;
  cx.a_off = 0;
  cx.b_off = (uint32_t)stages * g.a_stage_bytes;
  cx.st_off = cx.b_off + (uint32_t)stages * g.b_stage_bytes;     // 8 staging tiles
  const uint32_t bar_off = cx.st_off + 8u * kStageTileBytes;
  cx.full_bar = cx.base + bar_off;
  cx.empty_bar = cx.full_bar + 8u * stages;
  cx.accf_bar = cx.empty_bar + 8u * stages;   // 2: accumulator complete
  cx.acce_bar = cx.accf_bar + 16u;            // 2: accumulator drained (two-SM: the leader's is used)
  cx.done_bar = cx.acce_bar + 16u;            // exit path
  const uint32_t tmem_slot = cx.done_bar + 8u;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(cx.base_ptr + bar_off +
                                                                          16u * stages + 40u);
  const uint32_t base = cx.base;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  cx.rank = PAIR ? cluster_ctarank() : 0u;     // 0 = leader
  cx.unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  cx.n_units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const uint32_t rank = cx.rank;

  if (threadIdx.x == 0) {
    const uint32_t extra = (args.test_missing_arrival != 0 && blockIdx.x == 0) ? 1u : 0u;   // test hook
    for (int s = 0; s < stages; ++s) {
      // one arrival per producer warp (two-SM: of the leader, expecting both CTAs' bytes)
      mbar_init(cx.full_bar + 8u * s, 2 + extra);
      mbar_init(cx.empty_bar + 8u * s, 1);  // the (leader's) commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(cx.accf_bar + 8u * a, 1);                         // the (leader's) commit
      mbar_init(cx.acce_bar + 8u * a, kEpiWarps * (PAIR ? 2 : 1)); // the epilogue warps (of both CTAs)
    }
    mbar_init(cx.done_bar, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) tmem_alloc_all<PAIR>(tmem_slot);
  tcgen05_fence_before();
  __syncthreads();
  if constexpr (PAIR) {
    // Both CTAs' barriers exist before anything arrives on them from the peer.
    cluster_arrive();
    cluster_wait();
  }
  tcgen05_fence_after();
  cx.tmem_base = *tmem_slot_ptr;
  cx.leader_full = PAIR ? map_to_cta(cx.full_bar, 0) : cx.full_bar;
  cx.leader_acce = PAIR ? map_to_cta(cx.acce_bar, 0) : cx.acce_bar;

  const int n_ksteps = g.n_ksteps;
  const int mma_per_step = g.kc / (int)args.umma_k;

  if (warp == 0 || warp == 2) {
    // ----------------------------------------------------------- producers
    // Warp 0 copies the patch boxes, warp 2 the filter boxes: issuing a bulk tensor copy
    // costs the issuing warp a few hundred cycles, and a K step is short.  The whole warp
    // walks the loops, so coordinates and addresses are computed in warp-uniform control
    // flow; one elected lane arms the barrier and issues the copies.  A K step lasts a few
    // hundred nanoseconds, so this loop does not sleep while it waits for a ring slot.
    const bool patch_role = (warp == 0);
    if (lane == 0) {
      prefetch_tensormap(&map_filt);
      prefetch_tensormap(&map_in);
    }
    // Two-SM: only the leader arrives on its "full" barrier, expecting the bytes of BOTH
    // CTAs' copies of its kind; the peer's copies merely complete on that barrier.  A copy of
    // the peer that lands before the leader's arrival leaves the byte count negative for a
    // moment, which a phase tolerates: it cannot end before the arrival.
    const uint32_t tx_bytes = (PAIR ? 2u : 1u) *
        (patch_role ? (uint32_t)(g.b_boxes * g.b_box_bytes) : (uint32_t)g.a_stage_bytes);
    const int m_atoms = kUmmaM / (int)args.atom;
    const uint32_t a_atom_bytes = args.lbo_a_bytes;
    const uint64_t pol_last = l2_policy_evict_last();
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = cx.unit; tile < g.n_tiles && ok; tile += cx.n_units) {
      int r = tile;
      const int ob = r % g.o_blocks; r /= g.o_blocks;
      const int nch = r % g.n_chunks; r /= g.n_chunks;
      const int xr = r % g.x_runs;
      const int y = r / g.x_runs;
      const int o0 = ob * (PAIR ? 2 : 1) * kUmmaM + (int)rank * kUmmaM;      // this CTA's 128 filters
      // this CTA's share of the tile's columns (two-SM: half of the images or of the pixels)
      const int na0 = (nch * g.tile_n + (g.split_n ? (int)rank * g.cta_n : 0)) / (int)args.atom;
      const int h0 = y * g.stride_h - g.pad_h;
      const int w0 = (xr * g.tile_px + (g.split_n ? 0 : (int)rank * g.cta_px)) * g.stride_w - g.pad_w;
      maxdnn_kstep ks = args.table.s[0];
      for (int s = 0; s < n_ksteps; ++s) {
        const maxdnn_kstep ks_next = args.table.s[s + 1 < n_ksteps ? s + 1 : 0];
        if (!mbar_wait(cx.empty_bar + 8u * stage, phase ^ 1u, args.wc, kDevTimeoutEmpty)) {
          ok = false;
          break;
        }
        const uint32_t fb = cx.leader_full + 8u * stage;    // two-SM: both CTAs report to the leader
        const uint32_t a_dst = base + cx.a_off + (uint32_t)stage * g.a_stage_bytes;
        const uint32_t b_dst = base + cx.b_off + (uint32_t)stage * g.b_stage_bytes;
        if (elect_one()) {
          if (rank == 0) mbar_arrive_expect_tx(cx.full_bar + 8u * stage, tx_bytes);
          if (patch_role) {
            uint32_t dst = b_dst;
            int w = w0 + ks.kw0;
            for (int t = 0; t < g.b_boxes; ++t) {
              if constexpr (PAIR) tma_load_5d_pair(dst, &map_in, fb, 0, ks.c0, na0, w, h0 + ks.kh, pol_last);
              else tma_load_5d_hint(dst, &map_in, fb, 0, ks.c0, na0, w, h0 + ks.kh, pol_last);
              dst += g.b_slot_bytes;
              w += g.stride_w;
            }
          } else {
            uint32_t dst = a_dst;
            for (int m = 0; m < m_atoms; ++m) {
              if constexpr (PAIR)
                tma_load_4d_pair(dst, &map_filt, fb, o0 + m * (int)args.atom, ks.c0, ks.kw0, ks.kh, pol_last);
              else
                tma_load_4d_hint(dst, &map_filt, fb, o0 + m * (int)args.atom, ks.c0, ks.kw0, ks.kh, pol_last);
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
      // Leaving early: give copies already issued time to land.
      if constexpr (PAIR) {
        // (their barrier lives in the leader CTA and cannot be polled from the peer)
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) {}
      } else {
        for (int s = 0; s < stages; ++s) {
          const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
          mbar_wait_grace(cx.full_bar + 8u * s, par);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer (two-SM: leader only)
    // The whole warp walks the loops (so that addresses and descriptors are computed in
    // warp-uniform control flow); one elected lane issues each MMA and commit.
    if (rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      uint32_t chunk = 0;     // accumulators started so far: this one is chunk & 1
      const int chunk_steps = CHUNK ? (int)args.chunk_steps : n_ksteps;   // plain: one per tile
      // Descriptor halves that never change: offsets, version, swizzle mode.
      const uint64_t desc_hi_a = make_smem_desc(0, args.lbo_a_bytes, args.sbo_bytes, BF16 ? 2u : 1u);
      const uint64_t desc_hi_b = make_smem_desc(0, args.lbo_b_bytes, args.sbo_bytes, BF16 ? 2u : 1u);
      for (int tile = cx.unit; tile < g.n_tiles && ok; tile += cx.n_units) {
        // One chunk = up to chunk_steps K steps into one accumulator; the loop over its steps
        // has nothing but the step itself inside it.
        for (int s0 = 0; s0 < n_ksteps && ok; s0 += chunk_steps, ++chunk) {
          const uint32_t acc = chunk & 1u;
          // the accumulator must have been drained (it held the chunk before last)
          if (!mbar_wait(cx.acce_bar + 8u * acc, ((chunk >> 1) & 1u) ^ 1u, args.wc, kDevTimeoutAccFree)) {
            ok = false;
            break;
          }
          tcgen05_fence_after();
          const uint32_t d_tmem = cx.tmem_base + acc * kAccCols;
          const int s1 = s0 + chunk_steps < n_ksteps ? s0 + chunk_steps : n_ksteps;
          uint32_t accumulate = 0;
          for (int s = s0; s < s1; ++s) {
            if (!mbar_wait(cx.full_bar + 8u * stage, phase, args.wc, kDevTimeoutFull)) {
              ok = false;
              break;
            }
            tcgen05_fence_after();
            const uint32_t a_addr = base + cx.a_off + (uint32_t)stage * g.a_stage_bytes;
            const uint32_t b_addr = base + cx.b_off + (uint32_t)stage * g.b_stage_bytes;
            // One staged strip of tile_px + kwc - 1 pixels serves all kwc filter columns of
            // this filter row: the window of column kw starts kw pixels into the strip.
            const uint64_t a_base_desc = desc_hi_a | (uint64_t)((a_addr & 0x3FFFFu) >> 4);
            const uint64_t b_base_desc = desc_hi_b | (uint64_t)((b_addr & 0x3FFFFu) >> 4);
            const uint64_t kstep = (uint64_t)(args.kstep_bytes >> 4);
            const uint64_t tap_a = (uint64_t)(args.tap_a_bytes >> 4);
            const uint64_t tap_b = (uint64_t)(args.tap_b_bytes >> 4);
            if (elect_one()) {
              // start addresses only move inside the 14-bit address field: plain adds
              uint32_t acc_flag = accumulate;
              for (int kw = 0; kw < g.kwc; ++kw) {
                uint64_t adesc = a_base_desc + (uint64_t)kw * tap_a;
                uint64_t bdesc = b_base_desc + (uint64_t)kw * tap_b;
#pragma unroll 4
                for (int j = 0; j < mma_per_step; ++j) {
                  if constexpr (PAIR) tcgen05_mma_pair<BF16>(d_tmem, adesc, bdesc, args.idesc, acc_flag);
                  else tcgen05_mma<BF16>(d_tmem, adesc, bdesc, args.idesc, acc_flag);
                  acc_flag = 1;
                  adesc += kstep;
                  bdesc += kstep;
                }
              }
              // frees the stage (in both CTAs) when these MMAs finish
              if constexpr (PAIR) tcgen05_commit_pair(cx.empty_bar + 8u * stage);
              else tcgen05_commit(cx.empty_bar + 8u * stage);
            }
            accumulate = 1;
            __syncwarp();
            if (++stage == stages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          if (elect_one()) {                                     // accumulator complete
            if constexpr (PAIR) tcgen05_commit_pair(cx.accf_bar + 8u * acc);
            else tcgen05_commit(cx.accf_bar + 8u * acc);
          }
        }
      }
      // Exit path: every MMA issued so far has finished before TMEM is released.
      if (elect_one()) {
        if constexpr (PAIR) tcgen05_commit_pair(cx.done_bar, 1);
        else tcgen05_commit(cx.done_bar);
      }
      mbar_wait(cx.done_bar, 0, args.wc, kDevTimeoutDrain);
    }
  } else {
    // ------------------------------------------------------------ epilogue
    if constexpr (CHUNK) umma_epilogue_chunk<PAIR>(map_out, args, cx, warp, lane);
    else umma_epilogue_plain<PAIR>(map_out, args, cx, warp, lane);
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
    tmem_dealloc_all<PAIR>(cx.tmem_base);
  }
}

}  // namespace maxdnn
