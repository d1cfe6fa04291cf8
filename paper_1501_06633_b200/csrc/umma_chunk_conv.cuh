// TF32 FPROP on the tensor cores with the sum over K accumulated in CHUNKS.
//
// The tensor core truncates its fp32 accumulator at every MMA; over a long sum of
// same-signed terms that one-sided error grows linearly (about 1e-8 K of the result).
// Here the MMA warp starts a fresh TMEM accumulator every `chunk_steps` K steps, and the
// epilogue warps add the finished chunks into fp32 registers with round-to-nearest adds,
// so the truncation only ever acts on a chunk's short partial sum.  Used by the
// three-product TF32 entry point, whose split operands are exact to 2^-22 and whose
// remaining error was that accumulation.
//
// Same structure as umma_conv_kernel (one SM per tile, 128 filters x <= 256 columns, two
// accumulators in TMEM, bounded waits) with EIGHT epilogue warps: two per TMEM lane
// quarter, each holding 128 of the tile's columns of its 32 filters in registers
// (128 totals per thread).  Warp 0: patch copies, warp 1: MMA issue, warp 2: filter copies,
// warps 3-10: epilogue.  The MMA warp's loop over a chunk's K steps is exactly the plain
// kernel's, with the chunk loop around it: a K step can be as short as four MMAs, and a
// chunk test inside the step loop cost 17 % on such layers.
#pragma once
#include "umma_conv.cuh"

namespace maxdnn {

constexpr int kUmmaChunkThreads = 352;

// 32 lanes x 16 consecutive 32-bit columns: thread l receives row (lane base + l).
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

// Epilogue warps (3-10) of the chunked kernel, kept out of line: their 128 totals per
// thread fill the register file, and inlined they made the compiler spill values that
// the copy and MMA warps read in their short per-step loops.
__device__ __noinline__ void chunk_epilogue_role(const CUtensorMap& map_out, const UmmaArgs& args,
                                                 uint32_t base, uint8_t* base_ptr, uint32_t st_off,
                                                 uint32_t accf_bar, uint32_t acce_bar,
                                                 uint32_t tmem_base, int warp, int lane) {
  const ConvGeom& g = args.g;
  const int n_ksteps = g.n_ksteps;
  const int n_cols = g.tile_px * g.tile_n;
  {
    // Warps 3-10.  A warp may read the TMEM lanes 32 (warp % 4) ...; the two warps of a
    // quarter take the tile's columns 0-127 and 128-255.
    const int q = warp & 3;
    const int half = (warp - 3) >> 2;
    const int ew = warp - 3;                 // 0..7: one staging tile each
    const uint32_t stg = base + st_off + (uint32_t)ew * kStageTileBytes;
    uint8_t* stg_ptr = base_ptr + st_off + (size_t)ew * kStageTileBytes;
    const float alpha = g.alpha;
    const uint64_t pol_first = l2_policy_evict_first();
    const int chunk_steps = (int)args.chunk_steps;
    const int chunks_per_tile = (n_ksteps + chunk_steps - 1) / chunk_steps;
    bool ok = true;
    uint32_t chunk = 0;
    for (int tile = blockIdx.x; tile < g.n_tiles && ok; tile += gridDim.x) {
      int r = tile;
      const int ob = r % g.o_blocks; r /= g.o_blocks;
      const int nch = r % g.n_chunks; r /= g.n_chunks;
      const int xr = r % g.x_runs;
      const int y = r / g.x_runs;
      const int o0 = ob * kUmmaM + q * 32;
      const int n0 = nch * g.tile_n;
      const int x0 = xr * g.tile_px;
      // which of this warp's four groups of 32 columns hold results (warp-uniform bit mask)
      uint32_t live = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int col = half * 128 + 32 * k;
        const int p = col / g.tile_n;
        if ((col < n_cols) && (x0 + p < g.Wo) && (n0 + (col - p * g.tile_n) < g.Nb) && (o0 < g.No))
          live |= 1u << k;
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
        if (lane == 0) mbar_arrive(acce_bar + 8u * acc);
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
          const int col = half * 128 + 32 * k;
          const int p = col / g.tile_n;
          tma_store_4d_hint(&map_out, stg, n0 + (col - p * g.tile_n), x0 + p, y, o0, pol_first);
          bulk_commit();
        }
      }
    }
    if (lane == 0) bulk_wait_all();
  }
}

__global__ void __launch_bounds__(kUmmaChunkThreads, 1)
umma_chunk_conv_kernel(const __grid_constant__ CUtensorMap map_filt,
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
  const uint32_t acce_bar = accf_bar + 16u;            // 2: accumulator drained
  const uint32_t done_bar = acce_bar + 16u;            // exit path
  const uint32_t tmem_slot = done_bar + 8u;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(base_ptr + bar_off +
                                                                          16u * stages + 40u);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    const uint32_t extra = (args.test_missing_arrival != 0 && blockIdx.x == 0) ? 1u : 0u;   // test hook
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar + 8u * s, 2 + extra);   // one arrival per producer warp
      mbar_init(empty_bar + 8u * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar + 8u * a, 1);
      mbar_init(acce_bar + 8u * a, 8);
    }
    mbar_init(done_bar, 1);
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  const int n_ksteps = g.n_ksteps;
  const int mma_per_step = g.kc / (int)args.umma_k;

  if (warp == 0 || warp == 2) {
    // ----------------------------------------------------------- producers
    // Warp 0 copies the patch boxes, warp 2 the filter boxes: issuing a bulk tensor
    // copy costs the issuing warp a few hundred cycles, and a K step is short.
    const bool patch_role = (warp == 0);
    // The whole warp walks the loops, so coordinates and addresses are computed in
    // warp-uniform control flow; one elected lane arms the barrier and issues the
    // copies.  A K step lasts a few hundred nanoseconds, so this loop is short and
    // does not sleep while it waits for a ring slot.
    {
      if (lane == 0) {
        prefetch_tensormap(&map_filt);
        prefetch_tensormap(&map_in);
      }
      const uint32_t tx_bytes =
          patch_role ? (uint32_t)(g.b_boxes * g.b_box_bytes) : (uint32_t)g.a_stage_bytes;
      const int m_atoms = kUmmaM / (int)args.atom;
      const uint32_t a_atom_bytes = args.lbo_a_bytes;
      const uint64_t pol_last = l2_policy_evict_last();
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < g.n_tiles && ok; tile += gridDim.x) {
        int r = tile;
        const int ob = r % g.o_blocks; r /= g.o_blocks;
        const int nch = r % g.n_chunks; r /= g.n_chunks;
        const int xr = r % g.x_runs;
        const int y = r / g.x_runs;
        const int o0 = ob * kUmmaM;
        const int na0 = (nch * g.tile_n) / (int)args.atom;
        const int h0 = y * g.stride_h - g.pad_h;
        const int w0 = xr * g.tile_px * g.stride_w - g.pad_w;
        maxdnn_kstep ks = args.table.s[0];
        for (int s = 0; s < n_ksteps; ++s) {
          const maxdnn_kstep ks_next = args.table.s[s + 1 < n_ksteps ? s + 1 : 0];
          if (!mbar_wait(empty_bar + 8u * stage, phase ^ 1u, args.wc, kDevTimeoutEmpty)) {
            ok = false;
            break;
          }
          const uint32_t fb = full_bar + 8u * stage;
          const uint32_t a_dst = base + a_off + (uint32_t)stage * g.a_stage_bytes;
          const uint32_t b_dst = base + b_off + (uint32_t)stage * g.b_stage_bytes;
          if (elect_one()) {
            mbar_arrive_expect_tx(fb, tx_bytes);
            if (patch_role) {
              uint32_t dst = b_dst;
              int w = w0 + ks.kw0;
              for (int t = 0; t < g.b_boxes; ++t) {
                tma_load_5d_hint(dst, &map_in, fb, 0, ks.c0, na0, w, h0 + ks.kh, pol_last);
                dst += g.b_slot_bytes;
                w += g.stride_w;
              }
            } else {
              uint32_t dst = a_dst;
              for (int m = 0; m < m_atoms; ++m) {
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
        for (int s = 0; s < stages; ++s) {
          const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
          mbar_wait_grace(full_bar + 8u * s, par);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer
    // The whole warp walks the loops (so that addresses and descriptors are computed
    // in warp-uniform control flow); one elected lane issues each MMA and commit.
    {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      uint32_t chunk = 0;     // chunks started so far: accumulator chunk & 1
      const int chunk_steps = (int)args.chunk_steps;
      // Descriptor halves that never change: offsets, version, swizzle mode.
      const uint64_t desc_hi_a = make_smem_desc(0, args.lbo_a_bytes, args.sbo_bytes, 1u);
      const uint64_t desc_hi_b = make_smem_desc(0, args.lbo_b_bytes, args.sbo_bytes, 1u);
      for (int tile = blockIdx.x; tile < g.n_tiles && ok; tile += gridDim.x) {
        // One chunk = up to chunk_steps K steps into one accumulator; the loop over its
        // steps is the plain kernel's (nothing but the step itself inside it: a K step
        // can be as short as four MMAs).
        for (int s0 = 0; s0 < n_ksteps && ok; s0 += chunk_steps, ++chunk) {
          const uint32_t acc = chunk & 1u;
          // the accumulator must have been drained (it held the chunk before last)
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
                  tcgen05_mma<false>(d_tmem, adesc, bdesc, args.idesc, acc_flag);
                  acc_flag = 1;
                  adesc += kstep;
                  bdesc += kstep;
                }
              }
              tcgen05_commit(empty_bar + 8u * stage);   // frees the stage when these MMAs finish
            }
            accumulate = 1;
            __syncwarp();
            if (++stage == stages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          if (elect_one()) tcgen05_commit(accf_bar + 8u * acc);        // chunk complete
        }
      }
      // Exit path: every MMA issued so far has finished before TMEM is released.
      if (elect_one()) tcgen05_commit(done_bar);
      mbar_wait(done_bar, 0, args.wc, kDevTimeoutDrain);
    }
  } else {
    // ------------------------------------------------------------ epilogue
    chunk_epilogue_role(map_out, args, base, base_ptr, st_off, accf_bar, acce_bar, tmem_base, warp, lane);
  }

  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)kTmemCols)
                 : "memory");
  }
}

}  // namespace maxdnn
