// Tensor-core FPROP convolution kernel for sm_100a (tcgen05 MMA, TMEM accumulators).
//
// GEMM view (Section 3): Out[o, (x, n)] = sum_k F[k, o] * Patch[k, (x, n)].  Both
// operands are contiguous along their non-K dimension (filters along o, patches
// along n), so both are staged "MN-major": one bulk tensor copy writes, per group of
// 32 (fp32) or 64 (bf16) filters / images, kc rows of 128 bytes with the 128-byte
// swizzle, which is exactly the shared-memory layout the MMA descriptors read.
//
// A persistent CTA per SM walks tiles of 128 filters x (tile_px pixels x tile_n
// images) <= 256 columns.  Warps 0 and 6 walk the K-step table and issue the copies of
// the patch boxes and of the filter boxes (one elected lane each; apron zero-filled by
// the copy engine).  Warp 1: one lane issues the MMAs into one of two TMEM
// accumulators and commits to the ring's "empty" barriers.
// Warps 2-5: epilogue — TMEM -> registers, alpha, swizzled staging tile in shared
// memory, bulk tensor store of 32 filters x 32 images (full 128-byte lines), while
// the MMA warp already fills the other accumulator.
#pragma once
#include "plan.h"
#include "ptx_util.cuh"

namespace maxdnn {

constexpr int kUmmaThreads = 224;   // producers: warps 0 and 6; MMA: warp 1; epilogue: warps 2-5
constexpr int kUmmaM = 128;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr int kStageTileBytes = 4096;   // epilogue staging: 32 rows x 128 bytes

struct UmmaArgs {
  ConvGeom g;
  uint32_t idesc;       // instruction descriptor (formats, majors, M, N)
  uint32_t umma_k;      // channels per MMA (8 tf32, 16 bf16)
  uint32_t atom;        // elements per 128-byte row (32 fp32, 64 bf16)
  uint32_t lbo_a_bytes; // distance between groups of 32 / 64 filters in a staged filter tile
  uint32_t lbo_b_bytes; // distance between groups of 32 / 64 columns in a staged patch tile
  uint32_t sbo_bytes;   // distance between groups of channel rows along K
  uint32_t kstep_bytes; // start-address step between consecutive MMAs over the channels of a tap
  uint32_t tap_a_bytes; // filter tile: start-address step from one filter column (kw) to the next
  uint32_t tap_b_bytes; // patch strip: start-address step of one pixel (the next kw's window)
  uint32_t is_bf16;
  uint32_t test_missing_arrival;   // test hook: CTA 0's full barriers expect an arrival that never comes
  uint32_t chunk_steps;            // chunked kernel only: K steps per TMEM accumulator
  WaitCtx wc;          // status block and this launch's epoch (see ptx_util.cuh)
  KStepTable table;
};

// Shared-memory operand descriptor.  layout: 2 = 128-byte swizzle of 16-byte chunks
// (2-byte operands), 1 = 128-byte swizzle of 32-byte chunks (what MN-major 4-byte
// operands need; the copy engine writes the matching pattern).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo,
                                                   uint32_t layout) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of this architecture
  d |= (uint64_t)layout << 61;
  return d;
}

__device__ __forceinline__ void tcgen05_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tcgen05_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}

template <bool BF16>
__device__ __forceinline__ void tcgen05_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc,
                                            uint32_t idesc, uint32_t accumulate) {
  if constexpr (BF16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}

// 32 lanes x 32 consecutive 32-bit columns: thread l receives row (lane base + l).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
        "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}

__device__ __forceinline__ void tmem_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* m, uint32_t src, int c0, int c1,
                                             int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
          reinterpret_cast<uint64_t>(m)),
      "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// L2 eviction policies for bulk copies.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_store_4d_hint(const CUtensorMap* m, uint32_t src, int c0, int c1,
                                                  int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group.L2::cache_hint "
      "[%0, {%2, %3, %4, %5}], [%1], %6;" ::"l"(reinterpret_cast<uint64_t>(m)),
      "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                                 int c0, int c1, int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6}], [%2], %7;" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_5d_hint(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                                 int c0, int c1, int c2, int c3, int c4,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4),
      "l"(policy)
      : "memory");
}
__device__ __forceinline__ void bulk_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

template <bool BF16>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_conv_kernel(const __grid_constant__ CUtensorMap map_filt,
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
      mbar_init(acce_bar + 8u * a, 4);
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
  const int n_cols = g.tile_px * g.tile_n;   // MMA N

  if (warp == 0 || warp == 6) {
    // ----------------------------------------------------------- producers
    // Warp 0 copies the patch boxes, warp 6 the filter boxes: issuing a bulk tensor
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
      int it = 0;
      // Descriptor halves that never change: offsets, version, swizzle mode.
      const uint64_t desc_hi_a = make_smem_desc(0, args.lbo_a_bytes, args.sbo_bytes, BF16 ? 2u : 1u);
      const uint64_t desc_hi_b = make_smem_desc(0, args.lbo_b_bytes, args.sbo_bytes, BF16 ? 2u : 1u);
      for (int tile = blockIdx.x; tile < g.n_tiles && ok; tile += gridDim.x, ++it) {
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
          // One staged strip of tile_px + kwc - 1 pixels serves all kwc filter columns
          // of this filter row: the window of column kw starts kw pixels into the strip.
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
                tcgen05_mma<BF16>(d_tmem, adesc, bdesc, args.idesc, acc_flag);
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
        if (elect_one()) tcgen05_commit(accf_bar + 8u * acc);        // accumulator complete
      }
      // Exit path: every MMA issued so far has finished before TMEM is released.
      if (elect_one()) tcgen05_commit(done_bar);
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
    for (int tile = blockIdx.x; tile < g.n_tiles && ok; tile += gridDim.x, ++it) {
      const int acc = it & 1;
      const uint32_t acc_par = (uint32_t)(it >> 1) & 1u;
      int r = tile;
      const int ob = r % g.o_blocks; r /= g.o_blocks;
      const int nch = r % g.n_chunks; r /= g.n_chunks;
      const int xr = r % g.x_runs;
      const int y = r / g.x_runs;
      const int o0 = ob * kUmmaM + q * 32;
      const int n0 = nch * g.tile_n;
      const int x0 = xr * g.tile_px;
      if (!mbar_wait(accf_bar + 8u * acc, acc_par, args.wc, kDevTimeoutAccum)) {
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kAccCols;
      for (int col = 0; col < n_cols; col += 32) {
        const int p = col / g.tile_n;
        const int n = n0 + (col - p * g.tile_n);
        const int x = x0 + p;
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
      // all TMEM reads of this accumulator are complete: hand it back
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acce_bar + 8u * acc);
    }
    if (lane == 0) bulk_wait_all();
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
