// Filter gradient on the tensor cores (tcgen05 MMA, fp32 accumulators in TMEM), TF32 or
// BF16 operands: the GEMM
//     D[o][k] = sum_r dout[o][r] * patch[k][r],   r = (y, x, n),   dfilt[k][o] = alpha D[o][k]
// with both operands K-major — the reduction index is the contiguous one: a reduction
// step is the 128 bytes of images (32 fp32 / 64 bf16) of one output pixel, which a bulk
// tensor copy lands as rows of 128 bytes with the 128-byte swizzle, the canonical K-major
// operand layout.  A = 128 filters x 128 B, B = up to 256 gradient rows x 128 B (bc
// channels x bh filter rows x Sk filter columns: one box of a bh x Sk window of input
// pixels), four MMAs of 32 bytes of K per step.
//
// Warp 0: copies (one elected lane).  Warp 1: MMA issue and TMEM.  Warps 2-5: epilogue
// (TMEM -> registers -> global; a thread holds one filter, so each stored row of 32
// filters is one 128-byte line), which drains one accumulator while the MMA warp fills
// the other; where a gradient row goes in dfilt comes from a table in shared memory
// built once per CTA (the index arithmetic per element would otherwise cost more than
// the reduction of a split).  The reduction is split over CTAs as in the fp32 kernel;
// partial sums are added in a fixed order by wgrad_reduce_kernel.  Every wait is bounded.
#pragma once
#include "bprop.cuh"
#include "umma_conv.cuh"

namespace maxdnn {

constexpr int kWgUmmaThreads = 192;
constexpr uint32_t kWgUmmaABytes = 128 * 128;      // 128 filters x 128 B
constexpr uint32_t kWgUmmaBBytes = 256 * 128;      // up to 256 gradient rows x 128 B
constexpr uint32_t kWgUmmaTmemCols = 512;         // two accumulators of 256 columns

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

template <bool BF16>
__global__ void __launch_bounds__(kWgUmmaThreads, 1)
wgrad_umma_kernel(const __grid_constant__ CUtensorMap map_dout,
                  const __grid_constant__ CUtensorMap map_in,
                  const __grid_constant__ WgradUmmaArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const WgradGeom& g = args.g;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int stages = g.stages;
  const uint32_t stage_bytes = kWgUmmaABytes + kWgUmmaBBytes;
  const uint32_t bar_off = (uint32_t)stages * stage_bytes;
  const uint32_t full_bar = base + bar_off;
  const uint32_t empty_bar = full_bar + 8u * stages;
  const uint32_t accf_bar = empty_bar + 8u * stages;    // 2: accumulator complete
  const uint32_t acce_bar = accf_bar + 16u;             // 2: accumulator drained
  const uint32_t done_bar = acce_bar + 16u;
  const uint32_t tmem_slot = done_bar + 8u;
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(base_ptr + bar_off + 16u * stages + 40u);
  // row of the tile -> {offset of its dfilt row relative to the tile's first, in rows;
  // (channel within the tile) << 16 | filter row within the tile}
  int2* row_tab = reinterpret_cast<int2*>(base_ptr + bar_off + 1024u);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar + 8u * s, 1);
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
                 "r"(kWgUmmaTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int row = threadIdx.x; row < 256; row += kWgUmmaThreads) {
    const int w_l = row % g.bw;
    const int t = row / g.bw;
    const int h_l = t % g.bh;
    const int c_l = t / g.bh;
    row_tab[row] = make_int2((c_l * g.Skh + h_l) * g.Skw + w_l, (c_l << 16) | h_l);
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  if (warp == 0) {
    // ------------------------------------------------------------- copies
    if (lane == 0) {
      prefetch_tensormap(&map_dout);
      prefetch_tensormap(&map_in);
    }
    const uint32_t tx_bytes = (uint32_t)(g.box_o + g.rows) * 128u;
    const uint64_t pol_last = l2_policy_evict_last();
    WgradCursor pc;
    pc.start(g, blockIdx.x);
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    while (ok && !pc.done(g)) {
      if (!mbar_wait(empty_bar + 8u * stage, phase ^ 1u, args.wc, kDevTimeoutEmpty)) {
        ok = false;
        break;
      }
      const uint32_t fb = full_bar + 8u * stage;
      const uint32_t dst = base + (uint32_t)stage * stage_bytes;
      const int n0 = pc.nc * (int)args.atom;
      if (elect_one()) {
        mbar_arrive_expect_tx(fb, tx_bytes);
        tma_load_4d_hint(dst, &map_dout, fb, n0, pc.x, pc.y, pc.ob * 128, pol_last);
        tma_load_4d_hint(dst + kWgUmmaABytes, &map_in, fb, n0, pc.x * g.stride_w - g.pad_w,
                         pc.y * g.stride_h - g.pad_h + pc.khb * g.bh, pc.cb * g.bc, pol_last);
      }
      __syncwarp();
      if (++stage == stages) { stage = 0; phase ^= 1u; }
      pc.advance(g, (int)gridDim.x);
    }
    if (!ok) {
      for (int s = 0; s < stages; ++s) {
        const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
        mbar_wait_grace(full_bar + 8u * s, par);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issue
    WgradCursor cc;
    cc.start(g, blockIdx.x);
    int stage = 0;
    uint32_t phase = 0;
    uint32_t it = 0;
    bool ok = true;
    // K-major operands, 128-byte swizzle: rows of 128 B, groups of 8 rows 1024 B apart;
    // the next 32 bytes of K are the next 32 bytes of every row (start address + 32).
    const uint64_t desc_hi = make_smem_desc(0, 0, 1024, 2u);
    while (ok && !cc.done(g)) {
      const int n_steps = cc.r_end - cc.r;
      // the epilogue has drained this accumulator (used two items ago)
      const uint32_t acc = it & 1u;
      if (!mbar_wait(acce_bar + 8u * acc, ((it >> 1) & 1u) ^ 1u, args.wc, kDevTimeoutAccFree)) {
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const uint32_t d_tmem = tmem_base + acc * 256u;
      uint32_t accumulate = 0;
      for (int s = 0; s < n_steps; ++s) {
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
            tcgen05_mma<BF16>(d_tmem, adesc0 + (uint64_t)(2 * j), bdesc0 + (uint64_t)(2 * j),
                              args.idesc, accumulate | (uint32_t)(j > 0));
          }
          tcgen05_commit(empty_bar + 8u * stage);
        }
        accumulate = 1;
        __syncwarp();
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      if (elect_one()) tcgen05_commit(accf_bar + 8u * acc);
      __syncwarp();
      cc.start(g, cc.item + (int)gridDim.x);
      ++it;
    }
    if (elect_one()) tcgen05_commit(done_bar);
    mbar_wait(done_bar, 0, args.wc, kDevTimeoutDrain);
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;                      // TMEM lane quarter this warp may read
    WgradCursor cc;
    cc.start(g, blockIdx.x);
    uint32_t it = 0;
    bool ok = true;
    const bool direct = (g.splits == 1);
    const size_t K = (size_t)g.Nc * g.Skh * g.Skw;
    const float scale = direct ? g.alpha : 1.0f;
    while (ok && !cc.done(g)) {
      const uint32_t acc = it & 1u;
      if (!mbar_wait(accf_bar + 8u * acc, (it >> 1) & 1u, args.wc, kDevTimeoutAccum)) {
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const int o = cc.ob * 128 + q * 32 + lane;
      const int c_lim = g.Nc - cc.cb * g.bc;          // channels / filter rows of this tile
      const int h_lim = g.Skh - cc.khb * g.bh;         // that exist
      float* dst = (direct ? args.dfilt : args.partial + (size_t)cc.split * K * g.No) +
                   ((size_t)(cc.cb * g.bc) * g.Skh + (size_t)cc.khb * g.bh) * g.Skw * g.No + o;
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256u;
      for (int col = 0; col < g.rows; col += 32) {
        uint32_t v[32];
        tmem_ld_32x32(t_row + (uint32_t)col, v);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int2 e = row_tab[col + j];
          if (col + j < g.rows && (e.y >> 16) < c_lim && (e.y & 0xffff) < h_lim && o < g.No)
            dst[(size_t)e.x * g.No] = __uint_as_float(v[j]) * scale;
        }
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acce_bar + 8u * acc);
      cc.start(g, cc.item + (int)gridDim.x);
      ++it;
    }
  }

  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(kWgUmmaTmemCols)
                 : "memory");
  }
}

}  // namespace maxdnn
