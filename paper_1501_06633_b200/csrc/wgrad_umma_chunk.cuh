// Filter gradient on the tensor cores, TF32, with the reduction accumulated in CHUNKS (see
// umma_chunk_conv.cuh for why: the tensor core truncates its fp32 accumulator at every MMA).
// Same structure as wgrad_umma_kernel; the MMA warp starts a fresh TMEM accumulator every
// chunk_steps reduction steps and eight epilogue warps add the chunks in registers.  Used by
// maxdnn_conv_bprop_filter_tf32x3, whose three TF32 products are one reduction over three
// times the images (three passes over tensors stored [hi | lo] along the image axis).
// Warp 0: copies, warp 1: MMA issue and TMEM, warps 2-9: epilogue.
#pragma once
#include "umma_chunk_conv.cuh"
#include "wgrad_umma.cuh"

namespace maxdnn {

constexpr int kWgChunkThreads = 320;

// Epilogue warps (2-9) of the chunked filter-gradient kernel, out of line (128 totals per
// thread).  The two warps of a TMEM lane quarter take the tile's gradient rows 0-127 and
// 128-255 of their 32 filters; every finished chunk is added into the totals with
// round-to-nearest fp32 adds; after an item's last chunk the totals are stored through the
// row table like the plain kernel's accumulator.
__device__ __noinline__ void wgrad_chunk_epilogue_role(const WgradUmmaArgs& args, const int2* row_tab,
                                                       uint32_t accf_bar, uint32_t acce_bar,
                                                       uint32_t tmem_base, int warp, int lane) {
  const WgradGeom& g = args.g;
  const int q = warp & 3;                      // TMEM lane quarter this warp may read
  const int half = (warp - 2) >> 2;            // which 128 gradient rows
  const int chunk_steps = (int)args.chunk_steps;
  WgradCursor cc;
  cc.start(g, blockIdx.x);
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
        if (half * 128 + 16 * k >= g.rows) continue;          // warp-uniform
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
      if (lane == 0) mbar_arrive(acce_bar + 8u * acc);
    }
    if (!ok) break;
    const int o = cc.ob * 128 + q * 32 + lane;
    const int c_lim = g.Nc - cc.cb * g.bc;          // channels / filter rows of this tile
    const int h_lim = g.Skh - cc.khb * g.bh;         // that exist
    float* dst = (direct ? args.dfilt : args.partial + (size_t)cc.split * K * g.No) +
                 ((size_t)(cc.cb * g.bc) * g.Skh + (size_t)cc.khb * g.bh) * g.Skw * g.No + o;
#pragma unroll
    for (int j = 0; j < 128; ++j) {
      const int col = half * 128 + j;
      const int2 e = row_tab[col];
      if (col < g.rows && (e.y >> 16) < c_lim && (e.y & 0xffff) < h_lim && o < g.No)
        dst[(size_t)e.x * g.No] = tot[j] * scale;
    }
    cc.start(g, cc.item + (int)gridDim.x);
  }
}

__global__ void __launch_bounds__(kWgChunkThreads, 1)
wgrad_umma_chunk_kernel(const __grid_constant__ CUtensorMap map_dout,
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
      mbar_init(acce_bar + 8u * a, 8);
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
  for (int row = threadIdx.x; row < 256; row += kWgChunkThreads) {
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
      // The image axis of the reduction holds the three products one after another:
      // part 0 = gradient hi x map hi, 1 = hi x lo, 2 = lo x hi; both tensors are stored
      // as [hi | lo] along their image axis.
      const int per = (int)args.x3_per_part;
      const int part = pc.nc / per;
      const int within = pc.nc - part * per;
      const int n_g = ((part == 2 ? per : 0) + within) * (int)args.atom;
      const int n_x = ((part == 1 ? per : 0) + within) * (int)args.atom;
      if (elect_one()) {
        mbar_arrive_expect_tx(fb, tx_bytes);
        tma_load_4d_hint(dst, &map_dout, fb, n_g, pc.x, pc.y, pc.ob * 128, pol_last);
        tma_load_4d_hint(dst + kWgUmmaABytes, &map_in, fb, n_x, pc.x * g.stride_w - g.pad_w,
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
    uint32_t chunk = 0;     // chunks started so far: accumulator chunk & 1
    const int chunk_steps = (int)args.chunk_steps;
    bool ok = true;
    // K-major operands, 128-byte swizzle: rows of 128 B, groups of 8 rows 1024 B apart;
    // the next 32 bytes of K are the next 32 bytes of every row (start address + 32).
    const uint64_t desc_hi = make_smem_desc(0, 0, 1024, 2u);
    while (ok && !cc.done(g)) {
      const int n_steps = cc.r_end - cc.r;
      // chunk loop around the plain kernel's step loop: a fresh accumulator per chunk
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
              tcgen05_mma<false>(d_tmem, adesc0 + (uint64_t)(2 * j), bdesc0 + (uint64_t)(2 * j),
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
      }
      if (!ok) break;
      cc.start(g, cc.item + (int)gridDim.x);
    }
    if (elect_one()) tcgen05_commit(done_bar);
    mbar_wait(done_bar, 0, args.wc, kDevTimeoutDrain);
  } else {
    // ------------------------------------------------------------ epilogue
    wgrad_chunk_epilogue_role(args, row_tab, accf_bar, acce_bar, tmem_base, warp, lane);
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
