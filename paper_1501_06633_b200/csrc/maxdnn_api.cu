// C ABI of the library (see include/maxdnn.h): descriptor checks, per-device
// state, tensor-copy descriptor encoding and kernel launches.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "../../include/maxdnn.h"
#include "bprop.cuh"
#include "ffma_conv.cuh"
#include "plan.h"
#include "umma_conv.cuh"
#include "wgrad_umma.cuh"

namespace maxdnn {
namespace {

constexpr int kMaxDevices = 64;

struct DeviceState {
  bool ready = false;
  bool sm100 = false;
  int sm_count = 0;
  uint32_t* status = nullptr;   // the status block in device memory (see WaitCtx)
  std::atomic<uint32_t> epoch{0};   // number of the latest launch that reports into it
  // "dynamic shared memory limit raised" flags, one per kernel instance: set once under
  // attr_mu, read without it afterwards
  std::mutex attr_mu;
  std::atomic<bool> ffma_attr[80];
  std::atomic<bool> umma_attr[8];
  std::atomic<bool> wgrad_attr;
  std::atomic<bool> wgrad_umma_attr[8];
  // Side streams for the strided map gradient, whose residue classes are independent
  // launches: run side by side, the tail wave of one class overlaps the next class.
  // Workspaces of the fp32 kernel's split tail, one per stream that has used one (work on
  // one stream runs in order, so its launches can share a workspace; launches on different
  // streams may overlap and must not).  Allocated on a stream's first such call.
  struct SplitWs { cudaStream_t stream; void* ptr; };
  SplitWs split_ws[8] = {};
  int n_split_ws = 0;
  std::mutex split_mu;
  cudaStream_t aux[3] = {nullptr, nullptr, nullptr};
  cudaEvent_t ev_fork = nullptr;
  cudaEvent_t ev_join[3] = {nullptr, nullptr, nullptr};
  std::mutex fork_mu;   // one fork / join sequence at a time uses the events
};

std::mutex g_mu;
DeviceState g_dev[kMaxDevices];      // static storage: every flag starts false, every epoch 0
std::atomic<uint64_t> g_launches{0};

// Raises a kernel's dynamic shared-memory limit once per device.
template <class Kern>
maxdnn_status ensure_smem_attr(DeviceState* ds, std::atomic<bool>* done, Kern kern) {
  if (done->load(std::memory_order_acquire)) return MAXDNN_OK;
  std::lock_guard<std::mutex> lk(ds->attr_mu);
  if (done->load(std::memory_order_relaxed)) return MAXDNN_OK;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
      cudaSuccess) {
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  done->store(true, std::memory_order_release);
  return MAXDNN_OK;
}

// The split-tail workspace of `stream` on this device, or null when there is none and none
// can be had now: the stream is being captured (no allocation inside a capture), all eight
// slots belong to other streams, or the allocation fails.  The caller then plans without a
// split.
void* split_workspace(DeviceState* ds, cudaStream_t stream) {
  std::lock_guard<std::mutex> lk(ds->split_mu);
  for (int i = 0; i < ds->n_split_ws; ++i)
    if (ds->split_ws[i].stream == stream) return ds->split_ws[i].ptr;
  if (ds->n_split_ws >= 8) return nullptr;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  if (cap != cudaStreamCaptureStatusNone) return nullptr;
  void* p = nullptr;
  const size_t bytes = ffma_split_bytes(ds->sm_count);
  if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  // flags start at 0; a launch's epoch is never 0
  if (cudaMemset(static_cast<uint8_t*>(p) + ffma_split_flags_offset(ds->sm_count), 0,
                 bytes - ffma_split_flags_offset(ds->sm_count)) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(p);
    return nullptr;
  }
  ds->split_ws[ds->n_split_ws].stream = stream;
  ds->split_ws[ds->n_split_ws].ptr = p;
  ++ds->n_split_ws;
  return p;
}

// The status block and a fresh epoch for one launch (never 0: word 1 of a cleared block).
WaitCtx next_wait_ctx(DeviceState* ds) {
  uint32_t e = ds->epoch.fetch_add(1, std::memory_order_relaxed) + 1;
  if (e == 0) e = ds->epoch.fetch_add(1, std::memory_order_relaxed) + 1;
  return WaitCtx{ds->status, e};
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

maxdnn_status device_state(DeviceState** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return MAXDNN_CUDA_ERROR; }
  if (dev < 0 || dev >= kMaxDevices) return MAXDNN_NOT_SUPPORTED;
  std::lock_guard<std::mutex> lk(g_mu);
  DeviceState& s = g_dev[dev];
  if (!s.ready) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
      cudaGetLastError();
      return MAXDNN_CUDA_ERROR;
    }
    s.sm100 = (prop.major == 10);
    s.sm_count = prop.multiProcessorCount;
    if (s.sm100) {
      if (cudaMalloc(&s.status, 256) != cudaSuccess) { cudaGetLastError(); return MAXDNN_CUDA_ERROR; }
      if (cudaMemset(s.status, 0, 256) != cudaSuccess) { cudaGetLastError(); return MAXDNN_CUDA_ERROR; }
      bool ok = cudaEventCreateWithFlags(&s.ev_fork, cudaEventDisableTiming) == cudaSuccess;
      for (int i = 0; i < 3 && ok; ++i)
        ok = cudaStreamCreateWithFlags(&s.aux[i], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&s.ev_join[i], cudaEventDisableTiming) == cudaSuccess;
      if (!ok) { cudaGetLastError(); return MAXDNN_CUDA_ERROR; }
    }
    s.ready = true;
  }
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) !=
            cudaSuccess || !fn) {
      cudaGetLastError();
      return MAXDNN_CUDA_ERROR;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  *out = &s;
  return MAXDNN_OK;
}

// dims[0] is the contiguous dimension; strides[i] is the byte pitch of dims[i+1].
maxdnn_status encode_map(CUtensorMap* m, CUtensorMapDataType dt, int rank, const void* base,
                         const uint64_t* dims, const uint64_t* strides, const uint32_t* box,
                         CUtensorMapSwizzle swz) {
  cuuint64_t gd[5];
  cuuint64_t gs[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides[i];
  CUresult r = g_encode(m, dt, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? MAXDNN_OK : MAXDNN_CUDA_ERROR;
}

// Element pitch of the rows / channels of the maps: the caller's, or dense.
uint64_t dims_in_h(const ConvGeom& g, int64_t given) {
  return given > 0 ? (uint64_t)given : (uint64_t)g.Wi * g.Nb;
}
uint64_t dims_in_c(const ConvGeom& g, int64_t given) {
  return given > 0 ? (uint64_t)given : (uint64_t)g.Hi * g.Wi * g.Nb;
}

size_t round256(size_t b) { return (b + 255) & ~(size_t)255; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// What a forward plan depends on: the problem, the device's SM count and the tuning
// options (their generation number: any change of any option retires every cached plan).  A call that repeats the previous call's key on the
// same thread keeps the previous plan (planning costs 1.5-4 us, a third of the host time of
// a call; small layers are launch-bound).
struct PlanKey {   // trivial: cleared with memset so that padding compares equal
  ConvDims d;
  int32_t v[8];
  bool valid;
};

bool same_plan_key(const PlanKey& a, const PlanKey& b) {
  return a.valid && b.valid && memcmp(&a.d, &b.d, sizeof(ConvDims)) == 0 &&
         memcmp(a.v, b.v, sizeof(a.v)) == 0;
}

// The plans of the last few distinct problems of this thread (a strided map gradient
// alternates between its classes' sub-problems; a network between its layers).
constexpr int kPlanSlots = 8;
template <class Args>
struct PlanCache {
  Args args[kPlanSlots];
  PlanKey key[kPlanSlots];
  int next;
  // The slot that holds `k`'s plan, or -1.
  int find(const PlanKey& k) const {
    for (int i = 0; i < kPlanSlots; ++i)
      if (same_plan_key(k, key[i])) return i;
    return -1;
  }
  // The slot to plan into: the oldest one, marked invalid until the plan succeeds.
  int take() {
    const int i = next;
    next = (next + 1) % kPlanSlots;
    key[i].valid = false;
    return i;
  }
};

template <int MR, int NR, bool FIXED, bool SPLIT, bool RAGGED = false, int LB = 4>
maxdnn_status launch_ffma(DeviceState* ds, int slot, const CUtensorMap& mf, const CUtensorMap& mi,
                          const FfmaArgs& args, cudaStream_t stream) {
  auto kern = ffma_conv_kernel<MR, NR, FIXED, SPLIT, RAGGED, LB>;
  if (ensure_smem_attr(ds, &ds->ffma_attr[slot], kern) != MAXDNN_OK) return MAXDNN_CUDA_ERROR;
  kern<<<args.g.grid, ffma_threads(MR, NR, RAGGED), args.g.smem_bytes, stream>>>(mf, mi, args);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return MAXDNN_OK;
}

// Picks the kernel instance built for the plan's tile shape: the whole-tile kernel, or
// (split) the kernel that computes the split tail.
maxdnn_status dispatch_ffma(DeviceState* ds, const CUtensorMap& mf, const CUtensorMap& mi,
                            const FfmaArgs& args, cudaStream_t stream, bool split = false) {
  const ConvGeom& g = args.g;
  const bool fx = g.fixed_pitch != 0;
  // rows per iteration of the kernel's main loop: by block shape and step length
  const bool long_steps = g.rows >= 96;
#define MAXDNN_FFMA_LAUNCH(MR, NR, LB, SLOT)                                                        \
  do {                                                                                              \
    if (split)                                                                                      \
      return fx ? launch_ffma<MR, NR, true, true, false, LB>(ds, (SLOT) + 16, mf, mi, args, stream)   \
                : launch_ffma<MR, NR, false, true, false, LB>(ds, (SLOT) + 17, mf, mi, args, stream); \
    return fx ? launch_ffma<MR, NR, true, false, false, LB>(ds, (SLOT), mf, mi, args, stream)       \
              : launch_ffma<MR, NR, false, false, false, LB>(ds, (SLOT) + 1, mf, mi, args, stream); \
  } while (0)
#define MAXDNN_FFMA_CASE(M, C, MR, NR, SLOT)                                               \
  if (g.tile_m == (M) && g.tile_cols == (C)) {                                             \
    if (ffma_long_block(MR, NR, true) != ffma_long_block(MR, NR, false) && long_steps)     \
      MAXDNN_FFMA_LAUNCH(MR, NR, ffma_long_block(MR, NR, true), (SLOT) + 40);              \
    MAXDNN_FFMA_LAUNCH(MR, NR, ffma_long_block(MR, NR, false), (SLOT));                    \
  }
  MAXDNN_FFMA_CASE(256, 128, 16, 8, 0)
  MAXDNN_FFMA_CASE(128, 256, 8, 16, 2)
  MAXDNN_FFMA_CASE(96, 256, 6, 16, 4)
  MAXDNN_FFMA_CASE(128, 128, 8, 8, 6)
  MAXDNN_FFMA_CASE(96, 128, 6, 8, 8)
  MAXDNN_FFMA_CASE(64, 128, 4, 8, 10)
  MAXDNN_FFMA_CASE(64, 256, 4, 16, 14)
  MAXDNN_FFMA_CASE(32, 128, 2, 8, 12)
#undef MAXDNN_FFMA_CASE
#undef MAXDNN_FFMA_LAUNCH
  return MAXDNN_NOT_SUPPORTED;
}

// The ragged kernel's instances (tiles of 128 columns, up to 128 filters).
maxdnn_status dispatch_ffma_ragged(DeviceState* ds, const CUtensorMap& mf, const CUtensorMap& mi,
                                   const FfmaArgs& args, cudaStream_t stream) {
  const ConvGeom& g = args.g;
  if (g.tile_cols != 128 || g.fixed_pitch) return MAXDNN_NOT_SUPPORTED;
  if (g.tile_m == 128) return launch_ffma<8, 8, false, false, true>(ds, 32, mf, mi, args, stream);
  if (g.tile_m == 64) return launch_ffma<4, 8, false, false, true>(ds, 33, mf, mi, args, stream);
  if (g.tile_m == 32) return launch_ffma<2, 8, false, false, true>(ds, 34, mf, mi, args, stream);
  return MAXDNN_NOT_SUPPORTED;
}

// The one or two launches of a plan: whole tiles, then (if the plan splits its last wave)
// the split tail on the same stream.  `args` is modified (tile range) and restored.
maxdnn_status launch_ffma_plan(DeviceState* ds, const CUtensorMap& mf, const CUtensorMap& mi,
                               FfmaArgs& args, cudaStream_t stream) {
  ConvGeom& g = args.g;
  if (g.sk_tiles <= 0) return dispatch_ffma(ds, mf, mi, args, stream);
  const int32_t begin = g.tile_begin, end = g.tile_end;
  maxdnn_status st = MAXDNN_OK;
  if (g.sk_first > begin) {
    g.tile_end = g.sk_first;
    st = dispatch_ffma(ds, mf, mi, args, stream);
    g.tile_end = end;
  }
  if (st == MAXDNN_OK) {
    g.tile_begin = g.sk_first;         // the split kernel's items start at the first split tile
    st = dispatch_ffma(ds, mf, mi, args, stream, true);
    g.tile_begin = begin;
  }
  return st;
}

// ragged: Nb / No need not be multiples of 4 (the kernel with copy warps instead of bulk
// tensor copies); the tensors then only have to be 4-byte aligned.
maxdnn_status fprop_fp32(const ConvDims& cd, const float* in, const float* filt, float* out,
                         cudaStream_t stream, bool ragged = false) {
  int32_t Ho, Wo;
  maxdnn_status st = check_dims(cd, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  if (cd.out_x_stride != 0) return MAXDNN_INVALID_VALUE;   // this kernel writes dense results only
  if (!in || !filt || !out) return MAXDNN_INVALID_VALUE;
  if (!aligned16(in) || !aligned16(filt) || !aligned16(out)) return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;

  // A plan may split its tail wave along K when this stream has (or can get) a workspace.
  void* split_ws = (option(OPT_FFMA_STREAMK, 1) != 0 && !ragged) ? split_workspace(ds, stream) : nullptr;
  static thread_local PlanCache<FfmaArgs> cache;   // 4 KB tables: kept off the stack
  PlanKey key;
  memset(&key, 0, sizeof(key));
  key.d = cd;
  key.v[0] = ds->sm_count;
  key.v[1] = (int32_t)options_generation();
  key.v[2] = split_ws != nullptr;
  key.v[3] = ragged;
  key.valid = true;
  int slot = cache.find(key);
  if (slot < 0) {
    slot = cache.take();
    st = plan_ffma(cd, ds->sm_count, option(OPT_FFMA_TILE_M), option(OPT_FFMA_COLS),
                   &cache.args[slot].g, &cache.args[slot].table, split_ws != nullptr, ragged);
    if (st != MAXDNN_OK) return st;
    cache.key[slot] = key;
  }
  FfmaArgs& args = cache.args[slot];
  args.out = out;
  args.sk_partial = static_cast<float*>(split_ws);
  args.sk_flags = split_ws ? reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(split_ws) +
                                                         ffma_split_flags_offset(ds->sm_count))
                           : nullptr;
  args.wc = next_wait_ctx(ds);
  args.test_missing_arrival = (uint32_t)option(OPT_TEST_MISSING_ARRIVAL);   // see FfmaArgs
  args.clock_stamp = (uint32_t)option(OPT_KERNEL_CLOCK);
  if (args.clock_stamp != 0 &&
      cudaMemsetAsync(ds->status + 2, 0, 16, stream) != cudaSuccess) {   // this call's maxima
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  const ConvGeom& g = args.g;
  args.in = in;
  args.filt = filt;

  CUtensorMap mf, mi;
  if (ragged) {
    if (cd.in_h_stride != 0 || cd.in_c_stride != 0) return MAXDNN_INVALID_VALUE;   // dense maps only
    memset(&mf, 0, sizeof(mf));       // the copy warps read the tensors directly
    memset(&mi, 0, sizeof(mi));
  }
  if (!ragged || g.No % 4 == 0) {
    // filter bank as (o, kw, c, kh): a box lands as [kh][c][kw][o]
    const uint64_t dims[4] = {(uint64_t)g.No, (uint64_t)g.Skw, (uint64_t)g.Nc, (uint64_t)g.Skh};
    const uint64_t str[3] = {(uint64_t)g.No * 4, (uint64_t)g.Skh * g.Skw * g.No * 4,
                             (uint64_t)g.Skw * g.No * 4};
    const uint32_t box[4] = {(uint32_t)g.tile_m, (uint32_t)g.kwc, (uint32_t)g.kc, (uint32_t)g.box_kh};
    st = encode_map(&mf, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, filt, dims, str, box,
                    CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st != MAXDNN_OK) return st;
  }
  if (ragged) return dispatch_ffma_ragged(ds, mf, mi, args, stream);
  {
    // maps as (n, w, c, h): a box lands as [h][c][w][n]
    const uint64_t dims[4] = {(uint64_t)g.Nb, (uint64_t)g.Wi, (uint64_t)g.Nc, (uint64_t)g.Hi};
    const uint64_t hs = dims_in_h(g, cd.in_h_stride), cs = dims_in_c(g, cd.in_c_stride);
    const uint64_t str[3] = {(uint64_t)g.Nb * 4, cs * 4, hs * 4};
    const uint32_t box[4] = {(uint32_t)g.tile_n, (uint32_t)g.b_box_w, (uint32_t)g.kc, (uint32_t)g.box_kh};
    st = encode_map(&mi, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, in, dims, str, box,
                    CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st != MAXDNN_OK) return st;
  }
  return launch_ffma_plan(ds, mf, mi, args, stream);
}

maxdnn_status fprop_fp32(const maxdnn_conv_desc* desc, const float* in, const float* filt,
                         float* out, cudaStream_t stream) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  return fprop_fp32(dims_from(*desc), in, filt, out, stream);
}

// One launch of the tensor-core forward kernel: one-SM or two-SM tiles (a cluster of two
// CTAs), K in one accumulator or summed in chunks.
template <bool BF16, bool PAIR, bool CHUNK>
maxdnn_status launch_umma(DeviceState* ds, const CUtensorMap& mf, const CUtensorMap& mi,
                          const CUtensorMap& mo, const UmmaArgs& args, cudaStream_t stream) {
  auto kern = umma_conv_kernel<BF16, PAIR, CHUNK>;
  const int slot = (BF16 ? 1 : 0) + (PAIR ? 2 : 0) + (CHUNK ? 4 : 0);
  if (ensure_smem_attr(ds, &ds->umma_attr[slot], kern) != MAXDNN_OK) return MAXDNN_CUDA_ERROR;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)args.g.grid, 1, 1);
  cfg.blockDim = dim3(umma_threads(CHUNK), 1, 1);
  cfg.dynamicSmemBytes = (size_t)args.g.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = PAIR ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = PAIR ? 1 : 0;
  if (cudaLaunchKernelEx(&cfg, kern, mf, mi, mo, args) != cudaSuccess) {
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return MAXDNN_OK;
}

// One launch of the tensor-core filter-gradient kernel.
template <bool BF16, bool PAIR, bool CHUNK>
maxdnn_status launch_wgrad_umma(DeviceState* ds, const CUtensorMap& mg, const CUtensorMap& mi,
                                const WgradUmmaArgs& args, cudaStream_t stream) {
  auto kern = wgrad_umma_kernel<BF16, PAIR, CHUNK>;
  const int slot = (BF16 ? 1 : 0) + (PAIR ? 2 : 0) + (CHUNK ? 4 : 0);
  if (ensure_smem_attr(ds, &ds->wgrad_umma_attr[slot], kern) != MAXDNN_OK) return MAXDNN_CUDA_ERROR;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)args.g.grid, 1, 1);
  cfg.blockDim = dim3(wgrad_umma_threads(CHUNK), 1, 1);
  cfg.dynamicSmemBytes = (size_t)args.g.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = PAIR ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = PAIR ? 1 : 0;
  if (cudaLaunchKernelEx(&cfg, kern, mg, mi, args) != cudaSuccess) {
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  return MAXDNN_OK;
}

// chunk_rows > 0 (TF32 only): the chunked kernels, a fresh accumulator about every
// chunk_rows rows of K.
maxdnn_status fprop_umma(const ConvDims& cd, int elem_bytes, const void* in, const void* filt,
                         float* out, cudaStream_t stream, int chunk_rows = 0) {
  int32_t Ho, Wo;
  maxdnn_status st = check_dims(cd, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  if (!in || !filt || !out) return MAXDNN_INVALID_VALUE;
  if (!aligned16(in) || !aligned16(filt) || !aligned16(out)) return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;

  static thread_local PlanCache<UmmaArgs> cache;
  PlanKey key;
  memset(&key, 0, sizeof(key));
  key.d = cd;
  key.v[0] = ds->sm_count;
  key.v[1] = elem_bytes;
  key.v[2] = (int32_t)options_generation();
  key.valid = true;
  int slot = cache.find(key);
  if (slot < 0) {
    slot = cache.take();
    st = plan_umma(cd, elem_bytes, ds->sm_count, option(OPT_UMMA_KC), option(OPT_UMMA_PAIR),
                   &cache.args[slot].g, &cache.args[slot].table);
    if (st != MAXDNN_OK) return st;
    cache.key[slot] = key;
  }
  UmmaArgs& args = cache.args[slot];
  const ConvGeom& g = args.g;
  const uint64_t eb = (uint64_t)elem_bytes;
  const uint32_t atom = 128u / (uint32_t)elem_bytes;
  const bool bf16 = elem_bytes == 2;
  args.wc = next_wait_ctx(ds);
  args.atom = atom;
  args.umma_k = 32u / (uint32_t)elem_bytes;
  args.is_bf16 = bf16 ? 1u : 0u;
  args.test_missing_arrival = (uint32_t)option(OPT_TEST_MISSING_ARRIVAL);   // see UmmaArgs
  // Staged layouts: filters [group of 32/64][kw][channel][128 B], patches
  // [pixel][image group][channel][128 B].
  args.lbo_a_bytes = (uint32_t)(g.kwc * g.kc) * 128u;
  args.lbo_b_bytes = (uint32_t)g.kc * 128u;
  args.tap_a_bytes = (uint32_t)g.kc * 128u;
  args.tap_b_bytes = (uint32_t)(g.cta_n / (int)atom) * (uint32_t)g.kc * 128u;
  if (g.box_c != g.kc) {
    // few-channel plan (filter columns merged into K): a pixel's window starts
    // b_slot_bytes after its neighbour's (its own box, or a shift inside the one strip);
    // with the strip the MMA warp's outer loop walks the filter rows of the step, which
    // are one strip row (patches) / one box row (filters) apart
    args.lbo_b_bytes = (uint32_t)g.b_slot_bytes;
    args.tap_b_bytes = (uint32_t)(g.b_box_w * g.box_c) * 128u;
  }
  // next group of channel rows: 8 rows for the 16-byte-chunk swizzle, 4 rows for the
  // 32-byte-chunk swizzle of 4-byte operands
  args.sbo_bytes = bf16 ? 1024u : 512u;
  args.kstep_bytes = args.umma_k * 128u;      // next MMA along K inside a stage
  const uint32_t n_cols = (uint32_t)(g.tile_px * g.tile_n);
  const uint32_t fmt = bf16 ? 1u : 2u;        // operand format: bf16 / tf32
  args.idesc = (1u << 4)                      // fp32 accumulator
               | (fmt << 7) | (fmt << 10)     // A and B formats
               | (1u << 15) | (1u << 16)      // both operands contiguous along M / N, not K
               | ((n_cols >> 3) << 17) | ((uint32_t)(g.tile_m >> 4) << 24);
  const CUtensorMapDataType dt =
      bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;

  // 4-byte operands use the 128-byte swizzle with 32-byte chunks, 2-byte operands the
  // one with 16-byte chunks (the patterns the MMA descriptors of each kind read).
  const CUtensorMapSwizzle op_swz =
      bf16 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B;
  CUtensorMap mf, mi, mo;
  {
    // filter bank as (o, c, kw, kh); one box = 128 bytes of filters x kc channels of a tap
    const uint64_t dims[4] = {(uint64_t)g.No, (uint64_t)g.Nc, (uint64_t)g.Skw, (uint64_t)g.Skh};
    const uint64_t str[3] = {(uint64_t)g.Skh * g.Skw * g.No * eb, (uint64_t)g.No * eb,
                             (uint64_t)g.Skw * g.No * eb};
    const uint32_t box[4] = {atom, (uint32_t)g.box_c, (uint32_t)g.box_kw, (uint32_t)g.box_kh};
    st = encode_map(&mf, dt, 4, filt, dims, str, box, op_swz);
    if (st != MAXDNN_OK) return st;
  }
  {
    // maps as (n within group, c, n group, w, h): shared memory receives
    // [pixel][image group][channel][128 bytes of images]
    const uint64_t dims[5] = {atom, (uint64_t)g.Nc, (uint64_t)g.Nb / atom, (uint64_t)g.Wi,
                              (uint64_t)g.Hi};
    const uint64_t str[4] = {dims_in_c(g, cd.in_c_stride) * eb, 128u, (uint64_t)g.Nb * eb,
                             dims_in_h(g, cd.in_h_stride) * eb};
    const uint32_t box[5] = {atom, (uint32_t)g.box_c, (uint32_t)g.cta_n / atom, (uint32_t)g.b_box_w,
                             (uint32_t)g.box_kh};
    st = encode_map(&mi, dt, 5, in, dims, str, box, op_swz);
    if (st != MAXDNN_OK) return st;
  }
  {
    // output as (n, x, y, o): one store = 32 filters x 32 images
    const uint64_t dims[4] = {(uint64_t)g.Nb, (uint64_t)g.Wo, (uint64_t)g.Ho, (uint64_t)g.No};
    const bool sub = cd.out_x_stride > 0;     // the result is a sub-grid of a larger tensor
    const uint64_t str[3] = {(sub ? (uint64_t)cd.out_x_stride : (uint64_t)g.Nb) * 4,
                             (sub ? (uint64_t)cd.out_y_stride : (uint64_t)g.Wo * g.Nb) * 4,
                             (sub ? (uint64_t)cd.out_o_stride : (uint64_t)g.Ho * g.Wo * g.Nb) * 4};
    const uint32_t box[4] = {32u, 1u, 1u, 32u};
    st = encode_map(&mo, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, out, dims, str, box,
                    CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != MAXDNN_OK) return st;
  }
  if (chunk_rows > 0) {
    if (bf16) return MAXDNN_INVALID_VALUE;
    const int steps = chunk_rows / g.rows;
    args.chunk_steps = (uint32_t)(steps < 1 ? 1 : steps);
    return g.pair ? launch_umma<false, true, true>(ds, mf, mi, mo, args, stream)
                  : launch_umma<false, false, true>(ds, mf, mi, mo, args, stream);
  }
  if (g.pair)
    return bf16 ? launch_umma<true, true, false>(ds, mf, mi, mo, args, stream)
                : launch_umma<false, true, false>(ds, mf, mi, mo, args, stream);
  return bf16 ? launch_umma<true, false, false>(ds, mf, mi, mo, args, stream)
              : launch_umma<false, false, false>(ds, mf, mi, mo, args, stream);
}

maxdnn_status fprop_umma(const maxdnn_conv_desc* desc, int elem_bytes, const void* in,
                         const void* filt, float* out, cudaStream_t stream) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  return fprop_umma(dims_from(*desc), elem_bytes, in, filt, out, stream);
}

// ---------------------------------------------------------------------------
// Backward propagation.
// ---------------------------------------------------------------------------
bool kind_ok(maxdnn_kernel_kind k) {
  return k == MAXDNN_KERNEL_FP32 || k == MAXDNN_KERNEL_TF32 || k == MAXDNN_KERNEL_BF16;
}

// Checks that the forward kernel of `kind` takes the transposed problem.
maxdnn_status dgrad_plan_check(const ConvDims& fd, maxdnn_kernel_kind kind, int sm_count) {
  static thread_local ConvGeom g;
  static thread_local KStepTable t;
  if (kind == MAXDNN_KERNEL_FP32)
    return plan_ffma(fd, sm_count, option(OPT_FFMA_TILE_M), option(OPT_FFMA_COLS), &g, &t);
  return plan_umma(fd, kind == MAXDNN_KERNEL_BF16 ? 2 : 4, sm_count, option(OPT_UMMA_KC),
                   option(OPT_UMMA_PAIR), &g, &t);
}

// Workspace of the strided map gradient.  The classes run side by side, so each has its
// own region: its transformed sub-filter bank (together the classes' banks hold every tap
// once) and, for the fp32 kernel, its dense result (together: one din), each rounded up
// to 256 bytes.
struct DgradStridedPlan {
  size_t ft_bytes, sub_bytes, pre_bytes;
};

inline size_t dgrad_class_ft_bytes(const ConvDims& d, const DgradAxis& ah, const DgradAxis& aw,
                                   size_t eb) {
  return round256((size_t)d.No * ah.J * aw.J * d.Nc * eb);
}
inline size_t dgrad_class_sub_bytes(const ConvDims& d, const DgradAxis& ah, const DgradAxis& aw) {
  return round256((size_t)d.Nc * ah.n * aw.n * d.Nb * 4);
}
// A class takes part when it has positions and taps and its windows reach dout.
inline bool dgrad_class_live(const DgradAxis& ah, const DgradAxis& aw, int Ho, int Wo) {
  return ah.J > 0 && aw.J > 0 && ah.n > 0 && aw.n > 0 && ah.crop < Ho && aw.crop < Wo;
}

// x3 (three-product TF32 mode, kind = TF32): the gradient is split once into [hi; hi; lo]
// along its channels (pre_bytes, ahead of everything else in the workspace) and every class's
// bank is followed by its split [hi; lo; hi] (four times the bank in all).
maxdnn_status plan_dgrad_strided(const ConvDims& d, maxdnn_kernel_kind kind, DgradStridedPlan* p,
                                 bool x3 = false) {
  int32_t Ho, Wo;
  maxdnn_status st = check_dims(d, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  const size_t eb = kind == MAXDNN_KERNEL_BF16 ? 2 : 4;
  p->ft_bytes = p->sub_bytes = 0;
  p->pre_bytes = x3 ? round256((size_t)3 * d.No * Ho * Wo * d.Nb * 4) : 0;
  for (int rh = 0; rh < d.stride_h; ++rh)
    for (int rw = 0; rw < d.stride_w; ++rw) {
      const DgradAxis ah = dgrad_axis(rh, d.Skh, d.stride_h, d.pad_h, d.Hi);
      const DgradAxis aw = dgrad_axis(rw, d.Skw, d.stride_w, d.pad_w, d.Wi);
      if (!dgrad_class_live(ah, aw, Ho, Wo)) continue;
      p->ft_bytes += dgrad_class_ft_bytes(d, ah, aw, eb) * (x3 ? 4 : 1);
      if (kind == MAXDNN_KERNEL_FP32) p->sub_bytes += dgrad_class_sub_bytes(d, ah, aw);
    }
  return MAXDNN_OK;
}


maxdnn_status bprop_data_strided(const ConvDims& d, maxdnn_kernel_kind kind, const void* dout,
                                 const void* filt, float* din, void* ws, size_t ws_bytes,
                                 cudaStream_t stream, bool x3 = false) {
  const size_t eb = kind == MAXDNN_KERNEL_BF16 ? 2 : 4;
  DgradStridedPlan p;
  maxdnn_status st = plan_dgrad_strided(d, kind, &p, x3);
  if (st != MAXDNN_OK) return st;
  if (ws_bytes < p.pre_bytes + p.ft_bytes + p.sub_bytes) return MAXDNN_INVALID_VALUE;
  if (d.Nb % 4 != 0) return MAXDNN_NOT_SUPPORTED;
  DeviceState* ds = nullptr;
  st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;
  int32_t Ho, Wo;
  check_dims(d, &Ho, &Wo);
  const int sh = d.stride_h, sw = d.stride_w;
  // The FPROP that computes one residue class (dense result; the caller adds output pitches).
  auto class_dims = [&](const DgradAxis& ah, const DgradAxis& aw) {
    ConvDims fd;
    fd.Nb = d.Nb; fd.Wi = Wo - aw.crop; fd.Hi = Ho - ah.crop; fd.Nc = x3 ? 3 * d.No : d.No;
    fd.No = d.Nc; fd.Skw = aw.J; fd.Skh = ah.J; fd.stride_w = fd.stride_h = 1;
    fd.pad_w = aw.pad; fd.pad_h = ah.pad; fd.alpha = d.alpha;
    fd.in_h_stride = (int64_t)Wo * d.Nb;
    fd.in_c_stride = (int64_t)Ho * Wo * d.Nb;
    fd.Ho_given = ah.n; fd.Wo_given = aw.n;
    fd.out_x_stride = fd.out_y_stride = fd.out_o_stride = 0;
    return fd;
  };
  // Nothing is launched unless every class has a plan (its FPROP has No' = Nc filters: the
  // 16-byte row rule can refuse it) and the split kernels cover whole 16-byte groups.
  if (x3 && (((size_t)d.No * Ho * Wo * d.Nb) % 4 != 0 || 3 * (int64_t)d.No > 32767))
    return MAXDNN_NOT_SUPPORTED;
  for (int rh = 0; rh < sh; ++rh)
    for (int rw = 0; rw < sw; ++rw) {
      const DgradAxis ah = dgrad_axis(rh, d.Skh, sh, d.pad_h, d.Hi);
      const DgradAxis aw = dgrad_axis(rw, d.Skw, sw, d.pad_w, d.Wi);
      if (!dgrad_class_live(ah, aw, Ho, Wo)) continue;
      if (x3 && ((size_t)d.No * ah.J * aw.J * d.Nc) % 4 != 0) return MAXDNN_NOT_SUPPORTED;
      st = dgrad_plan_check(class_dims(ah, aw), kind, ds->sm_count);
      if (st != MAXDNN_OK) return st;
    }
  uint8_t* ft_next = static_cast<uint8_t*>(ws) + p.pre_bytes;
  uint8_t* sub_next = ft_next + p.ft_bytes;
  if (x3) {
    // the gradient as [hi; hi; lo] along its channels, once, ahead of the fork
    const size_t n4 = (size_t)d.No * Ho * Wo * d.Nb / 4;
    tf32_split3_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, stream>>>(
        static_cast<const float4*>(dout), static_cast<float4*>(ws), n4, 0x4u);
    if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    dout = ws;
  }
  // Positions that no tap reaches (a class without taps, or whose window lies outside
  // dout) must read zero: clear din first if there is such a class.
  bool all_covered = true;
  for (int rh = 0; rh < sh; ++rh)
    for (int rw = 0; rw < sw; ++rw) {
      const DgradAxis ah = dgrad_axis(rh, d.Skh, sh, d.pad_h, d.Hi);
      const DgradAxis aw = dgrad_axis(rw, d.Skw, sw, d.pad_w, d.Wi);
      if (ah.n == 0 || aw.n == 0) continue;                     // no positions: nothing to cover
      if (ah.J == 0 || aw.J == 0 || ah.crop >= Ho || aw.crop >= Wo) all_covered = false;
    }
  if (!all_covered &&
      cudaMemsetAsync(din, 0, (size_t)d.Nc * d.Hi * d.Wi * d.Nb * 4, stream) != cudaSuccess) {
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  // The tensor-core kernels store through a tensor map, which can address the class's
  // grid inside din directly; the fp32 kernel writes a dense scratch tensor that a copy
  // kernel scatters.
  const bool direct = kind != MAXDNN_KERNEL_FP32;
  // Fork: class i runs on the caller's stream (i % 4 == 0) or on one of three side
  // streams that wait for what the caller's stream has queued so far; join at the end.
  std::lock_guard<std::mutex> fork_lock(ds->fork_mu);
  if (cudaEventRecord(ds->ev_fork, stream) != cudaSuccess) { cudaGetLastError(); return MAXDNN_CUDA_ERROR; }
  bool aux_used[3] = {false, false, false};
  int class_index = 0;
  maxdnn_status result = MAXDNN_OK;
  for (int rh = 0; rh < sh && result == MAXDNN_OK; ++rh) {
    for (int rw = 0; rw < sw && result == MAXDNN_OK; ++rw) {
      const DgradAxis ah = dgrad_axis(rh, d.Skh, sh, d.pad_h, d.Hi);
      const DgradAxis aw = dgrad_axis(rw, d.Skw, sw, d.pad_w, d.Wi);
      if (!dgrad_class_live(ah, aw, Ho, Wo)) continue;
      uint8_t* w_ft = ft_next;
      ft_next += dgrad_class_ft_bytes(d, ah, aw, eb) * (x3 ? 4 : 1);
      float* w_sub = reinterpret_cast<float*>(sub_next);
      if (!direct) sub_next += dgrad_class_sub_bytes(d, ah, aw);
      const int lane = class_index++ % 4;
      cudaStream_t cs = stream;
      if (lane > 0) {
        cs = ds->aux[lane - 1];
        if (!aux_used[lane - 1]) {
          if (cudaStreamWaitEvent(cs, ds->ev_fork, 0) != cudaSuccess) { cudaGetLastError(); result = MAXDNN_CUDA_ERROR; break; }
          aux_used[lane - 1] = true;
        }
      }
      ConvDims fd = class_dims(ah, aw);
      const dim3 grid((unsigned)ceil_div(d.No, 32), (unsigned)ceil_div(d.Nc, 32),
                      (unsigned)(ah.J * aw.J));
      const dim3 block(32, 8);
      if (eb == 2)
        subfilter_flip_transpose_kernel<uint16_t><<<grid, block, 0, cs>>>(
            static_cast<const uint16_t*>(filt), reinterpret_cast<uint16_t*>(w_ft), d.Nc, d.Skh,
            d.Skw, d.No, sh, sw, ah.rho, aw.rho, ah.J, aw.J);
      else
        subfilter_flip_transpose_kernel<float><<<grid, block, 0, cs>>>(
            static_cast<const float*>(filt), reinterpret_cast<float*>(w_ft), d.Nc, d.Skh, d.Skw,
            d.No, sh, sw, ah.rho, aw.rho, ah.J, aw.J);
      if (cudaGetLastError() != cudaSuccess) { result = MAXDNN_CUDA_ERROR; break; }
      g_launches.fetch_add(1, std::memory_order_relaxed);
      const uint8_t* src = static_cast<const uint8_t*>(dout) +
                           ((size_t)ah.crop * Wo + aw.crop) * d.Nb * eb;
      if (direct) {
        fd.out_x_stride = (int64_t)sw * d.Nb;
        fd.out_y_stride = (int64_t)sh * d.Wi * d.Nb;
        fd.out_o_stride = (int64_t)d.Hi * d.Wi * d.Nb;
        float* dst = din + ((size_t)ah.first * d.Wi + aw.first) * d.Nb;
        if (x3) {
          // the class's bank as [hi; lo; hi] along its channels (the gradient's filters),
          // then the chunked TF32 kernels on the problem with 3 No channels
          const size_t n4 = (size_t)d.No * ah.J * aw.J * d.Nc / 4;
          float* w_ft3 = reinterpret_cast<float*>(w_ft + dgrad_class_ft_bytes(d, ah, aw, eb));
          tf32_split3_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, cs>>>(
              reinterpret_cast<const float4*>(w_ft), reinterpret_cast<float4*>(w_ft3), n4, 0x2u);
          if (cudaGetLastError() != cudaSuccess) { result = MAXDNN_CUDA_ERROR; break; }
          g_launches.fetch_add(1, std::memory_order_relaxed);
          result = fprop_umma(fd, 4, src, w_ft3, dst, cs, option(OPT_X3_CHUNK_ROWS, 768));
          continue;
        }
        result = fprop_umma(fd, (int)eb, src, w_ft, dst, cs);
        continue;
      }
      result = fprop_fp32(fd, reinterpret_cast<const float*>(src), reinterpret_cast<const float*>(w_ft),
                          w_sub, cs);
      if (result != MAXDNN_OK) break;
      const int nb4 = d.Nb / 4;
      const size_t total = (size_t)d.Nc * ah.n * aw.n * nb4;
      dgrad_scatter_kernel<<<(unsigned)((total + 255) / 256), 256, 0, cs>>>(
          reinterpret_cast<const float4*>(w_sub), reinterpret_cast<float4*>(din), d.Nc, ah.n, aw.n,
          nb4, d.Hi, d.Wi, sh, sw, ah.first, aw.first);
      if (cudaGetLastError() != cudaSuccess) { result = MAXDNN_CUDA_ERROR; break; }
      g_launches.fetch_add(1, std::memory_order_relaxed);
    }
  }
  // Join, also after an error: the caller's stream must not run ahead of the side streams.
  for (int i = 0; i < 3; ++i) {
    if (!aux_used[i]) continue;
    if (cudaEventRecord(ds->ev_join[i], ds->aux[i]) != cudaSuccess ||
        cudaStreamWaitEvent(stream, ds->ev_join[i], 0) != cudaSuccess) {
      cudaGetLastError();
      if (result == MAXDNN_OK) result = MAXDNN_CUDA_ERROR;
    }
  }
  return result;
}


maxdnn_status bprop_data(const ConvDims& d, maxdnn_kernel_kind kind, const void* dout,
                         const void* filt, float* din, void* ws, size_t ws_bytes,
                         cudaStream_t stream) {
  if (!kind_ok(kind)) return MAXDNN_INVALID_VALUE;
  maxdnn_status st = check_dims(d, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  if (!dout || !filt || !din || !ws) return MAXDNN_INVALID_VALUE;
  if (!aligned16(dout) || !aligned16(filt) || !aligned16(din) || !aligned16(ws))
    return MAXDNN_INVALID_VALUE;
  if (d.stride_w != 1 || d.stride_h != 1)
    return bprop_data_strided(d, kind, dout, filt, din, ws, ws_bytes, stream);
  ConvDims fd;
  st = plan_dgrad(d, &fd);
  if (st != MAXDNN_OK) return st;
  const size_t eb = kind == MAXDNN_KERNEL_BF16 ? 2 : 4;
  const int taps = d.Skh * d.Skw;
  const size_t need = (size_t)d.Nc * taps * d.No * eb;
  if (ws_bytes < need) return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;
  st = dgrad_plan_check(fd, kind, ds->sm_count);
  if (st != MAXDNN_OK) return st;
  const dim3 grid((unsigned)ceil_div(d.No, 32), (unsigned)ceil_div(d.Nc, 32), (unsigned)taps);
  const dim3 block(32, 8);
  if (eb == 2)
    flip_transpose_kernel<uint16_t><<<grid, block, 0, stream>>>(
        static_cast<const uint16_t*>(filt), static_cast<uint16_t*>(ws), d.Nc, taps, d.No);
  else
    flip_transpose_kernel<float><<<grid, block, 0, stream>>>(
        static_cast<const float*>(filt), static_cast<float*>(ws), d.Nc, taps, d.No);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (kind == MAXDNN_KERNEL_FP32)
    return fprop_fp32(fd, static_cast<const float*>(dout), static_cast<const float*>(ws), din, stream);
  return fprop_umma(fd, (int)eb, dout, ws, din, stream);
}

maxdnn_status bprop_data_workspace(const ConvDims& d, maxdnn_kernel_kind kind, size_t* bytes) {
  if (!bytes || !kind_ok(kind)) return MAXDNN_INVALID_VALUE;
  maxdnn_status st = check_dims(d, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  const size_t eb = kind == MAXDNN_KERNEL_BF16 ? 2 : 4;
  if (d.stride_w != 1 || d.stride_h != 1) {
    DgradStridedPlan p;
    st = plan_dgrad_strided(d, kind, &p);
    if (st != MAXDNN_OK) return st;
    *bytes = p.ft_bytes + p.sub_bytes;
    return MAXDNN_OK;
  }
  ConvDims fd;
  st = plan_dgrad(d, &fd);
  if (st != MAXDNN_OK) return st;
  *bytes = (size_t)d.Nc * d.Skh * d.Skw * d.No * eb;
  return MAXDNN_OK;
}

maxdnn_status bprop_filter(const ConvDims& d, maxdnn_kernel_kind kind, const void* in,
                           const void* dout, float* dfilt, void* ws, size_t ws_bytes,
                           cudaStream_t stream) {
  if (!kind_ok(kind)) return MAXDNN_INVALID_VALUE;
  maxdnn_status st = check_dims(d, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  if (!in || !dout || !dfilt) return MAXDNN_INVALID_VALUE;
  if (!aligned16(in) || !aligned16(dout) || !aligned16(dfilt) || !aligned16(ws))
    return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;
  const bool tensor = kind != MAXDNN_KERNEL_FP32;
  const bool bf16 = kind == MAXDNN_KERNEL_BF16;
  const int eb = bf16 ? 2 : 4;
  static thread_local WgradArgs fargs;
  static thread_local WgradUmmaArgs uargs;
  WgradGeom& g = tensor ? uargs.g : fargs.g;
  st = plan_wgrad(d, tensor ? eb : 0, ds->sm_count, option(OPT_WGRAD_SPLITS), &g,
                  option(OPT_WGRAD_PAIR));
  if (st != MAXDNN_OK) return st;
  const size_t kno = (size_t)g.Nc * g.Skh * g.Skw * g.No;
  const size_t need = g.splits > 1 ? (size_t)g.splits * kno * 4 : 0;
  if (need > 0 && (!ws || ws_bytes < need)) return MAXDNN_INVALID_VALUE;
  const CUtensorMapDataType dt =
      bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  const uint32_t chunk = 128u / (uint32_t)eb;     // images per reduction step = one 128-byte row
  CUtensorMap mg, mi;
  {
    // output gradient as (n, x, y, o): one box = 128 bytes of images of one pixel x the tile's filters
    const uint64_t dims[4] = {(uint64_t)g.Nb, (uint64_t)g.Wo, (uint64_t)g.Ho, (uint64_t)g.No};
    const uint64_t str[3] = {(uint64_t)g.Nb * eb, (uint64_t)g.Wo * g.Nb * eb,
                             (uint64_t)g.Ho * g.Wo * g.Nb * eb};
    const uint32_t box[4] = {chunk, 1u, 1u, (uint32_t)g.box_o};
    st = encode_map(&mg, dt, 4, dout, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != MAXDNN_OK) return st;
  }
  {
    // maps as (n, w, h, c): one box = 128 bytes of images of a bh x bw window of pixels x bc channels
    const uint64_t dims[4] = {(uint64_t)g.Nb, (uint64_t)g.Wi, (uint64_t)g.Hi, (uint64_t)g.Nc};
    const uint64_t str[3] = {(uint64_t)g.Nb * eb, (uint64_t)g.Wi * g.Nb * eb,
                             (uint64_t)g.Hi * g.Wi * g.Nb * eb};
    // (a pair's CTA stages half of the tile's channels)
    const uint32_t box[4] = {chunk, (uint32_t)g.bw, (uint32_t)g.bh,
                             (uint32_t)(g.pair ? g.bc_h : g.bc)};
    st = encode_map(&mi, dt, 4, in, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != MAXDNN_OK) return st;
  }
  if (!tensor) {
    fargs.dfilt = dfilt;
    fargs.partial = static_cast<float*>(ws);
    fargs.wc = next_wait_ctx(ds);
    if (ensure_smem_attr(ds, &ds->wgrad_attr, wgrad_kernel) != MAXDNN_OK) return MAXDNN_CUDA_ERROR;
    wgrad_kernel<<<g.grid, kWgThreads, g.smem_bytes, stream>>>(mg, mi, fargs);
  } else {
    uargs.dfilt = dfilt;
    uargs.partial = static_cast<float*>(ws);
    uargs.wc = next_wait_ctx(ds);
    uargs.atom = chunk;
    const uint32_t fmt = bf16 ? 1u : 2u;
    const uint32_t n_mma = (uint32_t)g.n_mma;
    const uint32_t m_mma = g.pair ? 256u : 128u;
    uargs.idesc = (1u << 4) | (fmt << 7) | (fmt << 10)      // fp32 accumulate, operand formats;
                  | ((n_mma >> 3) << 17) | ((m_mma >> 4) << 24);   // both operands K-major; N, M
    if (g.pair)
      st = bf16 ? launch_wgrad_umma<true, true, false>(ds, mg, mi, uargs, stream)
                : launch_wgrad_umma<false, true, false>(ds, mg, mi, uargs, stream);
    else
      st = bf16 ? launch_wgrad_umma<true, false, false>(ds, mg, mi, uargs, stream)
                : launch_wgrad_umma<false, false, false>(ds, mg, mi, uargs, stream);
    if (st != MAXDNN_OK) return st;
  }
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (g.splits > 1) {
    const size_t n4 = kno / 4;
    wgrad_reduce_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, stream>>>(
        static_cast<const float*>(ws), dfilt, n4, g.splits, g.alpha);
    if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
    g_launches.fetch_add(1, std::memory_order_relaxed);
  }
  return MAXDNN_OK;
}

// ---------------------------------------------------------------------------
// FPROP through zero-padded staging tensors (shapes outside the 16-byte row rule).
// ---------------------------------------------------------------------------
struct RaggedPlan {
  maxdnn_conv_desc padded;
  bool direct;                        // the shape needs no padding
  size_t in_bytes, filt_bytes, out_bytes;   // staging tensors, each rounded up to 256 bytes
};


// fp32, ragged counts: the rows can be staged inside the kernel (no extra pass over any
// tensor, but tiles of 128 columns and copy warps that take issue slots from the arithmetic)
// or the bulk-copy kernel can run on zero-padded copies (one extra read and write of maps
// and result).  Measured, the padded route is the faster one on every layer tried (3 x 3 x
// 128 -> 256, 62 images: 2.29 against 2.58 ms; 5 x 5 x 96 -> 256, 126 images: 2.12 against
// 2.35 ms; the 3-channel 11 x 11 layer, whose K steps have 3 channels: 0.72 against 9.1 ms),
// so it is the default; option RAGGED_PADDED = -1 selects the in-kernel route.
bool ragged_in_kernel(const maxdnn_conv_desc*, maxdnn_kernel_kind kind) {
  return kind == MAXDNN_KERNEL_FP32 && option(OPT_RAGGED_PADDED, 0) < 0;
}

maxdnn_status plan_ragged(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind, RaggedPlan* p) {
  if (!desc || !kind_ok(kind)) return MAXDNN_INVALID_VALUE;
  int32_t Ho, Wo;
  const maxdnn_status st = check_desc(desc, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  const int nb_mult = kind == MAXDNN_KERNEL_FP32 ? 4 : (kind == MAXDNN_KERNEL_TF32 ? 32 : 64);
  const int no_mult = kind == MAXDNN_KERNEL_FP32 ? 4 : 32;
  const size_t eb = kind == MAXDNN_KERNEL_BF16 ? 2 : 4;
  p->padded = *desc;
  p->padded.Nb = align_up(desc->Nb, nb_mult);
  p->padded.No = align_up(desc->No, no_mult);
  p->direct = p->padded.Nb == desc->Nb && p->padded.No == desc->No;
  p->in_bytes = round256((size_t)desc->Nc * desc->Hi * desc->Wi * p->padded.Nb * eb);
  p->filt_bytes = round256((size_t)desc->Nc * desc->Sk * desc->Sk * p->padded.No * eb);
  p->out_bytes = round256((size_t)p->padded.No * Ho * Wo * p->padded.Nb * 4);
  return MAXDNN_OK;
}

template <typename T>
maxdnn_status launch_pad(const void* src, void* dst, size_t rows, int n, int n_pad,
                         cudaStream_t stream) {
  const size_t total = rows * (size_t)n_pad;
  pad_inner_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(
      static_cast<const T*>(src), static_cast<T*>(dst), rows, n, n_pad);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return MAXDNN_OK;
}

maxdnn_status fprop_ragged(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind, const void* in,
                           const void* filt, float* out, void* ws, size_t ws_bytes,
                           cudaStream_t stream) {
  RaggedPlan p;
  maxdnn_status st = plan_ragged(desc, kind, &p);
  if (st != MAXDNN_OK) return st;
  const int eb = kind == MAXDNN_KERNEL_BF16 ? 2 : 4;
  if (p.direct) {
    if (kind == MAXDNN_KERNEL_FP32)
      return fprop_fp32(desc, static_cast<const float*>(in), static_cast<const float*>(filt), out, stream);
    return fprop_umma(desc, eb, in, filt, out, stream);
  }
  if (ragged_in_kernel(desc, kind)) {
    // the fp32 kernel stages ragged rows itself: no padded copies, no workspace
    if (!in || !filt || !out) return MAXDNN_INVALID_VALUE;
    return fprop_fp32(dims_from(*desc), static_cast<const float*>(in), static_cast<const float*>(filt),
                      out, stream, true);
  }
  if (!in || !filt || !out || !ws) return MAXDNN_INVALID_VALUE;
  if (!aligned16(ws) || ws_bytes < p.in_bytes + p.filt_bytes + p.out_bytes) return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;
  st = dgrad_plan_check(dims_from(p.padded), kind, ds->sm_count);   // the padded problem must have a plan
  if (st != MAXDNN_OK) return st;
  int32_t Ho, Wo;
  check_desc(desc, &Ho, &Wo);
  uint8_t* w_in = static_cast<uint8_t*>(ws);
  uint8_t* w_filt = w_in + p.in_bytes;
  float* w_out = reinterpret_cast<float*>(w_filt + p.filt_bytes);
  const size_t in_rows = (size_t)desc->Nc * desc->Hi * desc->Wi;
  const size_t f_rows = (size_t)desc->Nc * desc->Sk * desc->Sk;
  if (eb == 2) {
    st = launch_pad<uint16_t>(in, w_in, in_rows, desc->Nb, p.padded.Nb, stream);
    if (st == MAXDNN_OK) st = launch_pad<uint16_t>(filt, w_filt, f_rows, desc->No, p.padded.No, stream);
  } else {
    st = launch_pad<float>(in, w_in, in_rows, desc->Nb, p.padded.Nb, stream);
    if (st == MAXDNN_OK) st = launch_pad<float>(filt, w_filt, f_rows, desc->No, p.padded.No, stream);
  }
  if (st != MAXDNN_OK) return st;
  if (kind == MAXDNN_KERNEL_FP32)
    st = fprop_fp32(&p.padded, reinterpret_cast<const float*>(w_in),
                    reinterpret_cast<const float*>(w_filt), w_out, stream);
  else
    st = fprop_umma(&p.padded, eb, w_in, w_filt, w_out, stream);
  if (st != MAXDNN_OK) return st;
  // out[o][y][x][n] for o < No, n < Nb: the first No filter slabs, padding images dropped
  const size_t out_rows = (size_t)desc->No * Ho * Wo;
  const size_t total = out_rows * (size_t)desc->Nb;
  unpad_inner_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(w_out, out, out_rows,
                                                                         desc->Nb, p.padded.Nb);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return MAXDNN_OK;
}

// ---------------------------------------------------------------------------
// fp32-level accuracy on the tensor cores: three TF32 products as one FPROP over 3 Nc channels.
// ---------------------------------------------------------------------------
maxdnn_status tf32x3_sizes(const maxdnn_conv_desc* desc, size_t* in_bytes, size_t* filt_bytes) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  const maxdnn_status st = check_desc(desc, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  if (desc->Nc > 32767 / 3) return MAXDNN_NOT_SUPPORTED;
  if (desc->Nb % 4 != 0 || desc->No % 4 != 0) return MAXDNN_NOT_SUPPORTED;
  *in_bytes = round256((size_t)3 * desc->Nc * desc->Hi * desc->Wi * desc->Nb * 4);
  *filt_bytes = round256((size_t)3 * desc->Nc * desc->Sk * desc->Sk * desc->No * 4);
  return MAXDNN_OK;
}

maxdnn_status fprop_tf32x3(const maxdnn_conv_desc* desc, const float* in, const float* filt,
                           float* out, void* ws, size_t ws_bytes, cudaStream_t stream) {
  size_t in_bytes = 0, filt_bytes = 0;
  maxdnn_status st = tf32x3_sizes(desc, &in_bytes, &filt_bytes);
  if (st != MAXDNN_OK) return st;
  if (!in || !filt || !out || !ws) return MAXDNN_INVALID_VALUE;
  if (!aligned16(in) || !aligned16(filt) || !aligned16(out) || !aligned16(ws)) return MAXDNN_INVALID_VALUE;
  if (ws_bytes < in_bytes + filt_bytes) return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;
  maxdnn_conv_desc d3 = *desc;
  d3.Nc = 3 * desc->Nc;
  st = dgrad_plan_check(dims_from(d3), MAXDNN_KERNEL_TF32, ds->sm_count);   // the 3 Nc-channel problem has a plan
  if (st != MAXDNN_OK) return st;
  float* w_in = static_cast<float*>(ws);
  float* w_filt = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + in_bytes);
  const size_t n4_in = (size_t)desc->Nc * desc->Hi * desc->Wi * desc->Nb / 4;
  const size_t n4_f = (size_t)desc->Nc * desc->Sk * desc->Sk * desc->No / 4;
  // maps [hi; hi; lo] x filters [hi; lo; hi]  ->  hi*hi + hi*lo + lo*hi
  tf32_split3_kernel<<<(unsigned)((n4_in + 255) / 256), 256, 0, stream>>>(
      reinterpret_cast<const float4*>(in), reinterpret_cast<float4*>(w_in), n4_in, 0x4u);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  tf32_split3_kernel<<<(unsigned)((n4_f + 255) / 256), 256, 0, stream>>>(
      reinterpret_cast<const float4*>(filt), reinterpret_cast<float4*>(w_filt), n4_f, 0x2u);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(2, std::memory_order_relaxed);
  // A fresh accumulator about every 768 rows of the split problem's K (256 of the
  // original): the accumulator's truncation then acts on short partial sums only.
  const int chunk_rows = option(OPT_X3_CHUNK_ROWS, 768);
  if (chunk_rows > 0) return fprop_umma(dims_from(d3), 4, w_in, w_filt, out, stream, chunk_rows);
  return fprop_umma(&d3, 4, w_in, w_filt, out, stream);
}

// Map gradient in the three-product TF32 mode, stride 1: the FPROP of dout with the flipped,
// transposed filter bank (as maxdnn_conv_bprop_data), run through fprop_tf32x3.  Workspace:
// the transformed bank (fp32, rounded up to 256 bytes), then fprop_tf32x3's own.
maxdnn_status dgrad_tf32x3_desc(const maxdnn_conv_desc* desc, maxdnn_conv_desc* t, size_t* ft_bytes) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  maxdnn_status st = check_desc(desc, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  if (desc->stride != 1) return MAXDNN_NOT_SUPPORTED;
  ConvDims fd;
  st = plan_dgrad(dims_from(*desc), &fd);
  if (st != MAXDNN_OK) return st;
  t->Nb = fd.Nb; t->Wi = fd.Wi; t->Hi = fd.Hi; t->Nc = fd.Nc; t->No = fd.No;
  t->Sk = fd.Skw; t->stride = 1; t->pad = fd.pad_w; t->alpha = fd.alpha;
  *ft_bytes = round256((size_t)desc->Nc * desc->Sk * desc->Sk * desc->No * 4);
  return MAXDNN_OK;
}

maxdnn_status bprop_data_tf32x3(const maxdnn_conv_desc* desc, const float* dout, const float* filt,
                                float* din, void* ws, size_t ws_bytes, cudaStream_t stream) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  if (desc->stride > 1) {
    // the residue classes of maxdnn_conv_bprop_data, each through the chunked kernels
    maxdnn_status st0 = check_desc(desc, nullptr, nullptr);
    if (st0 != MAXDNN_OK) return st0;
    if (!dout || !filt || !din || !ws) return MAXDNN_INVALID_VALUE;
    if (!aligned16(dout) || !aligned16(filt) || !aligned16(din) || !aligned16(ws))
      return MAXDNN_INVALID_VALUE;
    return bprop_data_strided(dims_from(*desc), MAXDNN_KERNEL_TF32, dout, filt, din, ws, ws_bytes,
                              stream, true);
  }
  maxdnn_conv_desc t;
  size_t ft_bytes = 0, a = 0, b = 0;
  maxdnn_status st = dgrad_tf32x3_desc(desc, &t, &ft_bytes);
  if (st != MAXDNN_OK) return st;
  st = tf32x3_sizes(&t, &a, &b);
  if (st != MAXDNN_OK) return st;
  if (!dout || !filt || !din || !ws) return MAXDNN_INVALID_VALUE;
  if (!aligned16(dout) || !aligned16(filt) || !aligned16(din) || !aligned16(ws))
    return MAXDNN_INVALID_VALUE;
  if (ws_bytes < ft_bytes + a + b) return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;
  const int taps = desc->Sk * desc->Sk;
  const dim3 grid((unsigned)ceil_div(desc->No, 32), (unsigned)ceil_div(desc->Nc, 32), (unsigned)taps);
  flip_transpose_kernel<float><<<grid, dim3(32, 8), 0, stream>>>(filt, static_cast<float*>(ws),
                                                               desc->Nc, taps, desc->No);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return fprop_tf32x3(&t, dout, static_cast<const float*>(ws), din,
                      static_cast<uint8_t*>(ws) + ft_bytes, ws_bytes - ft_bytes, stream);
}

// Filter gradient in the three-product TF32 mode.  The reduction runs over pixels and
// images, so the three products are one reduction over three times the images: both
// tensors are split into [hi | lo] side by side along the image axis, and the chunked TF32
// filter-gradient kernel runs on the problem with 3 Nb images, reading for each third of
// them the parts of that product (hi x hi, hi x lo, lo x hi).  Workspace: the two
// split tensors (each rounded up to 256 bytes), then the partial sums of the split reduction.
struct WgradX3Plan {
  ConvDims d3;
  size_t in_bytes, dout_bytes, partial_bytes;
};

maxdnn_status plan_wgrad_x3(const maxdnn_conv_desc* desc, int sm_count, WgradX3Plan* p, WgradGeom* g) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  int32_t Ho, Wo;
  maxdnn_status st = check_desc(desc, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  if (desc->Nb % 32 != 0) return MAXDNN_NOT_SUPPORTED;      // whole 128-byte rows of each part
  if ((int64_t)desc->Nb * 3 > 0x7fffffff) return MAXDNN_NOT_SUPPORTED;
  p->d3 = dims_from(*desc);
  p->d3.Nb = 3 * desc->Nb;
  p->in_bytes = round256((size_t)desc->Nc * desc->Hi * desc->Wi * 2 * desc->Nb * 4);     // [hi | lo]
  p->dout_bytes = round256((size_t)desc->No * Ho * Wo * 2 * desc->Nb * 4);
  static thread_local WgradGeom scratch;
  WgradGeom* gg = g ? g : &scratch;
  st = plan_wgrad(p->d3, 4, sm_count, option(OPT_WGRAD_SPLITS), gg, option(OPT_WGRAD_PAIR));
  if (st != MAXDNN_OK) return st;
  const size_t kno = (size_t)desc->Nc * desc->Sk * desc->Sk * desc->No;
  p->partial_bytes = gg->splits > 1 ? (size_t)gg->splits * kno * 4 : 0;
  return MAXDNN_OK;
}

maxdnn_status bprop_filter_tf32x3(const maxdnn_conv_desc* desc, const float* in, const float* dout,
                                  float* dfilt, void* ws, size_t ws_bytes, cudaStream_t stream) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  if (!in || !dout || !dfilt || !ws) return MAXDNN_INVALID_VALUE;
  if (!aligned16(in) || !aligned16(dout) || !aligned16(dfilt) || !aligned16(ws))
    return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  maxdnn_status st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;
  static thread_local WgradUmmaArgs args;
  WgradX3Plan p;
  st = plan_wgrad_x3(desc, ds->sm_count, &p, &args.g);
  if (st != MAXDNN_OK) return st;
  if (ws_bytes < p.in_bytes + p.dout_bytes + p.partial_bytes) return MAXDNN_INVALID_VALUE;
  const WgradGeom& g = args.g;
  float* w_in = static_cast<float*>(ws);
  float* w_dout = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + p.in_bytes);
  float* w_part = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + p.in_bytes + p.dout_bytes);
  const int n4 = desc->Nb / 4;
  const size_t rows_in = (size_t)desc->Nc * desc->Hi * desc->Wi;
  const size_t rows_g = (size_t)desc->No * g.Ho * g.Wo;
  // both tensors as [hi | lo] along the image axis; the kernel's three passes over the
  // images pair them as hi*hi + hi*lo + lo*hi
  tf32_split2_rows_kernel<<<(unsigned)((rows_in * n4 + 255) / 256), 256, 0, stream>>>(
      reinterpret_cast<const float4*>(in), reinterpret_cast<float4*>(w_in), rows_in, n4);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  tf32_split2_rows_kernel<<<(unsigned)((rows_g * n4 + 255) / 256), 256, 0, stream>>>(
      reinterpret_cast<const float4*>(dout), reinterpret_cast<float4*>(w_dout), rows_g, n4);
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(2, std::memory_order_relaxed);
  CUtensorMap mg, mi;
  {
    const uint64_t nb2 = 2ull * desc->Nb;      // stored images per pixel: [hi | lo]
    const uint64_t dims[4] = {nb2, (uint64_t)g.Wo, (uint64_t)g.Ho, (uint64_t)g.No};
    const uint64_t str[3] = {nb2 * 4, (uint64_t)g.Wo * nb2 * 4, (uint64_t)g.Ho * g.Wo * nb2 * 4};
    const uint32_t box[4] = {32u, 1u, 1u, (uint32_t)g.box_o};
    st = encode_map(&mg, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, w_dout, dims, str, box,
                    CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != MAXDNN_OK) return st;
  }
  {
    const uint64_t nb2 = 2ull * desc->Nb;
    const uint64_t dims[4] = {nb2, (uint64_t)g.Wi, (uint64_t)g.Hi, (uint64_t)g.Nc};
    const uint64_t str[3] = {nb2 * 4, (uint64_t)g.Wi * nb2 * 4, (uint64_t)g.Hi * g.Wi * nb2 * 4};
    // (a pair's CTA stages half of the tile's channels)
    const uint32_t box[4] = {32u, (uint32_t)g.bw, (uint32_t)g.bh, (uint32_t)(g.pair ? g.bc_h : g.bc)};
    st = encode_map(&mi, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, w_in, dims, str, box,
                    CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != MAXDNN_OK) return st;
  }
  args.dfilt = dfilt;
  args.partial = w_part;
  args.wc = next_wait_ctx(ds);
  args.atom = 32u;
  // a fresh accumulator every 24 reduction steps: 768 terms of the tripled reduction
  const int cs = option(OPT_X3_CHUNK_ROWS, 768) / 32;
  args.chunk_steps = (uint32_t)(cs < 1 ? 1 : cs);
  args.x3_per_part = (uint32_t)(desc->Nb / 32);
  args.idesc = (1u << 4) | (2u << 7) | (2u << 10) | (((uint32_t)g.n_mma >> 3) << 17) |
               (((g.pair ? 256u : 128u) >> 4) << 24);
  st = g.pair ? launch_wgrad_umma<false, true, true>(ds, mg, mi, args, stream)
              : launch_wgrad_umma<false, false, true>(ds, mg, mi, args, stream);
  if (st != MAXDNN_OK) return st;
  if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (g.splits > 1) {
    const size_t n4f = (size_t)desc->Nc * desc->Sk * desc->Sk * desc->No / 4;
    wgrad_reduce_kernel<<<(unsigned)((n4f + 255) / 256), 256, 0, stream>>>(w_part, dfilt, n4f,
                                                                         g.splits, g.alpha);
    if (cudaGetLastError() != cudaSuccess) return MAXDNN_CUDA_ERROR;
    g_launches.fetch_add(1, std::memory_order_relaxed);
  }
  return MAXDNN_OK;
}

// ---------------------------------------------------------------------------
// Allocation-free fp32 entry point.  The status block its kernel reports into
// lives in this file-scope device array instead of cudaMalloc'd memory.  Every
// device that loads the library carries these 256 bytes until the process ends.
// In host code the array's name is only a handle for the runtime: the device
// address is obtained once per device with cudaGetSymbolAddress and passed on.
// ---------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = 256;
static __device__ __align__(256) uint32_t g_static_scratch[kStaticScratchBytes / sizeof(uint32_t)];

// Scratch the fp32 kernel needs for a plan: the two words of the status block (first code
// recorded; epoch of the latest launch that gave up).
size_t ffma_scratch_bytes(const ConvGeom&) { return 2 * sizeof(uint32_t); }

DeviceState g_static_dev[kMaxDevices];   // `status` points into g_static_scratch of that device

maxdnn_status static_state(DeviceState** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return MAXDNN_CUDA_ERROR; }
  if (dev < 0 || dev >= kMaxDevices) return MAXDNN_NOT_SUPPORTED;
  std::lock_guard<std::mutex> lk(g_mu);
  DeviceState& s = g_static_dev[dev];
  if (!s.ready) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
      cudaGetLastError();
      return MAXDNN_CUDA_ERROR;
    }
    s.sm100 = (prop.major == 10);
    s.sm_count = prop.multiProcessorCount;
    if (s.sm100) {
      void* p = nullptr;
      // device `dev` is current: this is the address of ITS copy of the array
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
        cudaGetLastError();
        return MAXDNN_CUDA_ERROR;
      }
      s.status = static_cast<uint32_t*>(p);
    }
    s.ready = true;
  }
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) !=
            cudaSuccess || !fn) {
      cudaGetLastError();
      return MAXDNN_CUDA_ERROR;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  *out = &s;
  return MAXDNN_OK;
}

maxdnn_status fprop_fp32_noalloc(const maxdnn_conv_desc* desc, const float* in, const float* filt,
                                 float* out, cudaStream_t stream) {
  int32_t Ho, Wo;
  maxdnn_status st = check_desc(desc, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  if (!in || !filt || !out) return MAXDNN_INVALID_VALUE;
  if (!aligned16(in) || !aligned16(filt) || !aligned16(out)) return MAXDNN_INVALID_VALUE;
  DeviceState* ds = nullptr;
  st = static_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->sm100) return MAXDNN_NOT_SUPPORTED;

  static thread_local FfmaArgs args;
  // the plan of maxdnn_conv_fprop for this problem (tile options included)
  st = plan_ffma(dims_from(*desc), ds->sm_count, option(OPT_FFMA_TILE_M), option(OPT_FFMA_COLS),
                 &args.g, &args.table);
  if (st != MAXDNN_OK) return st;
  if (ffma_scratch_bytes(args.g) > kStaticScratchBytes) return MAXDNN_NOT_SUPPORTED;
  args.out = out;
  args.sk_partial = nullptr;       // no workspace here: the plan never splits its tail
  args.sk_flags = nullptr;
  args.in = in;
  args.filt = filt;
  args.wc = next_wait_ctx(ds);
  args.test_missing_arrival = (uint32_t)option(OPT_TEST_MISSING_ARRIVAL);
  args.clock_stamp = 0;
  const ConvGeom& g = args.g;

  CUtensorMap mf, mi;
  {
    const uint64_t dims[4] = {(uint64_t)g.No, (uint64_t)g.Skw, (uint64_t)g.Nc, (uint64_t)g.Skh};
    const uint64_t str[3] = {(uint64_t)g.No * 4, (uint64_t)g.Skh * g.Skw * g.No * 4,
                             (uint64_t)g.Skw * g.No * 4};
    const uint32_t box[4] = {(uint32_t)g.tile_m, (uint32_t)g.kwc, (uint32_t)g.kc, (uint32_t)g.box_kh};
    st = encode_map(&mf, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, filt, dims, str, box,
                    CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st != MAXDNN_OK) return st;
  }
  {
    const uint64_t dims[4] = {(uint64_t)g.Nb, (uint64_t)g.Wi, (uint64_t)g.Nc, (uint64_t)g.Hi};
    const uint64_t hs = dims_in_h(g, 0), cs = dims_in_c(g, 0);
    const uint64_t str[3] = {(uint64_t)g.Nb * 4, cs * 4, hs * 4};
    const uint32_t box[4] = {(uint32_t)g.tile_n, (uint32_t)g.b_box_w, (uint32_t)g.kc, (uint32_t)g.box_kh};
    st = encode_map(&mi, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, in, dims, str, box,
                    CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st != MAXDNN_OK) return st;
  }
  // The block is shared by every call and keeps what earlier calls left.  Nothing in it
  // has to start at zero: word 0 is only ever written by a wait that ran out and is
  // cleared by maxdnn_last_device_status_noalloc; word 1 is compared with this launch's
  // epoch, which no earlier launch had.
  return dispatch_ffma(ds, mf, mi, args, stream);
}

// Waits for the stream, reads word 0 of the device's status block and clears it if set.
// No allocation: a 4-byte copy into host memory and, after a failure, a 4-byte memset.
maxdnn_status read_and_clear_status(DeviceState* ds, cudaStream_t stream) {
  uint32_t word = 0;
  if (cudaStreamSynchronize(stream) != cudaSuccess ||
      cudaMemcpy(&word, ds->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  if (word != 0) {
    if (option(OPT_DEBUG_STATUS)) fprintf(stderr, "maxdnn: device status word 0x%x\n", word);
    cudaMemset(ds->status, 0, 4);
    return MAXDNN_DEVICE_TIMEOUT;
  }
  return MAXDNN_OK;
}

}  // namespace
}  // namespace maxdnn

using namespace maxdnn;

extern "C" {

const char* maxdnn_status_string(maxdnn_status s) {
  switch (s) {
    case MAXDNN_OK: return "MAXDNN_OK";
    case MAXDNN_INVALID_VALUE: return "MAXDNN_INVALID_VALUE";
    case MAXDNN_NOT_SUPPORTED: return "MAXDNN_NOT_SUPPORTED";
    case MAXDNN_CUDA_ERROR: return "MAXDNN_CUDA_ERROR";
    case MAXDNN_DEVICE_TIMEOUT: return "MAXDNN_DEVICE_TIMEOUT";
    default: return "MAXDNN_UNKNOWN_STATUS";
  }
}

maxdnn_status maxdnn_conv_out_dims(const maxdnn_conv_desc* desc, int32_t* Ho, int32_t* Wo) {
  return check_desc(desc, Ho, Wo);
}

uint64_t maxdnn_conv_flops(const maxdnn_conv_desc* d) {
  int32_t Ho, Wo;
  if (check_desc(d, &Ho, &Wo) != MAXDNN_OK) return 0;
  return 2ull * (uint64_t)d->Nb * (uint64_t)Wo * (uint64_t)Ho *
         ((uint64_t)d->Nc * (uint64_t)d->Sk * (uint64_t)d->Sk + 1ull) * (uint64_t)d->No;
}

uint64_t maxdnn_conv_in_elems(const maxdnn_conv_desc* d) {
  if (check_desc(d, nullptr, nullptr) != MAXDNN_OK) return 0;
  return (uint64_t)d->Nc * d->Hi * d->Wi * d->Nb;
}

uint64_t maxdnn_conv_filt_elems(const maxdnn_conv_desc* d) {
  if (check_desc(d, nullptr, nullptr) != MAXDNN_OK) return 0;
  return (uint64_t)d->Nc * d->Sk * d->Sk * d->No;
}

uint64_t maxdnn_conv_out_elems(const maxdnn_conv_desc* d) {
  int32_t Ho, Wo;
  if (check_desc(d, &Ho, &Wo) != MAXDNN_OK) return 0;
  return (uint64_t)d->No * Ho * Wo * d->Nb;
}

maxdnn_status maxdnn_conv_plan_query(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                     int32_t sm_count, maxdnn_plan_info* info,
                                     maxdnn_kstep* steps, int32_t max_steps) {
  if (!desc || !info) return MAXDNN_INVALID_VALUE;
  maxdnn_status st = check_desc(desc, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  if (sm_count <= 0) {
    DeviceState* ds = nullptr;
    st = device_state(&ds);
    if (st != MAXDNN_OK) return st;
    sm_count = ds->sm_count;
  }
  static thread_local ConvGeom g;
  static thread_local KStepTable t;
  switch (kind) {
    case MAXDNN_KERNEL_FP32:
      st = plan_ffma(dims_from(*desc), sm_count, option(OPT_FFMA_TILE_M), option(OPT_FFMA_COLS), &g, &t,
                     true);
      break;
    case MAXDNN_KERNEL_TF32: st = plan_umma(dims_from(*desc), 4, sm_count, option(OPT_UMMA_KC), option(OPT_UMMA_PAIR), &g, &t); break;
    case MAXDNN_KERNEL_BF16: st = plan_umma(dims_from(*desc), 2, sm_count, option(OPT_UMMA_KC), option(OPT_UMMA_PAIR), &g, &t); break;
    default: return MAXDNN_INVALID_VALUE;
  }
  if (st != MAXDNN_OK) return st;
  info->Ho = g.Ho; info->Wo = g.Wo;
  info->tile_m = g.tile_m; info->tile_px = g.tile_px; info->tile_n = g.tile_n;
  info->kc = g.kc; info->kwc = g.kwc; info->n_ksteps = g.n_ksteps; info->stages = g.stages;
  info->n_tiles = g.n_tiles; info->grid = g.grid; info->smem_bytes = g.smem_bytes;
  info->tile_cols = g.tile_cols; info->pair = g.pair; info->khc = g.box_kh;
  info->split_tiles = kind == MAXDNN_KERNEL_FP32 ? g.sk_tiles : 0;
  if (steps)
    for (int i = 0; i < g.n_ksteps && i < max_steps; ++i) steps[i] = t.s[i];
  return MAXDNN_OK;
}

maxdnn_status maxdnn_conv_plan_items(const maxdnn_conv_desc* desc, int32_t sm_count, int32_t cta,
                                     maxdnn_work_item* items, int32_t max_items,
                                     int32_t* n_items) {
  if (!desc || !n_items || (max_items > 0 && !items)) return MAXDNN_INVALID_VALUE;
  maxdnn_status st = check_desc(desc, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  if (sm_count <= 0) {
    DeviceState* ds = nullptr;
    st = device_state(&ds);
    if (st != MAXDNN_OK) return st;
    sm_count = ds->sm_count;
  }
  static thread_local ConvGeom g;
  static thread_local KStepTable t;
  st = plan_ffma(dims_from(*desc), sm_count, option(OPT_FFMA_TILE_M), option(OPT_FFMA_COLS), &g, &t, true);
  if (st != MAXDNN_OK) return st;
  if (cta < 0 || cta >= g.grid) return MAXDNN_INVALID_VALUE;
  int n = 0;
  FfmaItem it;
  while (ffma_item_at(g, g.grid, cta, n, it)) {
    if (n < max_items) {
      items[n].tile = it.tile; items[n].s0 = it.s0; items[n].s1 = it.s1; items[n].kind = it.kind;
    }
    ++n;
  }
  *n_items = n;
  return MAXDNN_OK;
}

maxdnn_status maxdnn_conv_fprop(const maxdnn_conv_desc* desc, const float* in, const float* filt,
                                float* out, void* cuda_stream) {
  return fprop_fp32(desc, in, filt, out, static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_fprop_tf32(const maxdnn_conv_desc* desc, const float* in,
                                     const float* filt, float* out, void* cuda_stream) {
  return fprop_umma(desc, 4, in, filt, out, static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_fprop_bf16(const maxdnn_conv_desc* desc, const void* in,
                                     const void* filt, float* out, void* cuda_stream) {
  return fprop_umma(desc, 2, in, filt, out, static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_fprop_host(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                     const void* h_in, const void* h_filt, float* h_out,
                                     void* d_in, void* d_filt, float* d_out, void* cuda_stream) {
  if (!h_in || !h_filt || !h_out || !d_in || !d_filt || !d_out) return MAXDNN_INVALID_VALUE;
  if (check_desc(desc, nullptr, nullptr) != MAXDNN_OK) return MAXDNN_INVALID_VALUE;
  if (kind != MAXDNN_KERNEL_FP32 && kind != MAXDNN_KERNEL_TF32 && kind != MAXDNN_KERNEL_BF16)
    return MAXDNN_INVALID_VALUE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t eb = (kind == MAXDNN_KERNEL_BF16) ? 2 : 4;
  if (cudaMemcpyAsync(d_in, h_in, maxdnn_conv_in_elems(desc) * eb, cudaMemcpyHostToDevice,
                      stream) != cudaSuccess ||
      cudaMemcpyAsync(d_filt, h_filt, maxdnn_conv_filt_elems(desc) * eb, cudaMemcpyHostToDevice,
                      stream) != cudaSuccess) {
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  maxdnn_status st;
  if (kind == MAXDNN_KERNEL_FP32)
    st = fprop_fp32(desc, static_cast<const float*>(d_in), static_cast<const float*>(d_filt),
                    d_out, stream);
  else
    st = fprop_umma(desc, (int)eb, d_in, d_filt, d_out, stream);
  if (st != MAXDNN_OK) return st;
  if (cudaMemcpyAsync(h_out, d_out, maxdnn_conv_out_elems(desc) * 4, cudaMemcpyDeviceToHost,
                      stream) != cudaSuccess) {
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  return MAXDNN_OK;
}

static maxdnn::ConvDims dims_from2(const maxdnn_conv_desc2& d) {
  maxdnn::ConvDims c;
  c.Nb = d.Nb; c.Wi = d.Wi; c.Hi = d.Hi; c.Nc = d.Nc; c.No = d.No;
  c.Skw = d.Skw; c.Skh = d.Skh; c.stride_w = d.stride_w; c.stride_h = d.stride_h;
  c.pad_w = d.pad_w; c.pad_h = d.pad_h; c.alpha = d.alpha;
  c.in_h_stride = c.in_c_stride = 0;
  c.Ho_given = c.Wo_given = 0;
  c.out_x_stride = c.out_y_stride = c.out_o_stride = 0;
  return c;
}

maxdnn_status maxdnn_conv2_out_dims(const maxdnn_conv_desc2* desc, int32_t* Ho, int32_t* Wo) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  return check_dims(dims_from2(*desc), Ho, Wo);
}

maxdnn_status maxdnn_conv2_fprop(const maxdnn_conv_desc2* desc, maxdnn_kernel_kind kind,
                                 const void* in, const void* filt, float* out, void* cuda_stream) {
  if (!desc || !kind_ok(kind)) return MAXDNN_INVALID_VALUE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (kind == MAXDNN_KERNEL_FP32)
    return fprop_fp32(dims_from2(*desc), static_cast<const float*>(in),
                      static_cast<const float*>(filt), out, stream);
  return fprop_umma(dims_from2(*desc), kind == MAXDNN_KERNEL_BF16 ? 2 : 4, in, filt, out, stream);
}

maxdnn_status maxdnn_conv_fprop_tf32x3_workspace(const maxdnn_conv_desc* desc, size_t* bytes) {
  if (!bytes) return MAXDNN_INVALID_VALUE;
  size_t a = 0, b = 0;
  const maxdnn_status st = tf32x3_sizes(desc, &a, &b);
  if (st != MAXDNN_OK) return st;
  *bytes = a + b;
  return MAXDNN_OK;
}

maxdnn_status maxdnn_conv_fprop_tf32x3(const maxdnn_conv_desc* desc, const float* in,
                                       const float* filt, float* out, void* workspace,
                                       size_t workspace_bytes, void* cuda_stream) {
  return fprop_tf32x3(desc, in, filt, out, workspace, workspace_bytes,
                      static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_bprop_data_tf32x3_workspace(const maxdnn_conv_desc* desc, size_t* bytes) {
  if (!bytes || !desc) return MAXDNN_INVALID_VALUE;
  if (desc->stride > 1) {
    maxdnn_status st0 = check_desc(desc, nullptr, nullptr);
    if (st0 != MAXDNN_OK) return st0;
    DgradStridedPlan p;
    st0 = plan_dgrad_strided(dims_from(*desc), MAXDNN_KERNEL_TF32, &p, true);
    if (st0 != MAXDNN_OK) return st0;
    *bytes = p.pre_bytes + p.ft_bytes + p.sub_bytes;
    return MAXDNN_OK;
  }
  maxdnn_conv_desc t;
  size_t ft_bytes = 0, a = 0, b = 0;
  maxdnn_status st = dgrad_tf32x3_desc(desc, &t, &ft_bytes);
  if (st != MAXDNN_OK) return st;
  st = tf32x3_sizes(&t, &a, &b);
  if (st != MAXDNN_OK) return st;
  *bytes = ft_bytes + a + b;
  return MAXDNN_OK;
}

maxdnn_status maxdnn_conv_bprop_data_tf32x3(const maxdnn_conv_desc* desc, const float* dout,
                                            const float* filt, float* din, void* workspace,
                                            size_t workspace_bytes, void* cuda_stream) {
  return bprop_data_tf32x3(desc, dout, filt, din, workspace, workspace_bytes,
                           static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_bprop_filter_tf32x3_workspace(const maxdnn_conv_desc* desc, size_t* bytes) {
  if (!bytes) return MAXDNN_INVALID_VALUE;
  int sm = option(OPT_SM_COUNT);
  if (sm <= 0) {
    DeviceState* ds = nullptr;
    const maxdnn_status st = device_state(&ds);
    if (st != MAXDNN_OK) return st;
    sm = ds->sm_count;
  }
  WgradX3Plan p;
  const maxdnn_status st = plan_wgrad_x3(desc, sm, &p, nullptr);
  if (st != MAXDNN_OK) return st;
  *bytes = p.in_bytes + p.dout_bytes + p.partial_bytes;
  return MAXDNN_OK;
}

maxdnn_status maxdnn_conv_bprop_filter_tf32x3(const maxdnn_conv_desc* desc, const float* in,
                                              const float* dout, float* dfilt, void* workspace,
                                              size_t workspace_bytes, void* cuda_stream) {
  return bprop_filter_tf32x3(desc, in, dout, dfilt, workspace, workspace_bytes,
                             static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_fprop_ragged_workspace(const maxdnn_conv_desc* desc,
                                                 maxdnn_kernel_kind kind, size_t* bytes) {
  if (!bytes) return MAXDNN_INVALID_VALUE;
  RaggedPlan p;
  const maxdnn_status st = plan_ragged(desc, kind, &p);
  if (st != MAXDNN_OK) return st;
  const bool in_kernel = ragged_in_kernel(desc, kind);
  *bytes = (p.direct || in_kernel) ? 0 : p.in_bytes + p.filt_bytes + p.out_bytes;
  return MAXDNN_OK;
}

maxdnn_status maxdnn_conv_fprop_ragged(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                       const void* in, const void* filt, float* out,
                                       void* workspace, size_t workspace_bytes,
                                       void* cuda_stream) {
  return fprop_ragged(desc, kind, in, filt, out, workspace, workspace_bytes,
                      static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_bprop_data_workspace(const maxdnn_conv_desc* desc,
                                               maxdnn_kernel_kind kind, size_t* bytes) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  const maxdnn_status st = check_desc(desc, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  return bprop_data_workspace(dims_from(*desc), kind, bytes);
}

maxdnn_status maxdnn_conv_bprop_data(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                     const void* dout, const void* filt, float* din,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  const maxdnn_status st = check_desc(desc, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  return bprop_data(dims_from(*desc), kind, dout, filt, din, workspace, workspace_bytes,
                    static_cast<cudaStream_t>(cuda_stream));
}

static maxdnn_status bprop_filter_workspace(const maxdnn::ConvDims& d, maxdnn_kernel_kind kind,
                                            size_t* bytes) {
  if (!bytes || !kind_ok(kind)) return MAXDNN_INVALID_VALUE;
  int sm_count = option(OPT_SM_COUNT);   // planning without a device (tests)
  if (sm_count <= 0) {
    DeviceState* ds = nullptr;
    const maxdnn_status st = device_state(&ds);
    if (st != MAXDNN_OK) return st;
    sm_count = ds->sm_count;
  }
  WgradGeom g;
  const int eb = kind == MAXDNN_KERNEL_FP32 ? 0 : (kind == MAXDNN_KERNEL_BF16 ? 2 : 4);
  const maxdnn_status st = plan_wgrad(d, eb, sm_count, option(OPT_WGRAD_SPLITS), &g,
                                      option(OPT_WGRAD_PAIR));
  if (st != MAXDNN_OK) return st;
  *bytes = g.splits > 1 ? (size_t)g.splits * g.Nc * g.Skh * g.Skw * g.No * 4 : 0;
  return MAXDNN_OK;
}

maxdnn_status maxdnn_conv_bprop_filter_workspace(const maxdnn_conv_desc* desc,
                                                 maxdnn_kernel_kind kind, size_t* bytes) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  const maxdnn_status st = check_desc(desc, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  return bprop_filter_workspace(dims_from(*desc), kind, bytes);
}

maxdnn_status maxdnn_conv2_bprop_filter_workspace(const maxdnn_conv_desc2* desc,
                                                  maxdnn_kernel_kind kind, size_t* bytes) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  return bprop_filter_workspace(dims_from2(*desc), kind, bytes);
}

maxdnn_status maxdnn_conv2_bprop_filter(const maxdnn_conv_desc2* desc, maxdnn_kernel_kind kind,
                                        const void* in, const void* dout, float* dfilt,
                                        void* workspace, size_t workspace_bytes,
                                        void* cuda_stream) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  return bprop_filter(dims_from2(*desc), kind, in, dout, dfilt, workspace, workspace_bytes,
                      static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv2_bprop_data_workspace(const maxdnn_conv_desc2* desc,
                                                maxdnn_kernel_kind kind, size_t* bytes) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  return bprop_data_workspace(dims_from2(*desc), kind, bytes);
}

maxdnn_status maxdnn_conv2_bprop_data(const maxdnn_conv_desc2* desc, maxdnn_kernel_kind kind,
                                      const void* dout, const void* filt, float* din,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  return bprop_data(dims_from2(*desc), kind, dout, filt, din, workspace, workspace_bytes,
                    static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_bprop_filter(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                       const void* in, const void* dout, float* dfilt,
                                       void* workspace, size_t workspace_bytes,
                                       void* cuda_stream) {
  if (!desc) return MAXDNN_INVALID_VALUE;
  const maxdnn_status st = check_desc(desc, nullptr, nullptr);
  if (st != MAXDNN_OK) return st;
  return bprop_filter(dims_from(*desc), kind, in, dout, dfilt, workspace, workspace_bytes,
                      static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_last_device_status(void* cuda_stream) {
  DeviceState* ds = nullptr;
  maxdnn_status st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->status) return MAXDNN_NOT_SUPPORTED;
  return read_and_clear_status(ds, static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_conv_fprop_noalloc(const maxdnn_conv_desc* desc, const float* in,
                                        const float* filt, float* out, void* cuda_stream) {
  return fprop_fp32_noalloc(desc, in, filt, out, static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_last_device_status_noalloc(void* cuda_stream) {
  DeviceState* ds = nullptr;
  maxdnn_status st = static_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->status) return MAXDNN_NOT_SUPPORTED;
  return read_and_clear_status(ds, static_cast<cudaStream_t>(cuda_stream));
}

maxdnn_status maxdnn_last_kernel_clock(uint32_t* sm_cycles, uint32_t* nanoseconds,
                                       void* cuda_stream) {
  DeviceState* ds = nullptr;
  maxdnn_status st = device_state(&ds);
  if (st != MAXDNN_OK) return st;
  if (!ds->status || !sm_cycles || !nanoseconds) return MAXDNN_INVALID_VALUE;
  uint32_t w[4] = {0, 0, 0, 0};   // whole-tile kernel, split-tail kernel
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess ||
      cudaMemcpy(w, ds->status + 2, 16, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return MAXDNN_CUDA_ERROR;
  }
  *sm_cycles = w[0] + w[2];
  *nanoseconds = w[1] + w[3];
  return MAXDNN_OK;
}

maxdnn_status maxdnn_set_option(const char* name, int32_t value) { return set_option(name, value); }
maxdnn_status maxdnn_unset_option(const char* name) { return unset_option(name); }
void maxdnn_reset_options(void) { reset_options(); }
maxdnn_status maxdnn_get_option(const char* name, int32_t* value, int32_t* is_set) {
  return get_option(name, value, is_set);
}

uint64_t maxdnn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
