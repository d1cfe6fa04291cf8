// Issue-rate microbenchmark behind the fp32 kernel's design: what one SM sub-partition
// sustains when a stream of packed fp32 multiply-adds (the 8 x 16 register block of the
// convolution kernel: 64 FFMA2 per K row) is mixed with the operand traffic of Section 3.1
// — shared-memory loads of 16 / 8 / 4 bytes per lane under different lane -> address maps,
// or warp shuffles.  It answers three questions with numbers: the ceiling of the pure
// multiply-add stream, the cost of one operand load next to it as a function of how many
// shared-memory wavefronts the lane map needs, and the cost of a shuffle.
//
// Built as its own small shared library (libmaxdnn_ubench.so); run by
// `python -m paper_1501_06633_b200.ubench`.  Not part of the convolution path.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int kThreads = 256;        // two warps per scheduler, as the convolution kernel
constexpr int kRowsPerIter = 4;

enum Kind : int { kNone = 0, kLds128 = 1, kLds64 = 2, kLds32 = 3, kShfl = 4 };

// lane -> index of the word (16, 8 or 4 bytes wide) the lane reads
__device__ __forceinline__ int lane_word(int map, int lane) {
  switch (map) {
    case 0: return 0;                                   // one word for the whole warp
    case 1: return lane >> 3;                           // 4 words, 8 consecutive lanes each
    case 2: return lane & 7;                            // 8 words, repeated by every quarter-warp
    case 3: return lane;                                // 32 distinct words
    case 4: return (lane >> 1) & 7;                     // 8 words, lane pairs, repeated by each half
    case 5: return (lane & 1) | ((lane >> 4) << 1);     // 4 words: partner of map 4
    case 6: return lane >> 2;                           // 8 words, 4 consecutive lanes each
    case 7: return lane & 3;                            // 4 words, repeated 8 times: partner of 6
    case 8: return lane >> 4;                           // 2 words, one per half-warp
    case 9: return lane & 15;                           // 16 words, repeated by each half
    case 10: return lane >> 1;                          // 16 words, lane pairs
    case 11: return lane & 1;                           // 2 words, alternating lanes
    case 12: return (lane >> 2) & 3;                    // 4 words, 4 consecutive lanes, repeated
    case 13: return (lane & 3) | ((lane >> 4) << 2);    // 8 words: partner of map 12
    default: return 0;
  }
}

// ORDER: how the 64 multiply-adds of a row walk the 4 x 8 grid of accumulator pairs.
//   0 column pairs outer, filter pairs inner, serpentine, P then Q (the convolution kernel's)
//   1 filter pairs outer, column pairs inner
//   2 all P products, then all Q products
//   3 eight accumulators only, one operand pair each: no operand variety at all
template <int KIND, int NL, int ORDER>
__global__ void __launch_bounds__(kThreads, 1)
issue_mix_kernel(const float* __restrict__ seed, float* __restrict__ sink, long long* cycles,
                 int iters, int map) {
  __shared__ __align__(128) float ring[8192];            // 32 KB of operand rows
  for (int i = threadIdx.x; i < 8192; i += kThreads) ring[i] = seed[i & 255];
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int width = KIND == kLds128 ? 16 : KIND == kLds64 ? 8 : 4;
  const uint32_t addr0 = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) +
                         (uint32_t)(lane_word(map, lane) * width);
  const int src_lane = lane_word(map, lane);

  float2 a[4], bn[8], bs[8], P[4][8], Q[4][8];
#pragma unroll
  for (int i = 0; i < 4; ++i) a[i] = make_float2(seed[2 * i + lane], seed[2 * i + 1 + lane]);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    bn[j] = make_float2(seed[32 + 2 * j + lane], seed[33 + 2 * j + lane]);
    bs[j] = make_float2(bn[j].y, bn[j].x);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) { P[i][j] = make_float2(0.f, 0.f); Q[i][j] = make_float2(0.f, 0.f); }

  __syncthreads();
  const long long t0 = clock64();
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int r = 0; r < kRowsPerIter; ++r) {
      // the operand traffic of one K row: NL instructions, each to its own 512-byte row
#pragma unroll
      for (int k = 0; k < NL; ++k) {
        const uint32_t addr = addr0 + (uint32_t)(((r * NL + k) & 31) * 512);
        if (KIND == kLds128) {
          float d0, d1, d2, d3;
          asm volatile("ld.volatile.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                       : "=f"(d0), "=f"(d1), "=f"(d2), "=f"(d3) : "r"(addr));
        } else if (KIND == kLds64) {
          float d0, d1;
          asm volatile("ld.volatile.shared.v2.f32 {%0, %1}, [%2];" : "=f"(d0), "=f"(d1) : "r"(addr));
        } else if (KIND == kLds32) {
          float d0;
          asm volatile("ld.volatile.shared.f32 %0, [%1];" : "=f"(d0) : "r"(addr));
        } else if (KIND == kShfl) {
          float d0;
          asm volatile("shfl.sync.idx.b32 %0, %1, %2, 0x1f, 0xffffffff;"
                       : "=f"(d0) : "f"(a[k & 3].x), "r"(src_lane));
          a[k & 3].x = d0;     // the shuffled value is an operand of the next multiply-adds
        }
      }
      // the 64 packed multiply-adds of one K row of the 8 x 16 block
      if (ORDER == 0) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
          for (int ii = 0; ii < 4; ++ii) {
            const int i = (j & 1) ? 3 - ii : ii;
            P[i][j] = __ffma2_rn(a[i], bn[j], P[i][j]);
            Q[i][j] = __ffma2_rn(a[i], bs[j], Q[i][j]);
          }
      } else if (ORDER == 1) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            P[i][j] = __ffma2_rn(a[i], bn[j], P[i][j]);
            Q[i][j] = __ffma2_rn(a[i], bs[j], Q[i][j]);
          }
      } else if (ORDER == 2) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i) P[i][j] = __ffma2_rn(a[i], bn[j], P[i][j]);
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i) Q[i][j] = __ffma2_rn(a[i], bs[j], Q[i][j]);
      } else {
#pragma unroll
        for (int rep = 0; rep < 8; ++rep)
#pragma unroll
          for (int j = 0; j < 8; ++j) P[0][j] = __ffma2_rn(a[0], bn[0], P[0][j]);
      }
    }
  }
  const long long t1 = clock64();
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) s += P[i][j].x + P[i][j].y + Q[i][j].x + Q[i][j].y;
  sink[blockIdx.x * kThreads + threadIdx.x] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// The bare multiply-add stream: 8 accumulator pairs, fixed operands, BODY packed
// multiply-adds per loop iteration (16 bytes of code each), any number of warps.  Separates
// what the loop's code size and the number of warps per scheduler do to the issue rate.
template <int BODY>
__global__ void __launch_bounds__(1024, 1)
ffma2_stream_kernel(const float* __restrict__ seed, float* __restrict__ sink, long long* cycles,
                    int iters) {
  const int lane = threadIdx.x & 31;
  const float2 a = make_float2(seed[lane], seed[lane + 1]);
  const float2 b = make_float2(seed[lane + 32], seed[lane + 33]);
  float2 acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = make_float2(0.f, 0.f);
  __syncthreads();
  const long long t0 = clock64();
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int k = 0; k < BODY; ++k) acc[k & 7] = __ffma2_rn(a, b, acc[k & 7]);
  }
  const long long t1 = clock64();
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) s += acc[j].x + acc[j].y;
  sink[blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

template <int KIND, int NL, int ORDER = 0>
cudaError_t launch(const float* seed, float* sink, long long* cycles, int blocks, int iters,
                   int map, cudaStream_t s) {
  issue_mix_kernel<KIND, NL, ORDER><<<blocks, kThreads, 0, s>>>(seed, sink, cycles, iters, map);
  return cudaGetLastError();
}

template <int KIND>
cudaError_t launch_nl(int nl, const float* seed, float* sink, long long* cycles, int blocks,
                      int iters, int map, cudaStream_t s) {
  switch (nl) {
    case 0: return launch<kNone, 0>(seed, sink, cycles, blocks, iters, map, s);
    case 2: return launch<KIND, 2>(seed, sink, cycles, blocks, iters, map, s);
    case 4: return launch<KIND, 4>(seed, sink, cycles, blocks, iters, map, s);
    case 6: return launch<KIND, 6>(seed, sink, cycles, blocks, iters, map, s);
    case 8: return launch<KIND, 8>(seed, sink, cycles, blocks, iters, map, s);
    case 12: return launch<KIND, 12>(seed, sink, cycles, blocks, iters, map, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

// The bare stream: `body` (32, 64, 128, 256, 512 or 1024) packed multiply-adds per loop
// iteration, `threads` per CTA (a multiple of 128, at most 1024), `iters` iterations; `sink`
// needs blocks x threads floats.  Other arguments and the return value as below.
extern "C" int maxdnn_ubench_ffma2_stream(int body, int threads, int blocks, int iters,
                                          const float* seed, float* sink, long long* cycles,
                                          void* cuda_stream) {
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (blocks <= 0 || iters <= 0 || threads < 128 || threads > 1024 || threads % 128)
    return (int)cudaErrorInvalidValue;
  switch (body) {
    case 32: ffma2_stream_kernel<32><<<blocks, threads, 0, s>>>(seed, sink, cycles, iters); break;
    case 64: ffma2_stream_kernel<64><<<blocks, threads, 0, s>>>(seed, sink, cycles, iters); break;
    case 128: ffma2_stream_kernel<128><<<blocks, threads, 0, s>>>(seed, sink, cycles, iters); break;
    case 256: ffma2_stream_kernel<256><<<blocks, threads, 0, s>>>(seed, sink, cycles, iters); break;
    case 512: ffma2_stream_kernel<512><<<blocks, threads, 0, s>>>(seed, sink, cycles, iters); break;
    case 1024: ffma2_stream_kernel<1024><<<blocks, threads, 0, s>>>(seed, sink, cycles, iters); break;
    default: return (int)cudaErrorInvalidValue;
  }
  return (int)cudaGetLastError();
}

// One launch of the mix on `blocks` CTAs of 256 threads: per K row 64 FFMA2 and `n_loads`
// (0, 2, 4, 6, 8 or 12) instructions of `kind` (1 LDS.128, 2 LDS.64, 3 LDS.32, 4 SHFL; kind 0 =
// multiply-adds only, n_loads then selects their order 0..3) with
// lane map `map` (0..13, see lane_word), `iters` x 4 rows.  Device pointers: `seed` 512
// floats (finite values), `sink` blocks x 256 floats, `cycles` one int64 per block (elapsed
// SM cycles of the loop).  Returns the CUDA error code of the launch (0 = launched).
extern "C" int maxdnn_ubench_issue_mix(int kind, int n_loads, int map, int blocks, int iters,
                                       const float* seed, float* sink, long long* cycles,
                                       void* cuda_stream) {
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (blocks <= 0 || iters <= 0 || map < 0 || map > 13) return (int)cudaErrorInvalidValue;
  switch (kind) {
    case kNone:   // n_loads selects the order of the multiply-adds instead (see ORDER)
      switch (n_loads) {
        case 0: return (int)launch<kNone, 0, 0>(seed, sink, cycles, blocks, iters, map, s);
        case 1: return (int)launch<kNone, 0, 1>(seed, sink, cycles, blocks, iters, map, s);
        case 2: return (int)launch<kNone, 0, 2>(seed, sink, cycles, blocks, iters, map, s);
        case 3: return (int)launch<kNone, 0, 3>(seed, sink, cycles, blocks, iters, map, s);
        default: return (int)cudaErrorInvalidValue;
      }
    case kLds128: return (int)launch_nl<kLds128>(n_loads, seed, sink, cycles, blocks, iters, map, s);
    case kLds64: return (int)launch_nl<kLds64>(n_loads, seed, sink, cycles, blocks, iters, map, s);
    case kLds32: return (int)launch_nl<kLds32>(n_loads, seed, sink, cycles, blocks, iters, map, s);
    case kShfl: return (int)launch_nl<kShfl>(n_loads, seed, sink, cycles, blocks, iters, map, s);
    default: return (int)cudaErrorInvalidValue;
  }
}
