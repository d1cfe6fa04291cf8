// Host-side planning: descriptor checks, tile choice and the K-step table
// (the address-generation stage, Section 3.2: patch offsets are precomputed so
// one flat loop replaces the nested loops over channels, rows and columns).
// Plain C++ — no CUDA calls — so it can be exercised without a GPU.
#pragma once
#include <stdint.h>

#include "../../include/maxdnn.h"

namespace maxdnn {

constexpr int kMaxKSteps = 1024;   // capacity of the table carried in kernel parameters

// Tuning and test switches (ablations, tests; none is needed in normal use).  Each has a
// name; its value is "unset" until maxdnn_set_option gives it one.  The environment
// variable MAXDNN_<NAME> supplies the initial value, read ONCE, at the first use of any
// option in the process — never on the path of a call.  TEST_MISSING_ARRIVAL is the
// exception: it has no environment variable and can only be set through the C ABI.
enum OptionId : int {
  OPT_FFMA_TILE_M = 0, OPT_FFMA_COLS, OPT_FFMA_KH, OPT_FFMA_KC, OPT_FFMA_STREAMK,
  OPT_UMMA_KC, OPT_UMMA_PAIR, OPT_UMMA_MERGE, OPT_UMMA_STAGE_KB, OPT_UMMA_COLS,
  OPT_WGRAD_SPLITS, OPT_WGRAD_PAIR, OPT_SM_COUNT, OPT_X3_CHUNK_ROWS, OPT_DEBUG_STATUS,
  OPT_KERNEL_CLOCK, OPT_RAGGED_PADDED, OPT_TEST_MISSING_ARRIVAL, OPT_COUNT
};
bool option_is_set(OptionId id);
int option(OptionId id, int unset_value = 0);          // the value, or unset_value
maxdnn_status set_option(const char* name, int value); // name without the MAXDNN_ prefix
maxdnn_status unset_option(const char* name);
maxdnn_status get_option(const char* name, int32_t* value, int32_t* is_set);
void reset_options();                                  // back to the values the environment gave
uint32_t options_generation();                         // changes whenever an option changes

// The operation with per-axis filter size, stride and padding (Section 2 has one of each:
// the public square descriptor maps to Skw = Skh = Sk and so on).
struct ConvDims {
  int32_t Nb, Wi, Hi, Nc, No, Skw, Skh, stride_w, stride_h, pad_w, pad_h;
  float alpha;
  // Host-side extras (0 = not used), for the sub-convolutions of the strided map gradient:
  // the maps are a window of a larger tensor (element pitches of its rows and channels),
  // and the number of output rows / columns is given instead of derived (the window may
  // end before or after the last full filter position; what it lacks reads as zeros).
  int64_t in_h_stride, in_c_stride;
  int32_t Ho_given, Wo_given;
  // element pitches of the result's pixels / rows / filters when it is a sub-grid of a larger
  // tensor (tensor-core kernels only: their stores go through a tensor map)
  int64_t out_x_stride, out_y_stride, out_o_stride;
};

ConvDims dims_from(const maxdnn_conv_desc& d);
maxdnn_status check_dims(const ConvDims& d, int32_t* Ho, int32_t* Wo);

// What a kernel needs to know about the problem and its tiling.  Passed by
// value in kernel parameter space together with the K-step table.
struct ConvGeom {
  int32_t Nb, Wi, Hi, Nc, No, Skw, stride_w, pad_w;   // the w-axis filter size, stride, padding
  int32_t Ho, Wo;
  float alpha;
  int32_t tile_m;     // filters per tile
  int32_t tile_px;    // adjacent output pixels (x) per tile
  int32_t tile_n;     // images per tile
  int32_t kc, kwc;    // channels / filter columns per K step
  int32_t box_c, box_kw, box_kh;   // tensor kernels: extents of the copy boxes along c, kw (w), kh (h)
  int32_t rows;       // patch rows per K step = kc * kwc
  int32_t n_ksteps;
  int32_t stages;
  int32_t o_blocks, n_chunks, x_runs;
  int32_t n_tiles;
  int32_t tile_begin, tile_end;   // tiles this launch walks: [tile_begin, tile_end)
  int32_t tile_cols;       // columns of a tile the kernel is built for (128 or 256)
  int32_t pair;            // tensor-core kernel: 1 = tiles of 256 filters on a pair of CTAs
  int32_t split_n;         // pair: 1 = the CTAs split the tile's images, 0 = its pixels
  int32_t cta_px, cta_n;   // pixels x images whose patches ONE CTA stages (= tile_px, tile_n if not pair)
  int32_t a_stage_bytes;   // filter box bytes per stage
  int32_t a_box_bytes;
  int32_t fixed_pitch;     // 1: one patch box per stage, rows 128 floats apart
  int32_t b_boxes;         // patch boxes per K step (1, or tile_px)
  int32_t b_box_w;         // extent of a patch box along w
  int32_t b_box_bytes;
  int32_t b_slot_bytes;    // distance between the windows of adjacent pixels in a stage (separate boxes, or inside one strip)
  int32_t b_stage_bytes;   // patch bytes per stage
  int32_t grid;
  int32_t smem_bytes;
  int32_t Skh, stride_h, pad_h;                       // the h-axis filter size, stride, padding
  // fp32 kernel, split tail: tiles [sk_first, tile_end) are computed by all CTAs together,
  // their sk_units = sk_tiles x n_ksteps K steps dealt out evenly (0 tiles: no split)
  int32_t sk_first, sk_tiles, sk_units;
  // fp32 kernel: K steps from short_from on hold rows_short rows (the last group of filter
  // rows of a few-channel plan whose box_kh rows per step do not divide the filter height)
  int32_t short_from, rows_short;
};

struct KStepTable {
  maxdnn_kstep s[kMaxKSteps];
};

#ifdef __CUDACC__
#define MAXDNN_HD __host__ __device__ __forceinline__
#else
#define MAXDNN_HD inline
#endif

// Work items of the fp32 kernel (see ffma_conv.cuh): a whole tile, a contribution of
// partial sums to a tile of the split tail, or the piece that finishes such a tile.
enum FfmaItemKind : int { kItemWhole = 0, kItemContribute = 1, kItemFinish = 2 };
struct FfmaItem {
  int tile, s0, s1, kind;    // K steps [s0, s1) of `tile`
};

// K-step range of CTA `cta` in the split tail: units [u0, u1) of sk_units.
MAXDNN_HD void sk_range(const ConvGeom& g, int cta, int grid, int* u0, int* u1) {
  *u0 = (int)(((long long)cta * g.sk_units) / grid);
  *u1 = (int)(((long long)(cta + 1) * g.sk_units) / grid);
}

// The k-th item of CTA `cta` of a grid of `grid` CTAs, or false when there is none.
MAXDNN_HD bool ffma_item_at(const ConvGeom& g, int grid, int cta, int k, FfmaItem& it) {
  const int first = g.tile_begin + cta;
  const int n_whole = first < g.sk_first ? (g.sk_first - first + grid - 1) / grid : 0;
  if (k < n_whole) {
    it.tile = first + k * grid; it.s0 = 0; it.s1 = g.n_ksteps; it.kind = kItemWhole;
    return true;
  }
  if (g.sk_tiles <= 0) return false;
  int u0, u1;
  sk_range(g, cta, grid, &u0, &u1);
  if (u1 <= u0) return false;
  const int n = g.n_ksteps;
  const int ta = u0 / n;                       // tile (within the tail) where the range starts
  const int a0 = u0 - ta * n;
  const bool two = u1 > (ta + 1) * n;          // the range runs on into tile ta + 1
  int piece = k - n_whole;
  if (two) {
    if (piece == 0) {                          // the contribution to the next tile comes first
      it.tile = g.sk_first + ta + 1; it.s0 = 0; it.s1 = u1 - (ta + 1) * n; it.kind = kItemContribute;
      return true;
    }
    --piece;
  }
  if (piece != 0) return false;
  it.tile = g.sk_first + ta;
  it.s0 = a0;
  it.s1 = two ? n : u1 - ta * n;
  it.kind = it.s1 < n ? kItemContribute : (a0 == 0 ? kItemWhole : kItemFinish);
  return true;
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int align_up(int a, int b) { return ceil_div(a, b) * b; }

maxdnn_status check_desc(const maxdnn_conv_desc* d, int32_t* Ho, int32_t* Wo);

// FFMA kernel plan.  force_tile_m / force_cols > 0 pin the tile shape (ablations).
// allow_split: the caller can provide the workspace of a split tail (see ffma_split_bytes).
// ragged: Nb and No need not be multiples of 4 (the kernel instance with copy warps).
maxdnn_status plan_ffma(const ConvDims& d, int sm_count, int force_tile_m, int force_cols,
                        ConvGeom* g, KStepTable* t, bool allow_split = false, bool ragged = false);

// Workspace of the fp32 kernel's split tail for any plan on `sm_count` SMs: one slot of
// partial sums per CTA (the largest tile has 32768 columns x filters), then one flag per CTA.
// Register blocks of at least this many accumulators have no producer warp: their consumer
// warps take turns at issuing the copies (see ffma_conv.cuh), and their ring has >= 3 slots.
// (Measured: the smaller blocks are 4-8 % slower without their producer warp.)
constexpr int kFfmaInlineMinAcc = 96;
constexpr size_t kFfmaSplitSlotBytes = 32768 * 4;
inline size_t ffma_split_flags_offset(int sm_count) { return (size_t)sm_count * kFfmaSplitSlotBytes; }
inline size_t ffma_split_bytes(int sm_count) {
  return ffma_split_flags_offset(sm_count) + (((size_t)sm_count * 4 + 255) & ~(size_t)255);
}

// Tensor-core kernel plan (elem_bytes 4 = TF32, 2 = BF16).
// force_pair: 0 = choose, 1 = two-SM tiles (256 filters per CTA pair), -1 = one-SM tiles.
maxdnn_status plan_umma(const ConvDims& d, int elem_bytes, int sm_count, int force_kc,
                        int force_pair, ConvGeom* g, KStepTable* t);

// ---------------------------------------------------------------------------
// Backward propagation (the adjoints of the operation; the paper names BPROP in
// its Abstract and Section 3.5 ("Conclusion") as the place its techniques should carry over to).
// ---------------------------------------------------------------------------

// Gradient with respect to the maps, stride 1: FPROP of the output gradient with
// the filter bank transposed (channels <-> filters) and flipped in both axes and
// padding Sk - 1 - pad (per axis).  Fills the dims of that FPROP.  NOT_SUPPORTED for
// a stride != 1 or a pad > Sk - 1.
maxdnn_status plan_dgrad(const ConvDims& d, ConvDims* fprop_dims);

// Gradient with respect to the maps, stride s > 1: the map positions split into s x s
// classes by (h + pad) mod s, (w + pad) mod s; a class only meets the filter taps
// kh = rho_h + s j, kw = rho_w + s i, and on its own grid (h = s a + rho_h - pad) the
// gradient is a stride-1 convolution of dout with that sub-filter: an FPROP with the
// sub-filter flipped and transposed.  One axis of one class:
struct DgradAxis {
  int32_t rho;      // residue of (position + pad) mod s
  int32_t J;        // taps of the class along this axis (0: none, the gradient is zero)
  int32_t a_min;    // first grid index whose position s a + rho - pad is inside the map
  int32_t n;        // number of grid positions inside the map
  int32_t first;    // position of grid index a_min
  int32_t pad;      // padding of the equivalent FPROP (>= 0)
  int32_t crop;     // leading rows / columns of dout that FPROP's input window skips
};
DgradAxis dgrad_axis(int rho, int Sk, int s, int pad, int size_in);

// Gradient with respect to the filters: the (Nc Sk^2) x No matrix
//   dfilt[k][o] = alpha * sum_r patch[k][r] * dout[o][r],   r = (y, x, n),
// as a GEMM whose reduction runs over output pixels and images.  One tile = up to
// 128 gradient rows (bc channels x bh filter rows x bw = Sk filter columns: one
// bulk copy of a bh x bw window of input pixels) x up to 128 filters; a reduction
// step = 32 images of one output pixel.  The reduction is split over `splits`
// CTAs per tile whose partial sums a second kernel adds in a fixed order.
struct WgradGeom {
  int32_t Nb, Wi, Hi, Nc, No, Skw, stride_w, pad_w, Ho, Wo;   // w-axis filter size, stride, padding
  float alpha;
  int32_t bc, bh, bw;        // channels x filter rows x filter columns per tile
  int32_t rows;              // bc * bh * bw <= 128
  int32_t box_o;             // filters per tile, min(128, No)
  int32_t c_blocks, kh_blocks, o_blocks;
  int32_t n_chunks;          // groups of 32 images
  int32_t r_steps;           // Ho * Wo * n_chunks
  int32_t splits, steps_per_split;
  int32_t n_items;           // tiles x splits
  int32_t stages, grid, smem_bytes;
  // tensor-core kernel on a pair of CTAs (256 filters per tile; each CTA stages its 128
  // filters and half of the tile's channels): channels / gradient rows per CTA, MMA N
  int32_t pair, bc_h, rows_h, n_mma;
  int32_t Skh, stride_h, pad_h;   // h-axis filter size, stride, padding
};

// force_splits > 0 pins the number of reduction splits (tests, ablations).
// elem_bytes 0: the fp32 FFMA2 kernel (128 gradient rows per tile, 32 images per step);
// 4 / 2: the tensor-core kernel with TF32 / BF16 operands (256 rows; 32 / 64 images).
maxdnn_status plan_wgrad(const ConvDims& d, int elem_bytes, int sm_count, int force_splits,
                         WgradGeom* g, int force_pair = 0);

}  // namespace maxdnn
