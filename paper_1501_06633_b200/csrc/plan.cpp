#include "plan.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

namespace maxdnn {

// ---------------------------------------------------------------------------
// Options: a small table of named integers (see plan.h).
// ---------------------------------------------------------------------------
namespace {
const char* const kOptionNames[OPT_COUNT] = {
    "FFMA_TILE_M", "FFMA_COLS", "FFMA_KH", "FFMA_KC", "FFMA_STREAMK",
    "UMMA_KC", "UMMA_PAIR", "UMMA_MERGE", "UMMA_STAGE_KB", "UMMA_COLS",
    "WGRAD_SPLITS", "WGRAD_PAIR", "SM_COUNT", "X3_CHUNK_ROWS", "DEBUG_STATUS",
    "KERNEL_CLOCK", "RAGGED_PADDED", "TEST_MISSING_ARRIVAL"};
struct OptionSlot {
  std::atomic<int32_t> value{0};
  std::atomic<bool> set{false};
};
OptionSlot g_opt[OPT_COUNT];
std::once_flag g_opt_once;
std::atomic<uint32_t> g_opt_gen{1};

void load_options_from_env() {
  for (int i = 0; i < OPT_COUNT; ++i) {
    g_opt[i].set.store(false);
    g_opt[i].value.store(0);
    if (i == OPT_TEST_MISSING_ARRIVAL) continue;      // never from the environment
    char name[64] = "MAXDNN_";
    strncat(name, kOptionNames[i], sizeof(name) - 8);
    if (const char* v = getenv(name)) {
      g_opt[i].value.store(atoi(v));
      g_opt[i].set.store(true);
    }
  }
}
void ensure_options() { std::call_once(g_opt_once, load_options_from_env); }
int find_option(const char* name) {
  if (!name) return -1;
  if (strncmp(name, "MAXDNN_", 7) == 0) name += 7;
  for (int i = 0; i < OPT_COUNT; ++i)
    if (strcmp(name, kOptionNames[i]) == 0) return i;
  return -1;
}
}  // namespace

bool option_is_set(OptionId id) {
  ensure_options();
  return g_opt[id].set.load(std::memory_order_relaxed);
}
int option(OptionId id, int unset_value) {
  ensure_options();
  return g_opt[id].set.load(std::memory_order_relaxed) ? g_opt[id].value.load(std::memory_order_relaxed)
                                                       : unset_value;
}
maxdnn_status set_option(const char* name, int value) {
  ensure_options();
  const int i = find_option(name);
  if (i < 0) return MAXDNN_INVALID_VALUE;
  g_opt[i].value.store(value);
  g_opt[i].set.store(true);
  g_opt_gen.fetch_add(1);
  return MAXDNN_OK;
}
maxdnn_status unset_option(const char* name) {
  ensure_options();
  const int i = find_option(name);
  if (i < 0) return MAXDNN_INVALID_VALUE;
  g_opt[i].set.store(false);
  g_opt[i].value.store(0);
  g_opt_gen.fetch_add(1);
  return MAXDNN_OK;
}
maxdnn_status get_option(const char* name, int32_t* value, int32_t* is_set) {
  ensure_options();
  const int i = find_option(name);
  if (i < 0) return MAXDNN_INVALID_VALUE;
  if (value) *value = g_opt[i].value.load();
  if (is_set) *is_set = g_opt[i].set.load() ? 1 : 0;
  return MAXDNN_OK;
}
void reset_options() {
  ensure_options();
  load_options_from_env();
  g_opt_gen.fetch_add(1);
}
uint32_t options_generation() {
  ensure_options();
  return g_opt_gen.load(std::memory_order_relaxed);
}

maxdnn_status check_desc(const maxdnn_conv_desc* d, int32_t* Ho, int32_t* Wo) {
  if (!d) return MAXDNN_INVALID_VALUE;
  if (d->Nb <= 0 || d->Wi <= 0 || d->Hi <= 0 || d->Nc <= 0 || d->No <= 0 || d->Sk <= 0 ||
      d->stride <= 0 || d->pad < 0)
    return MAXDNN_INVALID_VALUE;
  if (!isfinite(d->alpha)) return MAXDNN_INVALID_VALUE;
  const int64_t span_h = (int64_t)d->Hi + 2 * (int64_t)d->pad - d->Sk;
  const int64_t span_w = (int64_t)d->Wi + 2 * (int64_t)d->pad - d->Sk;
  if (span_h < 0 || span_w < 0) return MAXDNN_INVALID_VALUE;
  if (Ho) *Ho = (int32_t)(span_h / d->stride + 1);
  if (Wo) *Wo = (int32_t)(span_w / d->stride + 1);
  return MAXDNN_OK;
}

ConvDims dims_from(const maxdnn_conv_desc& d) {
  ConvDims c;
  c.Nb = d.Nb; c.Wi = d.Wi; c.Hi = d.Hi; c.Nc = d.Nc; c.No = d.No;
  c.Skw = c.Skh = d.Sk; c.stride_w = c.stride_h = d.stride; c.pad_w = c.pad_h = d.pad;
  c.alpha = d.alpha;
  c.in_h_stride = c.in_c_stride = 0;
  c.Ho_given = c.Wo_given = 0;
  c.out_x_stride = c.out_y_stride = c.out_o_stride = 0;
  return c;
}

maxdnn_status check_dims(const ConvDims& d, int32_t* Ho, int32_t* Wo) {
  if (d.Nb <= 0 || d.Wi <= 0 || d.Hi <= 0 || d.Nc <= 0 || d.No <= 0 || d.Skw <= 0 || d.Skh <= 0 ||
      d.stride_w <= 0 || d.stride_h <= 0 || d.pad_w < 0 || d.pad_h < 0)
    return MAXDNN_INVALID_VALUE;
  if (!isfinite(d.alpha)) return MAXDNN_INVALID_VALUE;
  if (d.Ho_given > 0 && d.Wo_given > 0) {      // output size stated by the caller
    if (Ho) *Ho = d.Ho_given;
    if (Wo) *Wo = d.Wo_given;
    return MAXDNN_OK;
  }
  const int64_t span_h = (int64_t)d.Hi + 2 * (int64_t)d.pad_h - d.Skh;
  const int64_t span_w = (int64_t)d.Wi + 2 * (int64_t)d.pad_w - d.Skw;
  if (span_h < 0 || span_w < 0) return MAXDNN_INVALID_VALUE;
  if (Ho) *Ho = (int32_t)(span_h / d.stride_h + 1);
  if (Wo) *Wo = (int32_t)(span_w / d.stride_w + 1);
  return MAXDNN_OK;
}

DgradAxis dgrad_axis(int rho, int Sk, int s, int pad, int size_in) {
  DgradAxis c;
  c.rho = rho;
  c.J = rho < Sk ? (Sk - rho + s - 1) / s : 0;
  // positions s a + rho - pad in [0, size_in):  a >= (pad - rho) / s  (pad - rho > -s)
  c.a_min = pad > rho ? (pad - rho + s - 1) / s : 0;
  const int top = size_in - 1 + pad - rho;                 // s a <= top
  const int a_max = top >= 0 ? top / s : -1;
  c.n = a_max >= c.a_min ? a_max - c.a_min + 1 : 0;
  c.first = s * c.a_min + rho - pad;
  // grid index a reads dout rows a - J + 1 .. a: FPROP's window of output a - a_min starts at
  // (a - a_min) - pad, so pad = J - 1 - a_min; a negative value skips rows instead
  const int p = c.J - 1 - c.a_min;
  c.pad = p > 0 ? p : 0;
  c.crop = p < 0 ? -p : 0;
  return c;
}

static maxdnn_status common_limits(const ConvDims& d, int elem_bytes) {
  if (d.Skw > 127 || d.Skh > 127 || d.Nc > 32767) return MAXDNN_NOT_SUPPORTED;
  // Row pitches of the tensor-copy descriptors are 32-bit-safe byte counts here.
  const int64_t plane = (int64_t)d.Hi * d.Wi * d.Nb * elem_bytes;
  const int64_t frow = (int64_t)d.Skh * d.Skw * d.No * elem_bytes;
  if (plane >= ((int64_t)1 << 40) || frow >= ((int64_t)1 << 40)) return MAXDNN_NOT_SUPPORTED;
  const int64_t out_elems = (int64_t)d.No * d.Nb;
  if (out_elems <= 0) return MAXDNN_INVALID_VALUE;
  return MAXDNN_OK;
}

// Copies the problem into the geometry the kernels read.
static void fill_geom(const ConvDims& d, int32_t Ho, int32_t Wo, ConvGeom* g) {
  memset(g, 0, sizeof(*g));
  g->Nb = d.Nb; g->Wi = d.Wi; g->Hi = d.Hi; g->Nc = d.Nc; g->No = d.No;
  g->Skw = d.Skw; g->Skh = d.Skh; g->stride_w = d.stride_w; g->stride_h = d.stride_h;
  g->pad_w = d.pad_w; g->pad_h = d.pad_h; g->alpha = d.alpha; g->Ho = Ho; g->Wo = Wo;
}

// Tile shapes the fp32 kernel is built for, with the relative cost per
// multiply-accumulate measured for each on layers that fill the tile (smaller register
// blocks spend a larger share of issue slots on operand loads; with 16 rows of K per loop
// iteration and K steps of 64 or 96 rows the 8 x 8 block is ahead of the blocks of 128
// accumulators, whose rows of 1.5 KB leave room for steps of 32 to 48 rows only).
constexpr int kFfmaSmemBudget = 224 * 1024;   // ring stages of a CTA (227 KB is the device's limit)
struct FfmaShape { int m, cols; double cost; };
static const FfmaShape kFfmaShapes[] = {
    {128, 256, 1.000}, {256, 128, 1.010}, {128, 128, 0.980}, {96, 128, 1.025},
    {96, 256, 1.09},   {64, 128, 1.165},  {64, 256, 1.063},  {32, 128, 2.03},
};

static void build_table(const ConvDims& d, int kc, int kwc, KStepTable* t, int* n, int khc = 1) {
  int k = 0;
  for (int kh = 0; kh < d.Skh; kh += khc)
    for (int kw0 = 0; kw0 < d.Skw; kw0 += kwc)
      for (int c0 = 0; c0 < d.Nc; c0 += kc) {
        if (k < kMaxKSteps) {
          t->s[k].c0 = (int16_t)c0;
          t->s[k].kh = (int8_t)kh;
          t->s[k].kw0 = (int8_t)kw0;
        }
        ++k;
      }
  *n = k;
}

// Columns of a tile: tile_px adjacent output pixels x tile_n images <= cols.
static double pick_columns(const ConvDims& d, int Wo, int cols, int* nn_out, int* T_out) {
  int best_nn = 4, best_T = 1;
  double best_eff = -1.0;
  const int nb4 = align_up(d.Nb, 4);       // (ragged counts: the tile's images round up)
  for (int nn = (nb4 < cols ? nb4 : cols); nn >= 4; nn -= 4) {
    int T = cols / nn;
    if (T > Wo) T = Wo;
    const double eff =
        ((double)d.Nb * Wo) / ((double)ceil_div(d.Nb, nn) * ceil_div(Wo, T) * (double)cols);
    if (eff > best_eff + 1e-9) { best_eff = eff; best_nn = nn; best_T = T; }
  }
  *nn_out = best_nn;
  *T_out = best_T;
  return best_eff;
}

// K step of the fp32 kernel: kc channels of one filter tap, or (few channels) kc channels
// of a whole filter row of Skw taps.
static void ffma_kstep(const ConvDims& d, int kc_max, int* kc_out, int* kwc_out, int* khc_out) {
  int kc, kwc, khc = 1;
  if (d.Nc >= 8) {
    kwc = 1;
    if (option_is_set(OPT_FFMA_KC)) {
      const int v = option(OPT_FFMA_KC);
      if (v >= 8 && v <= 128 && v % 4 == 0 && v < kc_max) kc_max = v;   // an upper limit
    }
    kc = kc_max;
    int best_pad = 1 << 30;
    for (int c = kc_max; c >= 8; c -= 4) {
      const int padded = ceil_div(d.Nc, c) * c;
      if (padded < best_pad) { best_pad = padded; kc = c; }
    }
  } else {
    kwc = d.Skw;
    kc = 40 / d.Skw;
    if (kc < 1) kc = 1;
    if (kc > d.Nc) kc = d.Nc;
    // Several filter rows per step where one row is short (33 K rows for 11 x 11 x 3): every
    // step costs the consumers a barrier round trip and loop tails, a third of the
    // instructions on that layer.  About 100 rows per step (two ring stages) measured best.
    khc = 100 / (kc * kwc);
    if (option_is_set(OPT_FFMA_KH)) khc = option(OPT_FFMA_KH);
    if (khc < 1) khc = 1;
    if (khc > d.Skh) khc = d.Skh;
  }
  *kc_out = kc;
  *kwc_out = kwc;
  *khc_out = khc;
}

// Time of `tiles` tiles on `units` persistent CTAs, in tile times.  Without a split the
// last, partly filled wave costs a whole tile time.  With the tail split along K (see
// ffma_conv.cuh) it costs its share R / units plus the fix-up: every CTA writes or reads
// back partial sums (a tile's accumulators: about 16 K rows' worth of time per slot) and a
// finisher adds about units / R slots one after the other.
static double ffma_waves(int64_t tiles, int units, int k_rows_per_tile, bool allow_split,
                         bool* split_out) {
  const int64_t W = tiles / units, R = tiles % units;
  *split_out = false;
  if (R == 0) return (double)W;
  const double whole = (double)(W + 1);
  if (!allow_split) return whole;
  if (option(OPT_FFMA_STREAMK, 1) == 2) { *split_out = true; return whole - 0.5; }   // forced (tests)
  if (k_rows_per_tile < 512) return whole;   // short sums: the fix-up eats the gain
  const double slot = 16.0 / (double)k_rows_per_tile;
  const double split = (double)W + (double)R / units + 0.03 + slot * (1.0 + (double)units / (double)R);
  if (split < whole - 0.03) { *split_out = true; return split; }
  return whole;
}

maxdnn_status plan_ffma(const ConvDims& d, int sm_count, int force_tile_m, int force_cols,
                        ConvGeom* g, KStepTable* t, bool allow_split, bool ragged) {
  int32_t Ho, Wo;
  maxdnn_status st = check_dims(d, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  st = common_limits(d, 4);
  if (st != MAXDNN_OK) return st;
  if (!ragged && (d.Nb % 4 != 0 || d.No % 4 != 0)) return MAXDNN_NOT_SUPPORTED;
  if (sm_count <= 0) return MAXDNN_INVALID_VALUE;
  fill_geom(d, Ho, Wo, g);
  if (ragged) allow_split = false;

  // Tile shape: fewest SM-time units over the waves of persistent CTAs.
  double best_t = 1e300;
  int best_m = 0, best_cols = 0, best_nn = 0, best_T = 0;
  bool best_split = false;
  int kc0, kwc0, khc0;
  ffma_kstep(d, 32, &kc0, &kwc0, &khc0);
  const int k_rows = ceil_div(d.Nc, kc0) * kc0 * d.Skw * d.Skh;
  if (option(OPT_FFMA_STREAMK, 1) == 0) allow_split = false;
  for (const FfmaShape& sh : kFfmaShapes) {
    if (force_tile_m > 0 && sh.m != force_tile_m) continue;
    if (force_cols > 0 && sh.cols != force_cols) continue;
    // the ragged kernel is built for the blocks that leave room for two copy warps
    if (ragged && (sh.cols != 128 || sh.m > 128 || sh.m == 96)) continue;
    if (force_tile_m <= 0 && sh.m > align_up(d.No, 32) && sh.m != 32) continue;
    int nn, T;
    pick_columns(d, Wo, sh.cols, &nn, &T);
    if (force_cols <= 0 && sh.cols > 128 && nn * T <= 128) continue;   // would not fill it
    const int64_t tiles = (int64_t)ceil_div(d.No, sh.m) * ceil_div(Wo, T) * Ho * ceil_div(d.Nb, nn);
    bool split = false;
    const double waves = ffma_waves(tiles, sm_count, k_rows, allow_split && tiles > sm_count, &split);
    // few-channel layers: the 256-column tiles have shorter K steps (ring budget) and one
    // box per pixel; measured 3-12 % behind the 128-column tiles of the same height
    const double few = (d.Nc < 8 && sh.cols > 128) ? 1.15 : 1.0;
    const double tm = waves * sh.m * sh.cols * sh.cost * few;
    if (tm < best_t - 1e-9) {
      best_t = tm; best_m = sh.m; best_cols = sh.cols; best_nn = nn; best_T = T; best_split = split;
    }
  }
  if (best_m == 0) return MAXDNN_NOT_SUPPORTED;
  g->tile_m = best_m;
  g->tile_cols = best_cols;
  g->tile_n = best_nn;
  g->tile_px = best_T;
  g->n_chunks = ceil_div(d.Nb, best_nn);
  g->x_runs = ceil_div(Wo, best_T);
  g->o_blocks = ceil_div(d.No, best_m);
  const int64_t tiles = (int64_t)g->o_blocks * g->x_runs * Ho * g->n_chunks;
  if (tiles > 0x7fffffff) return MAXDNN_NOT_SUPPORTED;
  g->n_tiles = (int32_t)tiles;
  g->tile_begin = 0;
  g->tile_end = g->n_tiles;

  // K step: kc channels of one filter tap, or (few channels) kc channels of a
  // whole filter row of Sk taps.
  // two ring stages must fit (three where a consumer warp issues the copies)
  const bool inline_producer = !ragged && (best_m / 16) * (best_cols / 16) >= kFfmaInlineMinAcc;
  const int min_stages = inline_producer ? 3 : 2;
  // Many-channel layers: as many channels per step as leave that many stages — every step
  // costs the consumers a barrier round trip, pointer rebuilds and loop tails (about 200
  // instructions per warp), so long steps pay: 128 x 128 tiles with 64- or 96-row steps run
  // 2-3 % faster than with 32-row steps (and than the 128 x 256 tiles, whose 1.5 KB rows
  // leave room for 48).  The ragged kernel keeps 32.
  int kc_max = 32;
  if (!ragged) {
    kc_max = (kFfmaSmemBudget / (min_stages * (best_m + best_cols) * 4)) & ~3;
    if (kc_max > 112) kc_max = 112;
    if (kc_max < 32) kc_max = 32;
  }
  ffma_kstep(d, kc_max, &kc0, &kwc0, &khc0);
  int kc = kc0, kwc = kwc0;
  int khc = khc0;
  while (khc > 1 && min_stages * kc * kwc * khc * (best_m + best_cols) * 4 > kFfmaSmemBudget) --khc;
  int n = 0;
  build_table(d, kc, kwc, t, &n, khc);
  while (n > kMaxKSteps && kwc == 1 && kc < 256) {   // very deep filters: larger boxes
    kc *= 2;
    build_table(d, kc, kwc, t, &n);
  }
  if (n > kMaxKSteps) return MAXDNN_NOT_SUPPORTED;
  g->kc = kc; g->kwc = kwc; g->box_kh = khc; g->rows = kc * kwc * khc; g->n_ksteps = n;
  // The steps of the last group of filter rows are short when khc does not divide Skh
  // (the boxes' surplus filter rows are zeros; the consumers skip them).
  g->short_from = n;
  g->rows_short = g->rows;
  if (d.Skh % khc != 0) {
    const int per_group = n / ceil_div(d.Skh, khc);
    g->short_from = n - per_group;
    g->rows_short = kc * kwc * (d.Skh % khc);
  }

  g->a_box_bytes = g->rows * g->tile_m * 4;
  g->a_stage_bytes = g->a_box_bytes;
  // One box per stage whenever the tile's columns are one contiguous run of the map
  // (one pixel, or adjacent pixels of a stride-1 layer); else one box per pixel.
  g->fixed_pitch = (!ragged && g->tile_px * g->tile_n == g->tile_cols &&
                    (g->tile_px == 1 || (d.stride_w == 1 && kwc == 1))) ? 1 : 0;
  if (g->fixed_pitch) {
    g->b_boxes = 1;
    g->b_box_w = g->tile_px > 1 ? g->tile_px : kwc;
    g->b_box_bytes = g->rows * g->tile_cols * 4;
    g->b_slot_bytes = g->b_box_bytes;
    g->b_stage_bytes = g->b_box_bytes;
  } else {
    g->b_boxes = g->tile_px;
    g->b_box_w = kwc;
    g->b_box_bytes = g->rows * g->tile_n * 4;
    g->b_slot_bytes = align_up(g->b_box_bytes, 128);
    g->b_stage_bytes = g->b_slot_bytes * g->tile_px;
  }
  const int stage = g->a_stage_bytes + g->b_stage_bytes;
  int stages = kFfmaSmemBudget / stage;
  if (stages > 8) stages = 8;
  if (stages < (inline_producer ? 3 : 2)) return MAXDNN_NOT_SUPPORTED;
  g->stages = stages;
  g->smem_bytes = stages * stage + 1024;   // + barriers, + slack for alignment
  g->grid = g->n_tiles < sm_count ? g->n_tiles : sm_count;
  // Split tail: the tiles of the last, partly filled wave (whole K steps of the table are
  // dealt out, so there must be at least one for every CTA).
  g->sk_first = g->n_tiles;
  g->sk_tiles = 0;
  g->sk_units = 0;
  const int tail = g->n_tiles % g->grid;
  if (best_split && g->n_tiles > g->grid && tail > 0 && (int64_t)tail * n >= (int64_t)g->grid &&
      (size_t)best_m * best_cols * 4 <= kFfmaSplitSlotBytes) {
    g->sk_tiles = tail;
    g->sk_first = g->n_tiles - tail;
    g->sk_units = tail * n;
  }
  return MAXDNN_OK;
}

static maxdnn_status plan_umma_as(const ConvDims& d, int elem_bytes, int sm_count,
                                  int force_kc, bool pair, int max_cols, ConvGeom* g,
                                  KStepTable* t) {
  int32_t Ho, Wo;
  maxdnn_status st = check_dims(d, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  st = common_limits(d, elem_bytes);
  if (st != MAXDNN_OK) return st;
  if (elem_bytes != 4 && elem_bytes != 2) return MAXDNN_INVALID_VALUE;
  const int atom = 128 / elem_bytes;          // elements per 128-byte swizzled row
  if (d.Nb % atom != 0) return MAXDNN_NOT_SUPPORTED;
  if (d.No % 32 != 0) return MAXDNN_NOT_SUPPORTED;
  if (sm_count <= 0) return MAXDNN_INVALID_VALUE;
  fill_geom(d, Ho, Wo, g);

  // Columns of a tile: tile_px adjacent pixels x tile_n images <= 256 (the MMA's N).
  int best_nn = atom, best_T = 1;
  double best_eff = -1.0;
  for (int nn = (d.Nb < max_cols ? d.Nb : max_cols) / atom * atom; nn >= atom; nn -= atom) {
    int T = max_cols / nn;
    if (T > Wo) T = Wo;
    const double eff = ((double)d.Nb * Wo) /
                       ((double)ceil_div(d.Nb, nn) * ceil_div(Wo, T) * (double)max_cols);
    if (eff > best_eff + 1e-9) { best_eff = eff; best_nn = nn; best_T = T; }
  }
  // Few-channel layers (Nc below the MMA's K: the 3-channel first layers): a K step per
  // tap would be mostly zero padding (3 of 16 rows), so the filter COLUMNS are merged
  // into the K dimension.  One box of box_kw pixels x box_c channels per output pixel and
  // filter row lands as box_kw * box_c consecutive K rows, the filter box in the same
  // (kw, c) order; box_c >= Nc and box_kw >= Sk are rounded up so that the row count is
  // a multiple of the MMA's K, the surplus rows being out-of-bounds zeros in the filter
  // operand (c >= Nc in both, kw >= Sk in the filter box).  11 x 11 x 3: 33 of 48 rows
  // carry data instead of 3 of 16.  Needs one 128-byte group of images per tile column
  // group, so the tile is 256 / atom pixels x atom images.
  const int umma_k0 = 32 / elem_bytes;
  // Also taken just above the MMA's K where a step per tap would be less than two thirds
  // data (9 or 10 channels in tf32 — the three-product mode of a 3-channel layer — 17 to
  // 21 in bf16).
  const bool few = d.Nc < umma_k0 ||
                   (d.Nc < 2 * umma_k0 && 3 * d.Nc < 2 * align_up(d.Nc, umma_k0));
  const bool merged = few && d.Skw > 1 && !pair && force_kc == 0 && option(OPT_UMMA_MERGE, 0) >= 0;
  if (merged) {
    best_nn = atom;
    best_T = max_cols / atom < Wo ? max_cols / atom : Wo;
  }
  g->tile_n = best_nn;
  g->tile_px = best_T;
  g->n_chunks = ceil_div(d.Nb, best_nn);
  g->x_runs = ceil_div(Wo, best_T);
  // Two-SM tiles: 256 filters per pair of CTAs.  Each CTA stages its 128 filters and
  // HALF of the tile's patch columns, which cuts the bytes staged per SM and per FLOP -
  // the shared-memory fill rate is what bounds the one-SM kernel.  The columns are
  // split by image when the tile holds at least two 128-byte groups of images (the
  // strip of a split image range is shorter than two strips of split pixels), else by
  // pixel.
  g->pair = pair ? 1 : 0;
  g->tile_m = pair ? 256 : 128;
  g->o_blocks = ceil_div(d.No, g->tile_m);
  g->cta_px = g->tile_px;
  g->cta_n = g->tile_n;
  if (pair) {
    if (sm_count < 2) return MAXDNN_NOT_SUPPORTED;
    if (g->tile_n % (2 * atom) == 0) {
      g->split_n = 1;
      g->cta_n = g->tile_n / 2;
    } else if (g->tile_px % 2 == 0) {
      g->cta_px = g->tile_px / 2;
    } else {
      return MAXDNN_NOT_SUPPORTED;
    }
  }
  const int px_cta = g->cta_px;
  const int64_t tiles = (int64_t)g->o_blocks * g->x_runs * Ho * g->n_chunks;
  if (tiles > 0x7fffffff) return MAXDNN_NOT_SUPPORTED;
  g->n_tiles = (int32_t)tiles;
  g->tile_begin = 0;
  g->tile_end = g->n_tiles;
  g->tile_cols = max_cols;

  // K step.  Stride-1 layers with a small filter stage, per filter row, ONE strip of
  // tile_px + Sk - 1 pixels that serves all Sk filter columns (each column's window
  // is the strip shifted by one pixel), which cuts the patch traffic from L2 by up
  // to Sk x; otherwise one step = kc channels of one tap.  kc is a multiple of the
  // MMA's K (32 bytes of channel index: 8 for 4-byte, 16 for 2-byte elements).
  const int umma_k = 32 / elem_bytes;
  const int cols = px_cta * g->cta_n;                     // patch columns one CTA stages
  int kwc = (d.stride_w == 1 && d.Skw > 1 && d.Skw <= 5 && force_kc >= 0) ? d.Skw : 1;
  // A K step costs the issuing warps a fixed few hundred cycles, so a step should carry
  // many MMAs.  With the strip, a stage of up to 96 KB (two stages) pays off when it holds
  // at least 9 (bf16) / 12 (tf32) MMAs (measured on the 3x3 / 5x5 layers); otherwise one
  // tap per step and 48 KB stages (four or more stages).
  int stage_budget = kwc > 1 ? 96 * 1024 : 48 * 1024;
  if (option_is_set(OPT_UMMA_STAGE_KB)) { const int v = option(OPT_UMMA_STAGE_KB); if (v >= 16 && v <= 96) stage_budget = v * 1024; }
  auto stage_bytes = [&](int c) {
    return (kwc * 128 + (kwc > 1 ? (px_cta + kwc - 1) * g->cta_n : cols)) * c * elem_bytes;
  };
  // channels per step: at most 128 bytes' worth (32 tf32 / 64 bf16), within the stage
  // budget, with the least zero padding of the channel count
  auto pick_kc = [&]() {
    int kc_max = 128 / elem_bytes;
    while (kc_max > umma_k && stage_bytes(kc_max) > stage_budget) kc_max -= umma_k;
    int best = kc_max, best_pad = 1 << 30;
    for (int c = kc_max; c >= umma_k; c -= umma_k) {
      const int padded = ceil_div(d.Nc, c) * c;
      // the K-step table has room for kMaxKSteps steps (one per tap or filter row and block)
      if ((int64_t)ceil_div(d.Nc, c) * d.Skh * (kwc > 1 ? 1 : d.Skw) > kMaxKSteps && c != kc_max) continue;
      if (padded < best_pad) { best_pad = padded; best = c; }
    }
    return best;
  };
  int kc = pick_kc();
  const int min_mmas = elem_bytes == 2 ? 9 : 12;
  if (kwc > 1 && (kwc * (kc / umma_k) < min_mmas || stage_bytes(kc) > stage_budget) &&
      !option_is_set(OPT_UMMA_STAGE_KB)) {
    kwc = 1;
    stage_budget = 48 * 1024;
    kc = pick_kc();
  }
  if (force_kc > 0 && force_kc % umma_k == 0 && force_kc <= 256) kc = force_kc;
  int n = 0;
  bool merged_strip = false;
  int strip_w = 0;
  if (merged) {
    const int box_c = align_up(d.Nc, 4);
    // A filter row whose stage would not leave two ring stages is cut into as few parts
    // of box_kw filter columns as do (every part re-reads the strip's overlap), one K step each (the copies of a part start at its
    // first column; columns past the filter read zeros in the filter operand).
    int box_kw = d.Skw, kw_parts = 1;
    for (int parts = 1; parts <= d.Skw; ++parts) {
      int w = ceil_div(d.Skw, parts);
      while ((w * box_c) % umma_k != 0) ++w;
      const int sw = w + (px_cta - 1) * d.stride_w;
      const bool strip_ok = px_cta > 1 && (d.stride_w * box_c) % 8 == 0 && d.stride_w < w && sw <= 256;
      const int b_rows = strip_ok ? sw * box_c * (g->cta_n / atom) : cols / atom * w * box_c;
      box_kw = w;
      kw_parts = ceil_div(d.Skw, w);
      if ((128 / atom * w * box_c + b_rows) * 128 <= 96 * 1024) break;   // two stages fit
    }
    const int rows1 = box_kw * box_c;                     // K rows of one filter row (or part of it)
    // The windows of adjacent output pixels overlap (stride < Sk), so ONE box of
    // box_kw + (pixels - 1) * stride columns serves all pixels of the tile: pixel j's
    // operand starts j * stride * box_c rows into it, which the swizzle allows when that
    // is a whole number of 8-row groups.  11 x 11 stride 4: 24 columns instead of 4 x 12.
    strip_w = box_kw + (px_cta - 1) * d.stride_w;
    merged_strip = px_cta > 1 && (d.stride_w * box_c) % 8 == 0 && d.stride_w < box_kw &&
                   strip_w <= 256;
    const int b_rows1 = merged_strip ? strip_w * box_c * (g->cta_n / atom) : cols / atom * rows1;
    int khc = 1;   // filter rows per step: stages of at most 40 KB (a deep ring beat longer steps)
    while (kw_parts == 1 && khc < d.Skh && (128 / atom * rows1 + b_rows1) * 128 * (khc + 1) <= 40 * 1024) ++khc;
    if (option_is_set(OPT_UMMA_MERGE)) { const int v = option(OPT_UMMA_MERGE); if (v >= 1 && v <= d.Skh && kw_parts == 1) khc = v; }
    if (box_kw > 256 || rows1 * khc > 1024) return MAXDNN_NOT_SUPPORTED;
    // with the strip the rows of one filter row are contiguous in both operands, the
    // filter rows of a step are not (strip_w vs box_kw columns apart): kc counts the
    // rows of one filter row and the MMA warp's outer loop (kwc) walks the filter rows
    kc = merged_strip ? rows1 : rows1 * khc;
    kwc = merged_strip ? khc : 1;
    for (int kh = 0; kh < d.Skh; kh += khc)
      for (int part = 0; part < kw_parts; ++part) {
        if (n >= kMaxKSteps) return MAXDNN_NOT_SUPPORTED;
        t->s[n].c0 = 0; t->s[n].kh = (int8_t)kh; t->s[n].kw0 = (int8_t)(part * box_kw);
        ++n;
      }
    g->box_c = box_c; g->box_kw = box_kw; g->box_kh = khc;
  } else {
    build_table(d, kc, kwc, t, &n);
    g->box_c = kc; g->box_kw = kwc; g->box_kh = 1;
  }
  if (n > kMaxKSteps) return MAXDNN_NOT_SUPPORTED;
  g->kc = kc; g->kwc = kwc; g->rows = kc * kwc; g->n_ksteps = n;

  g->a_box_bytes = atom * kc * kwc * elem_bytes;        // one group of filters: kwc x kc rows x 128 B
  g->a_stage_bytes = 128 * kc * kwc * elem_bytes;
  const int strip = px_cta + kwc - 1;
  if (merged_strip) {
    g->b_boxes = 1;
    g->b_box_w = strip_w;
    g->b_box_bytes = strip_w * g->box_c * g->box_kh * g->cta_n * elem_bytes;
    g->b_stage_bytes = g->b_box_bytes;
  } else if (merged) {
    g->b_boxes = px_cta;                                // one window per output pixel
    g->b_box_w = g->box_kw;
    g->b_box_bytes = g->cta_n * kc * elem_bytes;
    g->b_stage_bytes = px_cta * g->b_box_bytes;
  } else if (kwc > 1) {
    g->b_boxes = 1;
    g->b_box_w = strip;
    g->b_box_bytes = strip * g->cta_n * kc * elem_bytes;
    g->b_stage_bytes = g->b_box_bytes;
  } else if (px_cta == 1 || d.stride_w == 1) {
    g->b_boxes = 1;
    g->b_box_w = px_cta;
    g->b_box_bytes = cols * kc * elem_bytes;
    g->b_stage_bytes = g->b_box_bytes;
  } else {
    g->b_boxes = px_cta;
    g->b_box_w = 1;
    g->b_box_bytes = g->cta_n * kc * elem_bytes;
    g->b_stage_bytes = cols * kc * elem_bytes;
  }
  g->b_slot_bytes = g->b_box_bytes;
  if (merged_strip) g->b_slot_bytes = d.stride_w * g->box_c * g->cta_n * elem_bytes;   // window to window
  const int stage = g->a_stage_bytes + g->b_stage_bytes;
  const int fixed = 8 * 4096 + 1024 + 512;    // epilogue staging, alignment slack, barriers
  int stages = (227 * 1024 - fixed) / stage;
  if (stages > 8) stages = 8;
  if (stages < 2) return MAXDNN_NOT_SUPPORTED;
  g->stages = stages;
  g->smem_bytes = stages * stage + fixed;
  if (pair) {
    const int pairs = sm_count / 2;
    g->grid = 2 * (g->n_tiles < pairs ? g->n_tiles : pairs);
  } else {
    g->grid = g->n_tiles < sm_count ? g->n_tiles : sm_count;
  }
  return MAXDNN_OK;
}

maxdnn_status plan_umma(const ConvDims& d, int elem_bytes, int sm_count, int force_kc,
                        int force_pair, ConvGeom* g, KStepTable* t) {
  // Candidates: tiles of at most 256 / 192 / 128 columns, on one SM or on a pair.  A
  // tile's time goes with (columns + 128) — the 128 filter rows are staged whatever the
  // columns — and a pair's tile (twice the work on twice the SMs) takes about 0.9 of
  // that where its steps are long enough (at least four MMAs each); the plan that
  // needs the least (waves of tiles) x (tile time) wins; a narrower tile has to win by 5 %.
  // (Measured: the 13 x 13 Alexnet layers gain 14-24 % from 192-column tiles, the 5 x 5
  // and long-K 3 x 3 layers 5-20 % from pairs.)  MAXDNN_UMMA_COLS / the pair argument
  // pin a choice.
  int cols_list[3] = {256, 192, 128};
  int n_cols = 3;
  if (option_is_set(OPT_UMMA_COLS)) {
    const int v = option(OPT_UMMA_COLS);
    if (v >= 32 && v <= 256 && v % 32 == 0) { cols_list[0] = v; n_cols = 1; }
  }
  static thread_local ConvGeom gc;
  static thread_local KStepTable tc;
  maxdnn_status first = MAXDNN_NOT_SUPPORTED;
  double best = 1e300;
  bool have = false;
  const bool peer_has_filters = (d.No % 256 == 0) || (d.No % 256 > 128);   // in every tile
  for (int ci = 0; ci < n_cols; ++ci) {
    for (int pair = 0; pair < 2; ++pair) {
      if ((force_pair > 0 && !pair) || (force_pair < 0 && pair)) continue;
      const maxdnn_status st = plan_umma_as(d, elem_bytes, sm_count, force_kc, pair != 0,
                                            cols_list[ci], &gc, &tc);
      if (ci == 0 && pair == (force_pair > 0 ? 1 : 0)) first = st;
      if (st != MAXDNN_OK) continue;
      if (pair && force_pair == 0) {
        const int mmas_per_step = gc.kwc * (gc.kc / (32 / elem_bytes));
        if (mmas_per_step < 4 || !peer_has_filters) continue;
      }
      const int units = pair ? sm_count / 2 : sm_count;
      const double cost = (double)ceil_div(gc.n_tiles, units) * (gc.tile_px * gc.tile_n + 128) *
                          (pair ? 0.9 : 1.0);
      // a narrower tile must promise at least 5 % where its K steps are short (measured:
      // 27 x 27, 64 channels, tf32, four MMAs per step: 192-column pair tiles 9 % slower
      // than the model's 2.8 % gain), 1 % where they are long (96 channels, 15 MMAs: 4 % faster)
      const int mmas = gc.kwc * (gc.kc / (32 / elem_bytes));
      const double bar = mmas >= 12 ? 0.99 : 0.95;
      if (!have || cost < (ci == 0 ? best - 1e-9 : bar * best)) {
        best = cost;
        have = true;
        *g = gc;
        *t = tc;
      }
    }
  }
  return have ? MAXDNN_OK : first;
}

maxdnn_status plan_dgrad(const ConvDims& d, ConvDims* f) {
  int32_t Ho, Wo;
  maxdnn_status st = check_dims(d, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  if (!f) return MAXDNN_INVALID_VALUE;
  if (d.stride_w != 1 || d.stride_h != 1 || d.pad_w > d.Skw - 1 || d.pad_h > d.Skh - 1)
    return MAXDNN_NOT_SUPPORTED;
  *f = d;
  f->Wi = Wo; f->Hi = Ho; f->Nc = d.No; f->No = d.Nc;
  f->pad_w = d.Skw - 1 - d.pad_w; f->pad_h = d.Skh - 1 - d.pad_h;
  f->in_h_stride = f->in_c_stride = 0;
  f->Ho_given = f->Wo_given = 0;
  f->out_x_stride = f->out_y_stride = f->out_o_stride = 0;
  return MAXDNN_OK;
}

maxdnn_status plan_wgrad(const ConvDims& d, int elem_bytes, int sm_count, int force_splits,
                         WgradGeom* g, int force_pair) {
  int32_t Ho, Wo;
  maxdnn_status st = check_dims(d, &Ho, &Wo);
  if (st != MAXDNN_OK) return st;
  if (elem_bytes != 0 && elem_bytes != 4 && elem_bytes != 2) return MAXDNN_INVALID_VALUE;
  const bool tensor = elem_bytes != 0;
  const int eb = tensor ? elem_bytes : 4;
  const int max_rows = tensor ? 256 : 128;
  const int chunk = 128 / eb;                                         // images per reduction step
  st = common_limits(d, eb);
  if (st != MAXDNN_OK) return st;
  if (!g || sm_count <= 0) return MAXDNN_INVALID_VALUE;
  if ((d.Nb * eb) % 16 != 0 || d.No % 4 != 0) return MAXDNN_NOT_SUPPORTED;   // 16-byte row rule
  memset(g, 0, sizeof(*g));
  g->Nb = d.Nb; g->Wi = d.Wi; g->Hi = d.Hi; g->Nc = d.Nc; g->No = d.No;
  g->Skw = d.Skw; g->Skh = d.Skh; g->stride_w = d.stride_w; g->stride_h = d.stride_h;
  g->pad_w = d.pad_w; g->pad_h = d.pad_h; g->alpha = d.alpha; g->Ho = Ho; g->Wo = Wo;
  g->bw = d.Skw;
  if (max_rows / g->bw < 1) return MAXDNN_NOT_SUPPORTED;
  // Two-SM tiles (tensor-core kernel): 256 filters per pair of CTAs, each CTA staging its
  // 128 filters and half of the tile's channels — per SM and per MMA 8 KB instead of 12 KB
  // are staged, and the kernel is bound by that fill rate.  Taken when the second CTA of
  // every tile has filters and the channels split evenly.
  const bool peer_has_filters = (d.No % 256 == 0) || (d.No % 256 > 128);
  g->pair = (tensor && force_pair >= 0 && (peer_has_filters || force_pair > 0) && d.Nc >= 2 &&
             max_rows / (g->bw * 1) >= 2 && sm_count >= 2) ? 1 : 0;
  // Tile = bc channels x bh filter rows x all Skw filter columns, at most max_rows
  // gradient rows.  Blocks of channels and of filter rows are filled evenly (256
  // channels, 3 x 3: ten blocks of 26 channels, not nine of 28 and one of 4), and the
  // shape that needs the fewest staged rows over all tiles wins — a tile stages its
  // gradient rows (rounded up to the MMA's N granule) plus, on the tensor cores, 128 filter
  // rows per step whatever its height; fewer, larger tiles win near-ties.  11 x 11 x 3:
  // two tiles of 3 channels x 6 filter rows (198 rows) instead of 2 channels x 11 rows
  // (242) and 1 x 11 (half empty).
  {
    const int bh_max = d.Skh < max_rows / g->bw ? d.Skh : max_rows / g->bw;
    double best = 1e300;
    int best_bh = 0, best_bc = 0;
    for (int bh = bh_max; bh >= 1; --bh) {
      int bc = max_rows / (g->bw * bh);
      if (bc > 256) bc = 256;                                   // a copy box has at most 256 per axis
      if (bc > d.Nc) bc = d.Nc;
      if (g->pair) bc &= ~1;
      if (bc < 1) continue;
      const int cb = ceil_div(d.Nc, bc);
      int bce = ceil_div(d.Nc, cb);
      if (g->pair && (bce & 1)) ++bce;
      if (bce > bc) bce = bc;
      const int kb = ceil_div(d.Skh, bh);
      const int bhe = ceil_div(d.Skh, kb);
      const int rows = bce * bhe * g->bw;
      const int staged = !tensor ? max_rows
                                 : 128 + (g->pair ? 2 * align_up(rows / 2, 8) : align_up(rows, 16));
      const double cost = (double)cb * kb * staged;
      if (cost < 0.95 * best) { best = cost; best_bh = bhe; best_bc = bce; }
    }
    if (best_bh == 0) {
      if (!g->pair) return MAXDNN_NOT_SUPPORTED;
      g->pair = 0;                                              // one channel per tile: no halves
      best_bh = bh_max;
      best_bc = 1;
    }
    g->bh = best_bh;
    g->bc = best_bc;
  }
  if (g->pair) g->bc_h = g->bc / 2;
  g->rows = g->bc * g->bh * g->bw;
  g->rows_h = g->pair ? g->rows / 2 : g->rows;
  g->n_mma = g->pair ? 2 * align_up(g->rows_h, 8) : align_up(g->rows, 16);
  g->box_o = d.No < 128 ? d.No : 128;
  g->c_blocks = ceil_div(d.Nc, g->bc);
  g->kh_blocks = ceil_div(d.Skh, g->bh);
  g->o_blocks = ceil_div(d.No, g->pair ? 256 : 128);
  g->n_chunks = ceil_div(d.Nb, chunk);
  const int64_t r_steps = (int64_t)Ho * Wo * g->n_chunks;
  const int64_t tiles = (int64_t)g->c_blocks * g->kh_blocks * g->o_blocks;
  if (r_steps > 0x3fffffff || tiles > 0x3fffffff) return MAXDNN_NOT_SUPPORTED;
  g->r_steps = (int32_t)r_steps;
  // Split the reduction over CTAs: with s splits the kernel runs ceil(tiles * s / units)
  // waves of items, each of ceil(r_steps / s) reduction steps plus a fixed cost (filling
  // the ring, draining the accumulator, writing the partial sums) of about a dozen steps
  // (fitted to timings of forced split counts on the 5x5, 3x3 and 13x13 layers: the best
  // counts are the largest that still fill a whole number of waves, and one full wave of
  // long items beats several waves of short ones).  At least 32 steps per split.
  const int units = g->pair ? sm_count / 2 : sm_count;
  int splits = 1;
  if (force_splits > 0) {
    splits = force_splits;
  } else {
    const int64_t most = r_steps / 32 > 0 ? r_steps / 32 : 1;
    const double fixed = tensor ? 12.0 : 4.0;   // the fp32 kernel's steps are longer
    double best = 1e300;
    for (int64_t sp = 1; sp <= most && sp <= 4096; ++sp) {
      const int64_t waves = (tiles * sp + units - 1) / units;
      const double cost = (double)waves * ((double)((r_steps + sp - 1) / sp) + fixed);
      if (cost < best * 0.995) { best = cost; splits = (int)sp; }   // more splits must pay
    }
  }
  if (splits > r_steps) splits = (int)r_steps;
  if (splits < 1) splits = 1;
  g->steps_per_split = ceil_div(g->r_steps, splits);
  g->splits = ceil_div(g->r_steps, g->steps_per_split);
  const int64_t items = tiles * g->splits;
  if (items > 0x7fffffff) return MAXDNN_NOT_SUPPORTED;
  g->n_items = (int32_t)items;
  g->stages = tensor ? (g->pair ? 6 : 4) : 6;
  g->smem_bytes = g->stages * (128 + (g->pair ? 128 : max_rows)) * 128 + 1024 + 1024 +
                  (tensor ? 2048 : 0);   // ring, alignment slack, barriers, row table
  if (g->pair) {
    const int pairs = sm_count / 2;
    g->grid = 2 * (g->n_items < pairs ? g->n_items : pairs);
  } else {
    g->grid = g->n_items < sm_count ? g->n_items : sm_count;
  }
  return MAXDNN_OK;
}

}  // namespace maxdnn
