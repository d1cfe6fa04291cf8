/*
 * maxdnn.h — C ABI of the B200-native FPROP direct convolution library.
 *
 * The operation (paper Section 2, "Convolution"): a minibatch of Nb maps of
 * Wi x Hi x Nc is convolved with a bank of No filters of Sk x Sk x Nc; products
 * are taken channel by channel and summed over channels; the filter moves with
 * a stride; the origin is offset by a padding parameter and the map is wrapped
 * in an apron of zeros; the result is scaled by alpha:
 *
 *   out[o,y,x,n] = alpha * sum_{c,kh,kw} filt[c,kh,kw,o]
 *                                        * in0[c, y*stride-pad+kh, x*stride-pad+kw, n]
 *
 * in0 is `in` inside the map and zero outside.  The filter is not flipped
 * (Section 3 multiplies the unrolled patch by the filter matrix as stored).
 * Ho = floor((Hi + 2*pad - Sk)/stride) + 1, Wo likewise.
 *
 * Layout (Section 3: batch / filter index innermost), all row-major:
 *   in   [Nc][Hi][Wi][Nb]
 *   filt [Nc][Sk][Sk][No]      = the (Sk^2 Nc) x No filter matrix of Section 3
 *   out  [No][Ho][Wo][Nb]
 *
 * Every fprop entry point computes this as the implicit GEMM of Section 3
 * (per output coordinate: unrolled patch Nb x Sk^2 Nc times filter matrix
 * Sk^2 Nc x No), with the patch gathered on the fly.
 *
 * Conventions for all entry points
 *   - Pointers named d_* (and in/filt/out of the device entry points) are
 *     DEVICE pointers of the current CUDA device, owned by the caller, at least
 *     16-byte aligned, non-overlapping.  h_* are HOST pointers.
 *   - `out` is overwritten in full (there is no accumulate mode; the paper has
 *     alpha only).
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls enqueue work and return; they never synchronise the stream.
 *   - Errors are return codes; nothing throws or aborts.  A call that returns
 *     an error other than MAXDNN_CUDA_ERROR has launched nothing.
 *   - The library keeps one small per-device status block (device memory,
 *     allocated on the first fprop call on that device — make that first call
 *     outside any stream capture).  Kernels give every internal wait a time
 *     limit; a wait that runs out records a code there instead of hanging and
 *     the kernel ends normally with an invalid result.  The code is STICKY: it
 *     stays until maxdnn_last_device_status() reads (and clears) it, whatever
 *     is launched in between, so one query after a batch of calls tells whether
 *     any of them gave up.  It does not disturb later launches: every launch
 *     carries its own number, and only a give-up of the same launch makes its
 *     other waits leave early.
 *   - There is no CPU fallback: without an sm_100 device the fprop calls fail
 *     with MAXDNN_NOT_SUPPORTED / MAXDNN_CUDA_ERROR.
 */
#ifndef MAXDNN_H_
#define MAXDNN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Section 2's symbols.  Sk is the (square) filter size; one stride and one
 * padding for both axes. */
typedef struct maxdnn_conv_desc {
  int32_t Nb, Wi, Hi, Nc, No, Sk, stride, pad;
  float alpha;
} maxdnn_conv_desc;

typedef enum maxdnn_status {
  MAXDNN_OK = 0,
  MAXDNN_INVALID_VALUE = 1,  /* null pointer, non-positive size, empty output, non-finite alpha */
  MAXDNN_NOT_SUPPORTED = 2,  /* valid problem this build cannot run (see each entry point) */
  MAXDNN_CUDA_ERROR = 3,     /* a CUDA runtime / driver call failed */
  MAXDNN_DEVICE_TIMEOUT = 4  /* a kernel's bounded wait ran out (reported by last_device_status) */
} maxdnn_status;

/* Arithmetic of the inner product (Section 3.2's inner loop). */
typedef enum maxdnn_kernel_kind {
  MAXDNN_KERNEL_FP32 = 0, /* exact fp32 fused multiply-add on the CUDA cores */
  MAXDNN_KERNEL_TF32 = 1, /* tensor cores, fp32 storage read as TF32, fp32 accumulate */
  MAXDNN_KERNEL_BF16 = 2  /* tensor cores, bf16 storage, fp32 accumulate */
} maxdnn_kernel_kind;

const char* maxdnn_status_string(maxdnn_status s);

/* Output map size (Section 2: the stride "yields the desired output map
 * size"; floor division, consistent with every row of Table 1).
 * INVALID_VALUE if desc is null, a size is <= 0, pad < 0, alpha is not finite
 * or the padded map is smaller than the filter.  Ho / Wo may be null. */
maxdnn_status maxdnn_conv_out_dims(const maxdnn_conv_desc* desc, int32_t* Ho, int32_t* Wo);

/* Section 2's complexity C = 2 Nb Wo Ho (Nc Sk^2 + 1) No, one multiply-
 * accumulate = 2 FLOPs.  0 for an invalid descriptor. */
uint64_t maxdnn_conv_flops(const maxdnn_conv_desc* desc);

/* Number of elements of in / filt / out for a descriptor (0 if invalid). */
uint64_t maxdnn_conv_in_elems(const maxdnn_conv_desc* desc);
uint64_t maxdnn_conv_filt_elems(const maxdnn_conv_desc* desc);
uint64_t maxdnn_conv_out_elems(const maxdnn_conv_desc* desc);

/*
 * The address-generation stage (Section 3.2's precomputed offset table: the
 * walk over a patch is a single pass over table entries, with no index
 * arithmetic left in the loop).  Here one table entry ("K step") names a box
 * of patch rows that one TMA transfer stages into shared memory, and the
 * matching box of filter-matrix rows.
 */
typedef struct maxdnn_kstep {
  int16_t c0;   /* first channel of the box */
  int8_t kh;    /* filter row of the box */
  int8_t kw0;   /* first filter column of the box */
} maxdnn_kstep;

typedef struct maxdnn_plan_info {
  int32_t Ho, Wo;
  int32_t tile_m;      /* filters per tile (rows of the GEMM block) */
  int32_t tile_px;     /* adjacent output pixels (along x) per tile */
  int32_t tile_n;      /* images per tile */
  int32_t kc;          /* channels per K step (few-channel tensor plans: K rows of one filter row) */
  int32_t kwc;         /* filter columns per K step (1 or Sk; few-channel plans with a shared strip: filter rows per step) */
  int32_t n_ksteps;    /* length of the K-step table */
  int32_t stages;      /* depth of the shared-memory ring */
  int32_t n_tiles;     /* tiles in the whole problem */
  int32_t grid;        /* persistent CTAs launched */
  int32_t smem_bytes;  /* dynamic shared memory per CTA */
  int32_t tile_cols;   /* columns the kernel instance is built for (fp32: 128 or 256) */
  int32_t pair;        /* tensor kernels: 1 = two-SM tiles of 256 filters */
  int32_t khc;         /* filter rows per K step (fp32 few-channel plans: a box spans khc rows,
                          clipped at the filter's last row) */
  int32_t split_tiles; /* fp32 kernel: tiles of the last, partly filled wave whose K steps
                          are dealt out over all CTAs (0 = every tile on one CTA) */
} maxdnn_plan_info;

/* One unit of a CTA's work in the fp32 kernel: K steps [s0, s1) of `tile`.  kind 0: the
 * whole tile; 1: a contribution of partial sums to a tile of the split tail; 2: the piece
 * that holds the tile's last K step, adds the other CTAs' partial sums in CTA order and
 * stores the tile. */
typedef struct maxdnn_work_item {
  int32_t tile, s0, s1, kind;
} maxdnn_work_item;

/* Host-only: fills *info and, if steps != NULL, up to max_steps table entries
 * (HOST memory, caller-owned).  Needs no GPU when sm_count > 0 is given
 * (sm_count <= 0 asks the current device).  NOT_SUPPORTED as for the matching
 * fprop call. */
maxdnn_status maxdnn_conv_plan_query(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                     int32_t sm_count, maxdnn_plan_info* info,
                                     maxdnn_kstep* steps, int32_t max_steps);

/* Host-only: the work items of CTA `cta` in the fp32 kernel's plan for `desc` on
 * `sm_count` SMs, in the order the CTA walks them (the paper's kernel gives every block
 * one output coordinate, Section 3.2; here persistent CTAs walk lists of tiles, and the
 * last, partly filled wave of tiles may be split along K — maxdnn_conv_fprop does that
 * whenever the stream's workspace is available; maxdnn_conv_plan_query reports the same
 * plan).  Writes up to max_items items (HOST memory) and their number to *n_items.
 * INVALID_VALUE for a cta outside the plan's grid. */
maxdnn_status maxdnn_conv_plan_items(const maxdnn_conv_desc* desc, int32_t sm_count, int32_t cta,
                                     maxdnn_work_item* items, int32_t max_items,
                                     int32_t* n_items);

/*
 * FPROP with exact fp32 arithmetic (Sections 3.1-3.2: register-blocked
 * multiply-accumulate inner loop over the staged patch, alpha scaling and
 * coalesced store).  in / filt / out: device fp32 buffers in the layout above.
 * NOT_SUPPORTED: Nb or No not a multiple of 4 (16-byte row rule of the bulk
 * tensor copies), Sk > 127, Nc > 32767, a map dimension that does not fit the
 * tensor-copy descriptor (>= 2^31 bytes in one row pitch), or a device that is
 * not sm_100.
 * Memory the library owns: where the plan splits its last wave of tiles along K (see
 * maxdnn_conv_plan_items) the partial sums go through a workspace of 128 KB per SM that
 * the library allocates once per (device, stream) — on the first such call on that
 * stream, never during stream capture (a capture on a stream that has no workspace yet
 * runs whole tiles only; up to eight streams per device get one, later ones run whole
 * tiles only).  The workspace belongs to the stream: launches on one stream are ordered
 * and share it safely; a graph captured on stream S uses S's workspace, so its replays
 * must not overlap each other or other fp32 FPROP work on S.  Results of the two plans
 * differ by rounding order only; each is bitwise reproducible from run to run.
 */
maxdnn_status maxdnn_conv_fprop(const maxdnn_conv_desc* desc, const float* in, const float* filt,
                                float* out, void* cuda_stream);

/*
 * FPROP on the tensor cores, fp32 accumulate.  _tf32 reads the same fp32
 * buffers as maxdnn_conv_fprop (the tensor core ignores the low 13 mantissa
 * bits of each operand).  _bf16 reads bfloat16 `in` and `filt` (same layout,
 * 2-byte elements, supplied by the caller) and writes fp32 `out`.
 * NOT_SUPPORTED: as above, and No not a multiple of 32, or Nb not a multiple
 * of 32 (tf32) / 64 (bf16).
 */
maxdnn_status maxdnn_conv_fprop_tf32(const maxdnn_conv_desc* desc, const float* in,
                                     const float* filt, float* out, void* cuda_stream);
maxdnn_status maxdnn_conv_fprop_bf16(const maxdnn_conv_desc* desc, const void* in,
                                     const void* filt, float* out, void* cuda_stream);

/*
 * The same operation from HOST buffers, for callers that keep their data on
 * the host: enqueues on `cuda_stream` the host->device copies of h_in and
 * h_filt into the caller's device staging buffers d_in / d_filt, the chosen
 * kernel, and the device->host copy of d_out into h_out.  Element types as for
 * the matching device entry point.  Pinned host memory makes the copies
 * asynchronous; the caller synchronises the stream before reading h_out.
 * Allocates nothing.
 */
maxdnn_status maxdnn_conv_fprop_host(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                     const void* h_in, const void* h_filt, float* h_out,
                                     void* d_in, void* d_filt, float* d_out, void* cuda_stream);

/*
 * maxdnn_conv_fprop for callers that must not allocate.  (The paper has no
 * counterpart; this is a deployment variant of the entry point above.)
 *
 * Who needs it: code that runs where a cudaMalloc is off limits — a serving or
 * control loop with a latency bound (cudaMalloc may synchronise the whole device
 * and takes the driver's allocation lock), a process that handed all device
 * memory to its own pool at start-up so that a late driver allocation can fail,
 * or a plug-in whose host application forbids allocation calls after
 * initialisation.  maxdnn_conv_fprop allocates its per-device status block with
 * cudaMalloc on first use; this entry point never calls cudaMalloc, cudaFree or
 * any allocating library routine.  The status block its kernel reports into is a
 * 256-byte device array compiled into the library (every GPU that loads the
 * library holds those 256 bytes until the process exits).
 *
 * Same arguments, layouts, result and NOT_SUPPORTED cases as maxdnn_conv_fprop
 * (the same kernel and tile choice, tile options included; bitwise the same
 * result whenever maxdnn_conv_fprop's plan runs whole tiles only — where that
 * plan splits its last wave along K, which needs a workspace, this entry point
 * runs the last wave as whole tiles and the two results differ by rounding
 * order).  In addition:
 *   - A problem whose kernel would need more than the 256 bytes of built-in
 *     scratch is refused with MAXDNN_NOT_SUPPORTED and nothing is launched.
 *     (The fp32 kernel needs 8 bytes for every descriptor it supports today;
 *     plans that need a workspace in global memory are never chosen here.)
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and sets kernel
 *     attributes; make that first call before any stream capture begins.
 *   - All calls on a device share the one block, which keeps what earlier
 *     calls left in it.  Nothing in it has to start at zero (a launch compares
 *     the block with its own launch number), so no clearing is enqueued; but
 *     two calls whose work overlaps on the GPU — different streams, no ordering
 *     between them — race on it: if both give up a wait, only one code
 *     survives, and one of them may take its full time limit to end.  Order
 *     them, or use maxdnn_conv_fprop for one of them.
 *   - A bounded wait that runs out ends the kernel instead of hanging it and
 *     leaves its code in the built-in block:
 *     maxdnn_last_device_status_noalloc() reads and clears it (a 4-byte copy to
 *     the host and, after a failure, a 4-byte memset: no allocation either).
 *     maxdnn_last_device_status() reports on maxdnn_conv_fprop's block only.
 */
maxdnn_status maxdnn_conv_fprop_noalloc(const maxdnn_conv_desc* desc, const float* in,
                                        const float* filt, float* out, void* cuda_stream);
maxdnn_status maxdnn_last_device_status_noalloc(void* cuda_stream);

/*
 * FPROP with fp32-level accuracy on the tensor cores (three-product TF32): every fp32
 * operand a is split into a_hi (a rounded to the nearest TF32 number, which a TF32 tensor
 * core reads unchanged) and a_lo = a - a_hi (rounded likewise), and the products
 * a_hi b_hi + a_hi b_lo + a_lo b_hi are accumulated in fp32 (the dropped a_lo b_lo term is
 * below 2^-22 of the product).  Because the operation sums over channels, the three
 * products are ONE TF32 FPROP over 3 Nc channels: a small kernel writes the split maps
 * [hi; hi; lo] and filters [hi; lo; hi] into the caller's workspace (size from
 * maxdnn_conv_fprop_tf32x3_workspace) and a TF32 kernel runs on them.  That kernel sums K
 * in chunks: the tensor core truncates its fp32 accumulator at every MMA, a one-sided error
 * that over a long sum of same-signed terms reaches 1e-8 K of the result, so a fresh
 * accumulator is started about every 768 rows of K and the finished chunks are added in
 * registers with round-to-nearest fp32 adds.  Same arguments, layouts and limits as
 * maxdnn_conv_fprop_tf32 (with 3 Nc <= 32767); in / filt / out are the fp32 tensors.  The
 * paper has no counterpart (its kernel is an fp32 CUDA-core kernel).  Accuracy: the exact
 * kernel's class — measured 1e-6 .. 3e-6 of the largest output against the fp64 oracle for
 * K = 144 .. 9216 (exact fp32 kernel: 5e-7 .. 4e-6; plain TF32: 7e-4) — at about four
 * times the exact kernel's speed on 3x3 / 5x5 layers.  (Option X3_CHUNK_ROWS = 0 selects
 * the one-accumulator path: 2-3 % faster, error about 1e-8 K.)
 */
maxdnn_status maxdnn_conv_fprop_tf32x3_workspace(const maxdnn_conv_desc* desc, size_t* bytes);
maxdnn_status maxdnn_conv_fprop_tf32x3(const maxdnn_conv_desc* desc, const float* in,
                                       const float* filt, float* out, void* workspace,
                                       size_t workspace_bytes, void* cuda_stream);
/* The gradient with respect to the maps (the adjoint defined under "Backward propagation"
 * below) in the same three-product mode: the FPROP of dout with the flipped, transposed
 * filter bank (stride 1) or, class by class, with its sub-filter banks (stride > 1: the
 * residue classes of maxdnn_conv_bprop_data, side by side on the library's streams), run
 * through the kernels of maxdnn_conv_fprop_tf32x3.  dout / filt / din are the fp32 tensors;
 * workspace and errors as there (NOT_SUPPORTED: stride 1 with pad > Sk-1, or what the TF32
 * kernel refuses for the transposed problem, whose filter count is Nc). */
maxdnn_status maxdnn_conv_bprop_data_tf32x3_workspace(const maxdnn_conv_desc* desc, size_t* bytes);
maxdnn_status maxdnn_conv_bprop_data_tf32x3(const maxdnn_conv_desc* desc, const float* dout,
                                            const float* filt, float* din, void* workspace,
                                            size_t workspace_bytes, void* cuda_stream);
/* The gradient with respect to the filters in the three-product mode.  Its reduction runs
 * over pixels and images, so the three products are ONE reduction over three times the
 * images: a small kernel writes both tensors as [hi | lo] side by side along the image axis
 * into the workspace, and a TF32 filter-gradient kernel that accumulates in chunks (a fresh
 * accumulator every 768 terms, the chunks added in round-to-nearest fp32) runs on the
 * problem with 3 Nb images, reading for each third the parts of that product; partial sums of the split reduction are added in a
 * fixed order as in maxdnn_conv_bprop_filter.  in / dout / dfilt are the fp32 tensors.
 * NOT_SUPPORTED: Nb not a multiple of 32, No not a multiple of 4, the limits of
 * maxdnn_conv_fprop.  Accuracy: the exact kernel's class (tested to 1e-5 of the largest
 * element). */
maxdnn_status maxdnn_conv_bprop_filter_tf32x3_workspace(const maxdnn_conv_desc* desc, size_t* bytes);
maxdnn_status maxdnn_conv_bprop_filter_tf32x3(const maxdnn_conv_desc* desc, const float* in,
                                              const float* dout, float* dfilt, void* workspace,
                                              size_t workspace_bytes, void* cuda_stream);

/*
 * FPROP for shapes the entry points above refuse because of the 16-byte row rule
 * (Nb or No not a multiple of 4 for fp32; of 32 / 64 and 32 for tf32 / bf16).
 * Two routes.  In-kernel (fp32 only): the kernel stages the ragged rows itself — four copy
 * warps move the patch rows (and the filter rows, if No is ragged) into shared memory with
 * 4- or 8-byte loads and stores, zeros for the apron and for the tails of Nb and No, in
 * place of the bulk tensor copies, and the epilogue stores element by element — so no
 * padded copy of any tensor is made and no workspace is needed.  Padded (every kind): the
 * maps and filters are copied into zero-padded staging tensors in the
 * caller's workspace (Nb, No rounded up), the matching kernel runs on the padded
 * problem, and the result is copied back without the padding.  Same arguments and
 * result as the matching entry point; `workspace` as for the backward entry points
 * below (size from maxdnn_conv_fprop_ragged_workspace; 0 when none is needed: an aligned
 * shape, which runs directly on the caller's tensors, or the in-kernel route).  The padded
 * route is the default for every kind: measured, the copy warps of the in-kernel route cost
 * the arithmetic warps more issue slots (12 % of a long-K layer's time, far more on a
 * 3-channel layer) than the padded route's extra passes over maps and result cost memory
 * time.  Option RAGGED_PADDED = -1 selects the in-kernel route for fp32.
 * The paper has no counterpart (Section 3.3 only notes that its kernel wants
 * multiples of 64 filters and 8 images for efficiency).
 */
maxdnn_status maxdnn_conv_fprop_ragged_workspace(const maxdnn_conv_desc* desc,
                                                 maxdnn_kernel_kind kind, size_t* bytes);
maxdnn_status maxdnn_conv_fprop_ragged(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                       const void* in, const void* filt, float* out,
                                       void* workspace, size_t workspace_bytes,
                                       void* cuda_stream);

/*
 * FPROP with per-axis filter size, stride and padding (Section 2 states one square filter
 * size, one stride and one padding; this lifts that restriction for the same kernels):
 *
 *   out[o,y,x,n] = alpha * sum_{c,kh,kw} filt[c,kh,kw,o]
 *                    * in0[c, y*stride_h - pad_h + kh, x*stride_w - pad_w + kw, n]
 *
 * with kh < Skh, kw < Skw, filt laid out [Nc][Skh][Skw][No], Ho = floor((Hi + 2 pad_h -
 * Skh)/stride_h) + 1 and Wo likewise with the w quantities.  `kind` selects the kernel as
 * in the entry points above (bf16: in and filt are bfloat16); same conventions, limits and
 * NOT_SUPPORTED cases, with Sk read as max(Skw, Skh).
 */
typedef struct maxdnn_conv_desc2 {
  int32_t Nb, Wi, Hi, Nc, No, Skw, Skh, stride_w, stride_h, pad_w, pad_h;
  float alpha;
} maxdnn_conv_desc2;

maxdnn_status maxdnn_conv2_out_dims(const maxdnn_conv_desc2* desc, int32_t* Ho, int32_t* Wo);
maxdnn_status maxdnn_conv2_fprop(const maxdnn_conv_desc2* desc, maxdnn_kernel_kind kind,
                                 const void* in, const void* filt, float* out, void* cuda_stream);
/* The two gradients of the per-axis operation: as maxdnn_conv_bprop_data / _filter below,
 * with every Sk, stride and pad read per axis (dfilt is [Nc][Skh][Skw][No]). */
maxdnn_status maxdnn_conv2_bprop_data_workspace(const maxdnn_conv_desc2* desc,
                                                maxdnn_kernel_kind kind, size_t* bytes);
maxdnn_status maxdnn_conv2_bprop_data(const maxdnn_conv_desc2* desc, maxdnn_kernel_kind kind,
                                      const void* dout, const void* filt, float* din,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream);
maxdnn_status maxdnn_conv2_bprop_filter_workspace(const maxdnn_conv_desc2* desc,
                                                  maxdnn_kernel_kind kind, size_t* bytes);
maxdnn_status maxdnn_conv2_bprop_filter(const maxdnn_conv_desc2* desc, maxdnn_kernel_kind kind,
                                        const void* in, const void* dout, float* dfilt,
                                        void* workspace, size_t workspace_bytes,
                                        void* cuda_stream);

/*
 * Backward propagation.  The paper builds FPROP only and names BPROP (Abstract,
 * Section 3.5 "Conclusion") as the operation its techniques should carry over to, without
 * defining it; these entry points compute the two exact adjoints of the
 * operation above, alpha included, with dout laid out like out, din like in and
 * dfilt like filt:
 *
 *   din  [c,h,w,n]   = alpha * sum over (o,y,x,kh,kw) with y*stride-pad+kh = h and
 *                      x*stride-pad+kw = w of filt[c,kh,kw,o] * dout[o,y,x,n]
 *   dfilt[c,kh,kw,o] = alpha * sum_{y,x,n} in0[c, y*stride-pad+kh, x*stride-pad+kw, n]
 *                                          * dout[o,y,x,n]
 *
 * Both need caller-owned device scratch (`workspace`, 16-byte aligned, at
 * least the size the matching *_workspace call reports; may be NULL when that
 * size is 0); the library allocates nothing.  Results are overwritten in full.
 *
 * maxdnn_conv_bprop_data: the gradient with respect to the maps on the kernel `kind`
 * names (fp32; tf32; bf16: dout and filt are bfloat16, din fp32).  Stride 1: an FPROP
 * of dout with the filter bank transposed (channels <-> filters) and flipped in both
 * axes (written into the workspace by a small kernel on the same stream) and padding
 * Sk-1-pad.  Stride s > 1: the map positions split into s x s classes by
 * (h+pad) mod s, (w+pad) mod s; each class meets only the taps kh = rho_h + s j,
 * kw = rho_w + s i and is, on its own grid, a stride-1 FPROP of dout with that
 * sub-filter (flipped, transposed), written onto the class's grid inside din;
 * positions no tap reaches are zero.  The classes are independent launches: they
 * are queued on the given stream and on three streams the library owns, which
 * start after the work already queued on the given stream and which the given
 * stream waits for before the call returns to it (a fork and join by events, valid
 * under stream capture); each class has its own part of the workspace.
 * NOT_SUPPORTED: stride 1 with
 * pad > Sk-1, Nb not a multiple of 4 (stride > 1), or what the matching fprop
 * entry point refuses for the transposed problem (its filter count is Nc).
 *
 * maxdnn_conv_bprop_filter: the gradient with respect to the filters as the GEMM
 * dfilt[k][o] = sum_r patch[k][r] * dout[o][r] with the reduction r over output
 * pixels and images, split over CTAs whose partial sums (in the workspace) are
 * added in a fixed order, so the result does not depend on scheduling.  `kind`
 * fp32: exact fp32 on the CUDA cores; tf32: the same fp32 buffers on the tensor
 * cores; bf16: `in` and `dout` are bfloat16.  dfilt is fp32 for every kind.
 * NOT_SUPPORTED: a row of images not a multiple of 16 bytes (Nb % 4 for fp32 /
 * tf32, % 8 for bf16), No not a multiple of 4, the limits of maxdnn_conv_fprop.
 */
maxdnn_status maxdnn_conv_bprop_data_workspace(const maxdnn_conv_desc* desc,
                                               maxdnn_kernel_kind kind, size_t* bytes);
maxdnn_status maxdnn_conv_bprop_data(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                     const void* dout, const void* filt, float* din,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream);
maxdnn_status maxdnn_conv_bprop_filter_workspace(const maxdnn_conv_desc* desc,
                                                 maxdnn_kernel_kind kind, size_t* bytes);
maxdnn_status maxdnn_conv_bprop_filter(const maxdnn_conv_desc* desc, maxdnn_kernel_kind kind,
                                       const void* in, const void* dout, float* dfilt,
                                       void* workspace, size_t workspace_bytes,
                                       void* cuda_stream);

/* Synchronises `cuda_stream`, then reads and clears the current device's
 * status word.  MAXDNN_OK, MAXDNN_DEVICE_TIMEOUT (a bounded wait inside some
 * kernel launched since the last query ran out; that kernel's output is not
 * valid) or MAXDNN_CUDA_ERROR. */
maxdnn_status maxdnn_last_device_status(void* cuda_stream);

/*
 * Section 3.3 measures efficiency in processor clocks.  With option KERNEL_CLOCK set to 1,
 * maxdnn_conv_fprop has every CTA of its kernel measure its own elapsed SM cycles
 * (clock64) and nanoseconds (%globaltimer) from its first instruction to its last store,
 * and keeps the maxima over the CTAs of the LATEST call in the status block (a memset of
 * those words is enqueued ahead of the kernel; a plan that runs its split tail as a second
 * kernel reports the sum of the two kernels' maxima).  This call synchronises `cuda_stream`
 * and returns them: sm_cycles / nanoseconds is the SM clock the kernel ran at, and
 * C / (2 * 128 * SMs * sm_cycles) the paper's clock-independent efficiency.  Both are 0 if
 * the option was off.  32-bit counters: kernels of up to about two seconds.
 */
maxdnn_status maxdnn_last_kernel_clock(uint32_t* sm_cycles, uint32_t* nanoseconds,
                                       void* cuda_stream);

/*
 * Tuning and test options (ablations and tests; none is needed in normal use; the
 * paper has no counterpart).  An option is a named integer, "unset" by default.  `name`
 * is one of FFMA_TILE_M, FFMA_COLS (pin the fp32 kernel's tile: filters 32/64/96/128/256,
 * columns 128/256), FFMA_KH (filter rows per K step of few-channel layers), FFMA_KC (upper
 * limit of the channels per K step of many-channel layers, a multiple of 4 in 8..128, below
 * what the tile's ring would hold), FFMA_STREAMK (0: never split tail tiles along K; 2: always, whatever
 * the model says), UMMA_KC, UMMA_PAIR (1 two-SM / -1 one-SM tiles), UMMA_MERGE, UMMA_STAGE_KB, UMMA_COLS, WGRAD_SPLITS, WGRAD_PAIR, SM_COUNT (SM
 * count for host-only workspace queries), X3_CHUNK_ROWS, DEBUG_STATUS, KERNEL_CLOCK (see
 * maxdnn_last_kernel_clock), RAGGED_PADDED (see maxdnn_conv_fprop_ragged), and
 * TEST_MISSING_ARRIVAL (test hook: CTA 0's "full" barriers expect an arrival that
 * never comes, so a bounded wait runs out).  The environment variable MAXDNN_<name>
 * gives an option its initial value; the environment is read once, at the first use of
 * any option in the process, never during a call.  TEST_MISSING_ARRIVAL has no
 * environment variable: only maxdnn_set_option can switch it on.  Setting an option
 * discards cached plans.  INVALID_VALUE for an unknown name.  Thread-safe; a call that is
 * planning concurrently sees either the old or the new value.
 */
maxdnn_status maxdnn_set_option(const char* name, int32_t value);
maxdnn_status maxdnn_unset_option(const char* name);
maxdnn_status maxdnn_get_option(const char* name, int32_t* value, int32_t* is_set);
void maxdnn_reset_options(void);   /* every option back to what the environment gave */

/* How many kernels this library has launched in this process (all devices). */
uint64_t maxdnn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* MAXDNN_H_ */
