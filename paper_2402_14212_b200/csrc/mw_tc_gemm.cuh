// Tensor-core product core for sm_100a: TMA-staged operand tiles, tcgen05.mma with the
// accumulators in tensor memory, fused epilogues.  Internal interface.
//
// Every dense step of the Moonwalk path is one product:
//   Phase I / recompute   z   = x W^T         (A = x K-major,  B = W K-major)
//   Phase II              h'  = g_z W         (A = g_z K-major, B = W MN-major)
//   dense vijp            g_z = h W^-1        (A = h K-major,  B = W^-1 MN-major)       Eq. "h_i"
//   weight vjp            dW  = g_z^T x       (A = g_z MN-major, B = x MN-major)        Eq. "g_i"
//   Newton-Schulz         R = I - W X, X' = X + X R
// and one launch of the persistent kernel runs a GROUP of up to kTcMaxGroup independent products
// (for the forward sweep: the recompute and the vijp of layer l+1 together with the weight vjp of
// layer l), its CTAs walking the union of their output tiles.
//
// An operand is a stack of 1..3 bf16 "term planes" whose sum is the value (term t holds the
// bf16 rounding of what the earlier terms left over).  A product of an a-term and a b-term
// operand accumulates, in fp32, the cross products (i, j) with i + j < max(a, b): 1 product for
// plain bf16, 3 for ~16-bit operands, 6 for fp32-accurate operands.
#pragma once
#include <cuda.h>

#include "mw_common.cuh"

namespace mw {

constexpr int kTcMaxGroup = 4;
constexpr int kTcMaxDeps = 4;
constexpr size_t kTcSplitCounterBytes = 65536;

struct TcOperand {
  const void* base = nullptr;   // bf16 planes, each [rows][cols] row-major
  int rows = 0, cols = 0;       // K-major: rows = M or N, cols = K.  MN-major: rows = K, cols = M or N
  int planes = 1;
  int64_t plane_stride = 0;     // elements between planes
  bool mn_major = false;
  int batch_planes = 0;         // batched product: planes between consecutive batch items (0 = planes)
  int64_t ld = 0;               // elements between consecutive rows (0 = cols): a window of wider rows
};

enum TcEpiMode : int {
  TC_EPI_PLAIN = 0,    // v = alpha*acc (+ addend);  out_f32 and/or planes
  TC_EPI_RESID = 1,    // v = (row == col) - acc, or with scale_dev (c = *scale_dev) v = c (2 (row == col) - c acc);
                       // planes; sum of squares -> sumsq
  TC_EPI_FWD = 2,      // z = acc; sign word written (write_mask) or read; x = phi(z) -> planes (+ out_f32)
  TC_EPI_BWD = 3,      // h = acc -> out_f32 / planes2 (optional), ReLU fragments (optional); g = h * phi'(mask) -> planes
  TC_EPI_VIJP = 4,     // g = alpha*acc (+ addend); activation vijp: h -> planes2 (+ out_f32); g (zero at dead
                       // ReLU units) -> planes
};

struct TcEpilogue {
  int mode = TC_EPI_PLAIN;
  float alpha = 1.f;
  const float* addend = nullptr;       // [M][N] fp32
  float* out_f32 = nullptr;            // [M][N] fp32
  __nv_bfloat16* planes = nullptr;     // primary split output, n_planes x [M][N]
  int n_planes = 0;
  int64_t plane_stride = 0;
  __nv_bfloat16* planes2 = nullptr;    // secondary split output (TC_EPI_VIJP: h)
  int n_planes2 = 0;
  int64_t plane_stride2 = 0;
  uint32_t* mask = nullptr;            // sign words [M][N/32]
  int write_mask = 0;
  int act = MW_ACT_NONE;
  float slope = 1.f;
  // TC_EPI_RESID: a scalar in device memory (one per batch item) that turns the residual of the
  // start X_0 = c W^T into the factor of the first Newton-Schulz step (see TC_EPI_RESID)
  const float* scale_dev = nullptr;
  // TC_EPI_RESID of a square product whose result the caller knows to be symmetric (W W^T; W X for an
  // iterate X = W^T p(W W^T)).  With 1 only the tiles that reach the diagonal or lie above it are
  // computed, and every tile wholly above it is also stored transposed below it (pair form: through
  // the copy engine).  Its sum-of-squares pieces count for both; in the one-CTA form the pieces of
  // the tiles that are left out are never written: the caller zeroes `sumsq` first.
  int symmetric = 0;
  // TC_EPI_RESID: ||v||_F^2 in pieces, one slot per 128-row block, column tile and epilogue warp
  // (tc_sumsq_slots of them; each is written, none accumulated: the reader adds them in order)
  double* sumsq = nullptr;
  // ReLU fragment stream (Section 5.1 applied to ReLU): row r keeps the cotangent at its dead
  // units from vals[frag_off[r]], in increasing column order; frag_rank[r][c/64] = number of
  // dead units of row r before column 64*(c/64).  TC_EPI_BWD writes the stream, TC_EPI_VIJP
  // reads it back.
  const uint32_t* frag_off = nullptr;
  const uint32_t* frag_rank = nullptr;
  float* frag_vals = nullptr;
  // batched product (one tile range per batch item): element strides between consecutive items
  int64_t bs_f32 = 0;                  // addend and out_f32
  int64_t bs_planes = 0, bs_planes2 = 0;
  int64_t bs_mask = 0;                 // words
  int64_t bs_sumsq = 0;                // doubles
  // row scatter (remap_s > 0): row r of the product is pixel (b, y, x) of a remap_ho x remap_wo
  // image and its outputs (and sign words) live at pixel (b, remap_s*y + remap_py,
  // remap_s*x + remap_px) of the remap_s times larger image: one parity class of a strided
  // TransposeConv
  int remap_s = 0, remap_ho = 0, remap_wo = 0, remap_py = 0, remap_px = 0;
  // TC_EPI_BWD with a row scatter: planes2 is addressed by the product's own row all the same
  // (the class of the pixels (s*y, s*x) written densely: all that a strided vijp reads of h)
  // elements between consecutive rows of addend, out_f32 and planes (0 = N): outputs that are a
  // column window of wider rows
  int64_t ld = 0;
  int compact2 = 0;
  // TC_EPI_VIJP (sub2_s > 0): the rows are pixels of sub2_h x sub2_w images and planes2 keeps
  // only the pixels (sub2_s*y, sub2_s*x), densely: [images][sub2_h/s][sub2_w/s][N]
  int sub2_s = 0, sub2_h = 0, sub2_w = 0;
};

// Convolution forms of a product.  The A operand is then a channel-last pixel array
// [images][H][W][C] per term plane (C a multiple of 64: one K block per tap and 64 channels),
// read through a window that starts at `stride` times the product's own pixel plus an offset
// (out-of-image pixels read as zero: the padding of Lemma 1).  The product's pixels form images
// of Ho x Wo; a tile covers part of a row, whole rows of one image, or whole images.
//   TC_CONV_PIXELS  rows of A = pixels (b, y, x) of the Ho x Wo image, K = (window, channel).
//                   Window t reads pixel (stride*y + dy[t], stride*x + dx[t]) and the B block
//                   tb[t].  With ntaps = 0 the list is derived from k, pad, sgn, skip_tap: every
//                   tap (j0, j1) but skip_tap, offset sgn*(j - pad), B block = tap.  sgn = +1:
//                   forward convolution (Lemma 1), sgn = -1: TransposeConv (Eq. "conv-vjp").
//   TC_CONV_WGRAD   weight vjp (Eq. "g_i" for a convolution): rows of the result = (tap, c);
//                   K = pixels of the Ho x Wo image; batch item z covers the K blocks
//                   [z*K/64, (z+1)*K/64) of the pixel range, so that `batch` slices of the pixel sum
//                   land in separate outputs.  A (MN-major) is the activation read at
//                   stride*pixel + tap - pad, B (MN-major) the cotangent [pixels][N].
enum TcConvMode : int { TC_CONV_NONE = 0, TC_CONV_PIXELS = 1, TC_CONV_WGRAD = 2 };
constexpr int kTcMaxTaps = 25;

struct TcConv {
  int mode = TC_CONV_NONE;
  int H = 0, W = 0;         // image of the pixel array A reads
  int C = 64;               // its channels
  int stride = 1;
  int Ho = 0, Wo = 0;       // image of the product's pixels (0: H, W)
  int k = 0, pad = 0;       // kernel k x k (k*k <= kTcMaxTaps)
  int sgn = 1;
  int skip_tap = -1;        // tap left out of the sum (the centre tap of the folded kernel), or -1
  int b_tap_rows = 0;       // B is K-major with rows (block, n): used by TransposeConv
  int one_d = 0;            // TC_CONV_WGRAD: the kernel is 1 x k (taps along x only, no row offset)
  int ntaps = 0;            // explicit window list (TC_CONV_PIXELS)
  signed char dy[kTcMaxTaps] = {}, dx[kTcMaxTaps] = {}, tb[kTcMaxTaps] = {};
};

// One product of a group.
struct TcGemm {
  TcOperand A, B;
  int M = 0, N = 0, K = 0;
  int batch = 1;
  TcEpilogue epi;
  TcConv conv;
  // K split: the K range of every output tile is cut into `split_k` pieces computed by
  // different CTAs; partial tiles meet in `split_scratch` (kTcSplitCounterBytes of arrival
  // counters, zero before the first use and left zero by every launch, then split_k * tiles *
  // 128 * bn floats; see tc_split_scratch_bytes) and the warp that arrives last adds the pieces
  // in fixed order, so the result does not depend on scheduling.  0 / 1 = no split.
  int split_k = 1;
  void* split_scratch = nullptr;
  // 1: keep the widest tile the term count allows even if the product alone then has fewer
  // tiles than SMs (for throughput work that shares its launch with other products)
  int wide_tiles = 0;
};

// Cache of encoded tensor maps (host side), owned by the caller.
struct TcMapCache;
TcMapCache* tc_cache_create();
void tc_cache_destroy(TcMapCache*);

// Requirements per product: N % 64 == 0; K % 64 == 0 unless both operands are MN-major; M % 64 == 0
// for an MN-major A; all bases 16-byte aligned.  batch > 1 runs `batch` independent products of the same shape: item b reads
// planes b*batch_planes + t of each operand and offsets the epilogue pointers by b times the
// bs_* strides.
mw_status tc_gemm_group(TcMapCache* cache, const TcGemm* g, int count, DeviceStatus* st,
                        cudaStream_t s);
// single product
mw_status tc_gemm(TcMapCache* cache, const TcOperand& A, const TcOperand& B, int M, int N, int K,
                  const TcEpilogue& epi, DeviceStatus* st, cudaStream_t s, int batch = 1);

// A program: many products in ONE cooperative launch, each starting when the products it names
// (earlier ones only) are complete -- a whole phase of the method without a launch per layer.
// The product table lives in device memory (`table_dev`, tc_program_table_bytes(n), 64-byte
// aligned) beside one completion counter per product (`done_dev`); both are the caller's.  The
// table is uploaded and the counters are cleared at every launch.
// Units are taken in order of insertion, so insertion order must be a valid execution order.
struct TcProgram;
TcProgram* tc_program_create();
void tc_program_destroy(TcProgram*);
// pair: run every product in the pair form (each must satisfy tc_pair_ok, else tc_program_add fails)
void tc_program_begin(TcProgram*, void* table_dev, unsigned int* done_dev, bool pair = false);
// returns the product's index (negative on error, *status says why); deps: up to kTcMaxDeps
// indices of earlier entries (products or groups), -1 = none.  group: index of a group entry
// (tc_program_add_group) that this product's tiles also report to, or -1: a later product that
// names the group waits for all its members.
int tc_program_add(TcProgram*, TcMapCache* cache, const TcGemm& g, const int* deps, int ndep,
                   mw_status* status, int group = -1);
// an entry without work that stands for "all products added to it"; add it before its members
int tc_program_add_group(TcProgram*);
// units handed to the CTAs by a load-balanced schedule (call after tc_program_begin; default off)
void tc_program_balance(TcProgram*, bool on);
size_t tc_program_table_bytes(int products);
mw_status tc_program_launch(TcProgram*, DeviceStatus* st, cudaStream_t s);
constexpr int kTcMaxProgram = 768;

// tile width the kernel will use for this product, and the scratch a K split of it needs
int tc_tile_n(int a_planes, int b_planes, int M, int N, int batch);
size_t tc_split_scratch_bytes(int a_planes, int b_planes, int M, int N, int batch, int split_k);
// K split that gives every SM a work unit when the product alone has too few tiles (1 = none)
int tc_auto_split(int a_planes, int b_planes, int M, int N, int K, int batch);

// Pair form: two CTAs (a cluster of two SMs) share every 256-row tile and each stages half of the
// B tile.  Grouped launches choose it by themselves when every product of the launch qualifies.
bool tc_pair_ok(int a_planes, int b_planes, int M, int N);
int tc_set_pair_mode(int mode);           // 0: never (for comparisons), 1: where it qualifies; returns the old mode
// bound of the device-side waits of later launches (0 = default, 2 s)
void tc_set_wait_limit_ns(uint64_t ns);
// slots of TcEpilogue::sumsq for one product
size_t tc_sumsq_slots(int a_planes, int b_planes, int M, int N, bool pair = false);
// pair form, two-term operands: one accumulator block for all kept cross products (1, default) or
// a block per order (0); returns the old setting
int tc_set_merge_orders(int mode);
// epilogue outputs through the copy engine (1, default) or per-lane stores only (0)
int tc_set_bulk_epilogue(int mode);
// program launches with (1, default) or without (0) the cooperative-launch attribute
int tc_set_cooperative(int mode);

// Per-launch timing of the product kernel (CUDA events around every launch while enabled).
void tc_profile_begin();
mw_status tc_profile_end(double* total_ms, long long* launches, double* flops, double* mma_flops);

// fp32 [n] -> `planes` bf16 term planes (plane p at out + p*plane_stride)
mw_status split_planes(const float* in, int64_t n, __nv_bfloat16* out, int planes,
                       int64_t plane_stride, cudaStream_t s);
// batched: item b reads in + b*in_stride and writes out + b*out_stride
mw_status split_planes_batched(const float* in, int64_t n, int batch, int64_t in_stride,
                               __nv_bfloat16* out, int planes, int64_t plane_stride,
                               int64_t out_stride, cudaStream_t s);

}  // namespace mw
