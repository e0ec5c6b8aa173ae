// tcgen05 / TMA product kernel for sm_100a (see mw_tc_gemm.cuh for the role of each product).
//
// One launch runs a group of independent products.  Their output tiles (128 rows x bn columns,
// optionally cut along K) form one list of work units, sorted by cost; the grid is persistent
// (at most one CTA per SM) and CTA c takes units c, 2G-1-c, 2G+c, ... ("snake" order, which keeps
// the per-CTA sums close).  192 threads per CTA:
//   warp 0      TMA producer: stages the bf16 term planes of A and B for one 64-deep K block
//               (cp.async.bulk.tensor, 128-byte swizzle, no multicast) in a ring of shared-memory
//               stages that runs on across units;
//   warp 1      allocates tensor memory (two accumulator sets of 256 columns), then one lane
//               issues tcgen05.mma (kind::f16, bf16 in, fp32 accumulate).  Term planes of B sit
//               next to each other in a stage, so ONE instruction of width (planes x bn) forms
//               the products of one A plane with several B planes; the cross products of equal
//               order land in the same column block;
//   warps 2..5  epilogue: tcgen05.ld 32 columns at a time (one row per thread), add the column
//               blocks in registers (round to nearest), apply the fused step (activation + sign
//               word, vjp scaling, activation vijp with the ReLU fragment stream, residual, ...)
//               and store.  While they drain one accumulator set the next unit fills the other.
//
// Accuracy: the tensor core truncates its fp32 accumulator at every instruction, a bias that grows
// with the number of instructions feeding one accumulator.  For fp32-accurate products the
// leading term therefore alternates between two column blocks from one K block to the next, and
// the small cross terms have blocks of their own.
// Every wait is bounded; on expiry the kernel records MW_ERR_TIMEOUT and unwinds (tensor memory
// is always released).
//
// Pair form (kPair): two CTAs of a cluster (two SMs) own one 256-row tile.  Each stages its own
// 128 rows of A and HALF of the B tile; one lane of the even CTA issues tcgen05.mma.cta_group::2,
// which reads both halves of B from the two shared memories and writes each CTA's 128 rows of the
// accumulator into that CTA's tensor memory.  B then crosses the L2-to-SM path once per 256 rows
// instead of once per 128.  Copies of both CTAs complete on the even CTA's barrier (plain
// cp.async.bulk.tensor with .cta_group::2; nothing is multicast), the commits that free a stage or
// publish an accumulator set arrive at both CTAs, and the odd CTA's epilogue warps hand the set
// back with a remote arrive.  Operands of at most two terms; every cross product is its own
// instruction of the tile's width (a stacked instruction would interleave the halves of the planes).
#include <cudaTypedefs.h>

#include <algorithm>
#include <map>
#include <tuple>
#include <vector>

#include "mw_tc_gemm.cuh"

namespace mw {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kThreadsTc = 192;
constexpr int kEpiWarps = 4;     // one per tensor-memory lane quarter
constexpr uint64_t kDefaultWaitLimitNs = 2000000000ull;   // 2 s: far above any legitimate wait
constexpr int kMaxStages = 8;
constexpr int kMaxOps = 6;
constexpr uint32_t kATileBytes = BM * BK * 2;  // one A term plane of one stage
constexpr uint32_t kEpiStageBytes = 4096;       // one 32 x 32 fp32 block (or two bf16 blocks) per epilogue warp
constexpr int kSetCols = 256;                  // tensor-memory columns of one accumulator set
constexpr int kTmemCols = 512;

// one tcgen05.mma per 16-deep K step: A plane at a_off16, `width` columns of B starting at b_off16
struct TcOp {
  uint32_t a_off16, b_off16;   // offsets inside a stage, in 16-byte units
  uint32_t idesc;
  uint16_t dcol;               // first accumulator column (inside the set)
  uint16_t rot;                // added to dcol on odd K blocks (alternating leading block)
  uint32_t first_kbs;          // the first K step of this many leading K blocks overwrites
};

struct alignas(64) TcProblem {
  CUtensorMap tmA, tmB;
  // maps of the outputs for the epilogue's bulk stores: fp32 output, term planes, second planes
  // (out_tma bit 0, 1, 2: the map exists)
  CUtensorMap tmO, tmP, tmP2;
  int out_tma;
  TcEpilogue epi;
  int M, N, K, num_kb, kb_per_split, split;
  int bn, tiles_n, tiles_mn, unit_begin, unit_count;
  int bm;                      // rows of one tile: 128, or 256 in the pair form
  int sym;                     // 1: square symmetric result, tiles (mt, nt >= mt) only (see TcEpilogue::symmetric)
  int pa, pb, a_mn, b_mn, a_batch_planes, b_batch_planes;
  uint32_t b_tile_bytes, tx_bytes;   // per CTA: in the pair form a CTA stages half of the B tile
  // Layout of a stage (operands without a convolution window): every operand arrives with ONE
  // copy per K block.  K-major: [plane][rows][64 k], box {64 k, rows, planes} of the array seen as
  // (k, row, plane).  MN-major: [plane][64-column group][64 k][64], box {64, 64 k, groups, planes}
  // of the array seen as (column inside its group, k, group, plane).
  uint32_t a_desc_base, b_desc_base; // descriptor low word without the address (group distance << 16)
  int nops, nblocks;
  float* split_partials;
  unsigned int* split_counters;
  // convolution forms (TcConv)
  int conv_mode, cHo, cWo, ck, cpad, cstride, ccb, b_tap_rows, cntaps, c1d;
  int cbx, cby, cbi;           // pixels, rows and images of one A box
  signed char tdy[28], tdx[28], ttb[28];
  // program launches: products (by index) that must be complete before this one starts, and
  // the number of warp arrivals that completes each of them (one per epilogue warp and tile)
  int ndep, dep[kTcMaxDeps];
  unsigned int dep_target[kTcMaxDeps];
  int done2;                   // a second counter this product's tiles report to (a group), or -1
  TcOp ops[kMaxOps];
};

constexpr int kMaxProgram = 768;   // products of one program launch

struct alignas(64) TcGroupParams {
  int nprob, total_units, stages;
  int sched_len;              // program launch with a unit schedule: entries per CTA (pair)
  uint32_t stage_bytes, pad1;
  uint64_t wait_limit_ns;     // bound of every device-side wait
  uint32_t epi_stage_off;     // byte offset (from the first stage) of the epilogue's transposition
  uint32_t pad2;              // buffers, kEpiStageBytes per epilogue warp; 0 = none
  DeviceStatus* st;
  const TcProblem* table;     // program launch: the products live in global memory ...
  unsigned int* done;         // ... and count their finished tiles here (zero at launch)
  const int* sched;           // [CTAs or pairs][sched_len] units of each, in list order, -1 ends; or null
  TcProblem prob[kTcMaxGroup];
};

struct Unit {
  int q, m0, n0, z, kb0, kb1, tl, ks;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// arrive at a barrier of another CTA of the cluster (`bar` is a shared::cluster address)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
// shared::cluster address of this CTA's shared-memory address `addr` inside CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// all threads of all CTAs of the cluster
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// kCluster: the phase may have been completed from another CTA of the cluster
template <bool kCluster>
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  if (kCluster) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
  }
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// what every bounded wait of a CTA shares
struct WaitCtx {
  DeviceStatus* st;
  volatile int* abort_flag;
  uint64_t limit_ns;
};
// Bounded wait: try_wait suspends the thread in hardware until the phase completes or its own
// time slice ends.  The bound is wall time (checked every 256 polls); a wait also gives up when
// another role of the CTA has already failed.  On expiry the timeout is recorded.
template <bool kCluster>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& wc, unsigned who) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait<kCluster>(bar, parity)) return true;
    if ((i & 255u) == 255u) {
      if (*wc.abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > wc.limit_ns) break;
    }
  }
  record_error(wc.st, MW_ERR_TIMEOUT, who, blockIdx.x, 0u, 0u);
  *wc.abort_flag = 1;
  return false;
}

// Bounded wait for a product of the same (co-resident) launch: its tiles count themselves in
// global memory.  Same bound and failure path as mbar_wait.
__device__ __forceinline__ bool wait_done(const unsigned int* counter, unsigned int target, const WaitCtx& wc) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    __nanosleep(40);
    if ((i & 63u) == 63u) {
      if (*wc.abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > wc.limit_ns) break;
    }
  }
  record_error(wc.st, MW_ERR_TIMEOUT, 5u, blockIdx.x, target, 0u);
  *wc.abort_flag = 1;
  return false;
}

// Bulk tensor copies into this CTA's shared memory.  kPair: the completion bytes are counted on
// `bar`, a shared::cluster address that may lie in the other CTA of the pair (.cta_group::2); the
// data itself always lands in the executing CTA.  No copy is multicast.
template <bool kPair>
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar,
                                            int c0, int c1, int c2) {
  if (kPair) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
        "%4, %5}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
  } else {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
        "%4, %5}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
  }
}

template <bool kPair>
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
  if (kPair) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
        "%4, %5, %6}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
  } else {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
        "%4, %5, %6}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
  }
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* tm, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, "
      "%4, %5, %6, %7}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

// shared-memory operand descriptor, 128-byte swizzle: the upper word is constant, the lower word
// holds the start address (and, for MN-major tiles, the distance between 64-element groups)
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);

// kPair: one instruction for both CTAs of the pair (256 rows); the descriptors name the same
// offsets in both shared memories, the accumulator address the same columns in both tensor memories
template <bool kPair>
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo,
                                          uint32_t idesc, uint32_t accumulate) {
  if (kPair) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}" ::"r"(tmem_d),
        "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}" ::"r"(tmem_d),
        "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
  }
}
// arrive at `bar` once the products issued so far have retired; kPair: at the barrier at this
// offset in BOTH CTAs of the pair (the arrival is sent to two CTAs; no data is)
template <bool kPair>
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  if (kPair) {
    asm volatile(
        "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}" ::"r"(bar)
        : "memory");
  } else {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
  }
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// How an epilogue warp writes its 32 x 32 blocks.  Direct: every lane stores its own row (16-byte
// stores; a warp instruction then touches 32 different lines, one sector-sized piece each, which the
// load/store unit works off at about one piece per cycle).  Bulk (`sbuf` != 0): the block is laid
// into the warp's shared-memory buffer as 32 rows of 64 bytes (32 bf16 or 16 fp32 values) in the
// 64-byte swizzle of a tensor map (conflict-free 16-byte stores) and one lane hands it to the copy
// engine (cp.async.bulk.tensor, shared -> global), which writes whole lines and clips rows beyond
// the product.  The buffer holds two such blocks used in turn: a block is rewritten once the
// engine has read it, i.e. when at most one later hand-over of this lane is still unread.
struct EpiOut {
  uint32_t sbuf = 0;                 // 4 KB, 1024-byte aligned; 0 = direct stores only
  const CUtensorMap* m_f32 = nullptr;   // fp32 output  (col, row, batch item), blocks of 16 columns
  const CUtensorMap* m_pl = nullptr;    // term planes  (col, row, plane, batch item), blocks of 32 columns
  const CUtensorMap* m_pl2 = nullptr;   // second set of term planes
  int row0 = 0;                      // first row of the warp's block
  int z = 0;                         // batch item
  uint32_t half = 0;                 // which 2 KB half the next block takes
  bool mirror = false;               // symmetric product, off-diagonal tile: blocks are stored transposed too
};

__device__ __forceinline__ void bulk_wait_read_all() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_read_but_one() {
  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_store_3d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(tm)),
               "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_store_4d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(tm)),
               "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// write 32 consecutive values as `planes` bf16 term planes (v is left holding the remainder).
// Direct (map == nullptr, only lanes with `valid` rows store) or through the copy engine (all
// lanes of the warp take part; block (col0, eo.row0) of every plane).
__device__ __forceinline__ void store_planes32(float (&v)[32], __nv_bfloat16* base, int planes,
                                               int64_t plane_stride, int64_t off, bool valid,
                                               const CUtensorMap* map, EpiOut& eo, int col0, bool mirror = false,
                                               int64_t off_t = 0, int64_t ld_t = 0) {
  const int lane = threadIdx.x & 31;
  for (int p = 0; p < planes; ++p) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      __nv_bfloat16 a = __float2bfloat16_rn(v[2 * i]);
      __nv_bfloat16 b = __float2bfloat16_rn(v[2 * i + 1]);
      v[2 * i] -= __bfloat162float(a);
      v[2 * i + 1] -= __bfloat162float(b);
      pk[i] = (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
    }
    if (map == nullptr) {
      if (valid) {
        uint4* dst = reinterpret_cast<uint4*>(base + (int64_t)p * plane_stride + off);
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
        if (mirror) {
          // the same values transposed: value i of this lane's row is element (col0 + i, row); the
          // lanes of a warp write consecutive two-byte elements of one row
          unsigned short* dt = reinterpret_cast<unsigned short*>(base + (int64_t)p * plane_stride + off_t);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            dt[(int64_t)(2 * i) * ld_t] = (unsigned short)(pk[i] & 0xffffu);
            dt[(int64_t)(2 * i + 1) * ld_t] = (unsigned short)(pk[i] >> 16);
          }
        }
      }
      continue;
    }
    // rows of 64 bytes in the 64-byte swizzle: 16-byte piece c of row r sits at c ^ ((r >> 1) & 3)
    if (lane == 0) bulk_wait_read_but_one();
    __syncwarp();
    const uint32_t tile = eo.sbuf + eo.half * 2048u;
    eo.half ^= 1u;
    const uint32_t rowp = tile + (uint32_t)lane * 64u;
    const uint32_t sw = ((uint32_t)lane >> 1) & 3u;
#pragma unroll
    for (uint32_t c = 0; c < 4; ++c)
      st_shared_v4(rowp + ((c ^ sw) << 4), pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) bulk_store_4d(map, tile, col0, eo.row0, p, eo.z);
    if (mirror) {
      // the same block transposed: value i of lane r is element (i, r); two-byte stores of a warp
      // fill one 64-byte row, piece (r >> 3) of row i at (r >> 3) ^ ((i >> 1) & 3)
      if (lane == 0) bulk_wait_read_but_one();
      __syncwarp();
      const uint32_t tt = eo.sbuf + eo.half * 2048u;
      eo.half ^= 1u;
      const uint32_t piece = (uint32_t)lane >> 3, inside = ((uint32_t)lane & 7u) * 2u;
#pragma unroll
      for (uint32_t i = 0; i < 16; ++i) {
        const uint32_t r0 = 2u * i, r1 = 2u * i + 1u;
        const uint32_t a0 = tt + r0 * 64u + ((piece ^ ((r0 >> 1) & 3u)) << 4) + inside;
        const uint32_t a1 = tt + r1 * 64u + ((piece ^ ((r1 >> 1) & 3u)) << 4) + inside;
        asm volatile("st.shared.b16 [%0], %1;" ::"r"(a0), "h"((unsigned short)(pk[i] & 0xffffu)) : "memory");
        asm volatile("st.shared.b16 [%0], %1;" ::"r"(a1), "h"((unsigned short)(pk[i] >> 16)) : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) bulk_store_4d(map, tt, eo.row0, col0, p, eo.z);
    }
  }
}

// 32 consecutive fp32 values of this lane's row: direct (16-byte stores of the lanes with `valid`
// rows) or through the copy engine (all lanes; block (col0, eo.row0))
__device__ __forceinline__ void store_f32x32(const float (&v)[32], float* dst, bool valid, EpiOut& eo, int col0) {
  if (eo.m_f32 == nullptr) {
    if (valid) {
      float4* d4 = reinterpret_cast<float4*>(dst);
#pragma unroll
      for (int i = 0; i < 8; ++i) d4[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    }
    return;
  }
  const int lane = threadIdx.x & 31;
  const uint32_t sw = ((uint32_t)lane >> 1) & 3u;
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {       // two blocks of 16 columns: rows of 64 bytes, as for bf16
    if (lane == 0) bulk_wait_read_but_one();
    __syncwarp();
    const uint32_t tile = eo.sbuf + eo.half * 2048u;
    eo.half ^= 1u;
    const uint32_t rowp = tile + (uint32_t)lane * 64u;
#pragma unroll
    for (uint32_t c = 0; c < 4; ++c)
      st_shared_v4(rowp + ((c ^ sw) << 4), __float_as_uint(v[16 * hh + 4 * c]), __float_as_uint(v[16 * hh + 4 * c + 1]),
                   __float_as_uint(v[16 * hh + 4 * c + 2]), __float_as_uint(v[16 * hh + 4 * c + 3]));
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) bulk_store_3d(eo.m_f32, tile, col0 + 16 * hh, eo.row0, eo.z);
  }
}

// position in the fragment stream of the first dead unit of (row, 32-column chunk at col0)
__device__ __forceinline__ uint32_t frag_base(const TcEpilogue& e, int N, int row, int col0,
                                              int64_t woff) {
  uint32_t b = e.frag_off[row] + e.frag_rank[(int64_t)row * (N >> 6) + (col0 >> 6)];
  if (col0 & 32) b += 32u - __popc(e.mask[woff - 1]);
  return b;
}

// the fused step applied to one row chunk of 32 accumulator columns
// (`prow`: the row inside the product, `row`: where its outputs live; they differ under a scatter;
// `valid`: the row exists.  With bulk output every lane of the warp comes here, rows beyond the
// product included: they touch no global memory and the copy engine clips their part of a block.)
// `mword`: the row's sign word of this chunk, fetched ahead of the accumulator (modes that read it)
__device__ __forceinline__ void epilogue_chunk(const TcEpilogue& e, int N, int prow, int row, int col0,
                                               float (&v)[32], double& sumsq_local, bool valid, EpiOut& eo,
                                               uint32_t mword) {
  const int64_t ldo = e.ld ? e.ld : (int64_t)N;
  const int64_t off = (int64_t)row * ldo + col0;
  const int64_t woff = (int64_t)row * (N >> 5) + (col0 >> 5);
  switch (e.mode) {
    case TC_EPI_PLAIN: {
      if (e.addend) {
        if (valid) {
          const float4* a4 = reinterpret_cast<const float4*>(e.addend + off);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float4 a = a4[i];
            v[4 * i] = fmaf(e.alpha, v[4 * i], a.x);
            v[4 * i + 1] = fmaf(e.alpha, v[4 * i + 1], a.y);
            v[4 * i + 2] = fmaf(e.alpha, v[4 * i + 2], a.z);
            v[4 * i + 3] = fmaf(e.alpha, v[4 * i + 3], a.w);
          }
        }
      } else if (e.alpha != 1.f) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= e.alpha;
      }
      if (e.out_f32) store_f32x32(v, e.out_f32 + off, valid, eo, col0);
      if (e.n_planes) store_planes32(v, e.planes, e.n_planes, e.plane_stride, off, valid, eo.m_pl, eo, col0);
      break;
    }
    case TC_EPI_RESID: {
      if (e.scale_dev) {
        // acc = W W^T: the factor T = c (2 I - c W W^T) of the first step X_1 = W^T T
        const float cs = __ldg(e.scale_dev);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = cs * (((col0 + i) == row ? 2.f : 0.f) - cs * v[i]);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          v[i] = ((col0 + i) == row ? 1.f : 0.f) - v[i];
          if (valid) sumsq_local += (double)v[i] * (double)v[i];
        }
      }
      if (e.out_f32) store_f32x32(v, e.out_f32 + off, valid, eo, col0);
      if (e.n_planes)
        store_planes32(v, e.planes, e.n_planes, e.plane_stride, off, valid, eo.m_pl, eo, col0, eo.mirror,
                       (int64_t)col0 * ldo + row, ldo);
      break;
    }
    case TC_EPI_FWD: {
      uint32_t word = 0xffffffffu;
      if (e.write_mask) {
        if (e.act != MW_ACT_NONE) {
          word = 0;
#pragma unroll
          for (int i = 0; i < 32; ++i) word |= (v[i] > 0.f ? 1u : 0u) << i;
        }
        if (valid) e.mask[woff] = word;
      } else if (e.act != MW_ACT_NONE && valid) {
        word = mword;
      }
      const float nf = e.act == MW_ACT_LEAKY_RELU ? e.slope : (e.act == MW_ACT_RELU ? 0.f : 1.f);
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = ((word >> i) & 1u) ? v[i] : nf * v[i];
      if (e.out_f32) store_f32x32(v, e.out_f32 + off, valid, eo, col0);
      if (e.n_planes) store_planes32(v, e.planes, e.n_planes, e.plane_stride, off, valid, eo.m_pl, eo, col0);
      break;
    }
    case TC_EPI_BWD: {
      if (e.out_f32) store_f32x32(v, e.out_f32 + off, valid, eo, col0);
      if (e.n_planes2) {   // cotangent checkpoint as term planes (the sweep reads it as an operand)
        float h[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) h[i] = v[i];
        store_planes32(h, e.planes2, e.n_planes2, e.plane_stride2,
                       e.compact2 ? (int64_t)prow * N + col0 : off, valid, eo.m_pl2, eo, col0);
      }
      const uint32_t word = (e.act != MW_ACT_NONE && valid) ? mword : 0xffffffffu;
      if (e.act == MW_ACT_RELU && e.frag_vals && valid) {
        // fragments: the cotangent at dead units, in column order
        uint32_t pos = frag_base(e, N, row, col0, woff);
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (!((word >> i) & 1u)) e.frag_vals[pos++] = v[i];
      }
      if (e.n_planes) {
        if (e.act != MW_ACT_NONE) {
          const float nf = e.act == MW_ACT_LEAKY_RELU ? e.slope : 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = ((word >> i) & 1u) ? v[i] : nf * v[i];
        }
        store_planes32(v, e.planes, e.n_planes, e.plane_stride, off, valid, eo.m_pl, eo, col0);
      }
      break;
    }
    case TC_EPI_VIJP: {
      if (e.addend && valid) {
        const float4* a4 = reinterpret_cast<const float4*>(e.addend + off);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float4 a = a4[i];
          v[4 * i] = fmaf(e.alpha, v[4 * i], a.x);
          v[4 * i + 1] = fmaf(e.alpha, v[4 * i + 1], a.y);
          v[4 * i + 2] = fmaf(e.alpha, v[4 * i + 2], a.z);
          v[4 * i + 3] = fmaf(e.alpha, v[4 * i + 3], a.w);
        }
      }
      float h[32];
      if (e.act == MW_ACT_LEAKY_RELU) {
        const uint32_t word = valid ? mword : 0xffffffffu;
        // one division per chunk: the inverse derivative is applied as a product with the
        // correctly rounded reciprocal of the slope (within an ulp of the quotient)
        const float rs = 1.f / e.slope;
#pragma unroll
        for (int i = 0; i < 32; ++i) h[i] = ((word >> i) & 1u) ? v[i] : v[i] * rs;
      } else if (e.act == MW_ACT_RELU) {
        // live units pass g_z on (phi' = 1); dead units take their stored cotangent back and
        // contribute nothing to the weight vjp
        const uint32_t word = valid ? mword : 0xffffffffu;
        uint32_t pos = valid ? frag_base(e, N, row, col0, woff) : 0u;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if ((word >> i) & 1u) {
            h[i] = v[i];
          } else {
            h[i] = e.frag_vals[pos++];
            v[i] = 0.f;
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) h[i] = v[i];
      }
      if (e.out_f32) store_f32x32(h, e.out_f32 + off, valid, eo, col0);
      if (e.n_planes2) {
        if (e.sub2_s) {
          const int hw = e.sub2_h * e.sub2_w;
          const int b = prow / hw, rem = prow - b * hw;
          const int y = rem / e.sub2_w, x = rem - y * e.sub2_w;
          if (valid && y % e.sub2_s == 0 && x % e.sub2_s == 0) {
            const int64_t r2 = ((int64_t)b * (e.sub2_h / e.sub2_s) + y / e.sub2_s) * (e.sub2_w / e.sub2_s) +
                               x / e.sub2_s;
            store_planes32(h, e.planes2, e.n_planes2, e.plane_stride2, r2 * N + col0, true, nullptr, eo, col0);
          }
        } else {
          store_planes32(h, e.planes2, e.n_planes2, e.plane_stride2, off, valid, eo.m_pl2, eo, col0);
        }
      }
      if (e.n_planes) store_planes32(v, e.planes, e.n_planes, e.plane_stride, off, valid, eo.m_pl, eo, col0);
      break;
    }
    default:
      break;
  }
}

// The K loop of one unit on the issuing lane.  A tcgen05.mma is accepted only while at most one
// earlier instruction is still running, so whatever this lane executes between the last
// instruction of a K block and the first of the next must fit into the run time of one
// instruction (128 cycles at 256 columns) or the tensor pipe idles.  Hence: straight-line code
// specialised by the instruction count, all addresses advanced by additions, and the barrier of
// the NEXT stage polled (and the next K block's operands prepared) between the first K step and
// the other three of the current block, where the latency is hidden behind the running products.
struct MmaRing {
  uint32_t stage, phase, stages;
  uint32_t sb16, tiles16, stage16;        // operand base of the stage (16-byte units), ring start, stage size
  uint32_t full, empty, full0, empty0;    // barriers of the stage, and of stage 0
};

template <int NOPS, bool kPair>
__device__ __forceinline__ bool mma_unit(MmaRing& r, const TcOp* ops, uint32_t d_set, uint32_t a_base,
                                         uint32_t b_base, uint32_t a_kadv, uint32_t b_kadv, int nkb,
                                         const WaitCtx& wc) {
  uint32_t oa[NOPS], ob[NOPS], oi[NOPS], od[NOPS], orot[NOPS], ofk[NOPS];
#pragma unroll
  for (int o = 0; o < NOPS; ++o) {
    const TcOp op = ops[o];
    oa[o] = op.a_off16 | a_base;
    ob[o] = op.b_off16 | b_base;
    oi[o] = op.idesc;
    od[o] = d_set + op.dcol;
    orot[o] = op.rot;
    ofk[o] = op.first_kbs;
  }
  bool ready = mbar_try_wait<kPair>(r.full, r.phase);
  for (int kbl = 0; kbl < nkb; ++kbl) {
    if (!ready && !mbar_wait<kPair>(r.full, r.phase, wc, 3u)) return false;
    tc_fence_after();
    uint32_t d[NOPS], a[NOPS], b[NOPS];
#pragma unroll
    for (int o = 0; o < NOPS; ++o) {
      d[o] = od[o] + ((kbl & 1) ? orot[o] : 0u);
      a[o] = oa[o] + r.sb16;
      b[o] = ob[o] + r.sb16;
      umma_bf16<kPair>(d[o], a[o], b[o], oi[o], (uint32_t)kbl < ofk[o] ? 0u : 1u);
    }
    // the ring moves on while the first products run
    const uint32_t freed = r.empty;
    r.sb16 += r.stage16; r.full += 8u; r.empty += 8u;
    if (++r.stage == r.stages) {
      r.stage = 0; r.phase ^= 1u; r.sb16 = r.tiles16; r.full = r.full0; r.empty = r.empty0;
    }
    ready = (kbl + 1 < nkb) && mbar_try_wait<kPair>(r.full, r.phase);
#pragma unroll
    for (int k4 = 1; k4 < BK / 16; ++k4) {
#pragma unroll
      for (int o = 0; o < NOPS; ++o)
        umma_bf16<kPair>(d[o], a[o] + (uint32_t)k4 * a_kadv, b[o] + (uint32_t)k4 * b_kadv, oi[o], 1u);
    }
    umma_commit<kPair>(freed);   // frees the stage once these products retire
  }
  return true;
}

// unit u of the sorted list -> product, tile, batch item and K range
__device__ __forceinline__ void decode_unit(const TcProblem* probs, const int* ub, int nprob, int u,
                                            int& q, Unit& w) {
  while (q + 1 < nprob && u >= ub[q + 1]) ++q;    // units come in increasing order
  const TcProblem& P = probs[q];
  const int local = u - P.unit_begin;
  const int tl = local / P.split;
  const int ks = local - tl * P.split;
  const int z = tl / P.tiles_mn;
  const int r = tl - z * P.tiles_mn;
  int mt = r / P.tiles_n, nt = r - mt * P.tiles_n;
  if (P.sym) {
    // tiles that reach the diagonal or lie above it, row by row: row m starts at the tile that
    // holds column m * bm
    int t = r;
    mt = 0;
    for (;;) {
      const int start = (mt * P.bm) / P.bn, len = P.tiles_n - start;
      if (t < len) { nt = start + t; break; }
      t -= len;
      ++mt;
    }
  }
  w.q = q;
  w.tl = tl;
  w.ks = ks;
  w.z = z;
  w.m0 = mt * P.bm;
  w.n0 = nt * P.bn;
  w.kb0 = ks * P.kb_per_split;
  const int e = w.kb0 + P.kb_per_split;
  w.kb1 = e < P.num_kb ? e : P.num_kb;
}

// Units of this CTA (pair form: of this pair of CTAs).  Grouped launch: round r takes index
// r*G + c (even r) or r*G + G-1-c (odd r).  Program launch: the host's schedule (balance_units)
// when there is one, else r*G + c throughout, so that one CTA never holds two units of one short
// product (they would run one after the other and hold up everything that waits for it).
// (Handing units out at run time from a counter, in list order, was tried twice and is not
// faster: CTAs pile up behind the one product that is not complete yet.)
template <bool kProgram, bool kPair>
__device__ __forceinline__ int next_unit(const TcGroupParams& p, int& r) {
  const int G = (int)(gridDim.x >> (kPair ? 1 : 0)), c = (int)(blockIdx.x >> (kPair ? 1 : 0));
  if (kProgram && p.sched) {
    if (r >= p.sched_len) return -1;
    const int u = __ldg(p.sched + (size_t)c * p.sched_len + r);
    ++r;
    return u;
  }
  while (r * G < p.total_units) {
    const int u = r * G + (((r & 1) && !kProgram) ? G - 1 - c : c);
    ++r;
    if (u < p.total_units) return u;
  }
  return -1;
}

// kProgram: the products live in global memory and wait for one another (program launch);
// otherwise they are read straight from the kernel parameters.
// kPair: launched as clusters of two CTAs that share every tile (see the top of the file).
template <bool kProgram, bool kPair>
__global__ void __launch_bounds__(kThreadsTc, 1)
tc_group_kernel(const __grid_constant__ TcGroupParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kMaxStages];
  __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
  __shared__ __align__(8) uint64_t acc_full[2];
  __shared__ __align__(8) uint64_t acc_empty[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ int ub[kMaxProgram + 1];     // first unit of every product

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // pair form: rank 0 (the even CTA) issues the products and owns the barriers both CTAs report to
  const uint32_t rank = kPair ? cluster_cta_rank() : 0u;
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;  // 1024-byte aligned for the swizzle
  // Launched with programmatic stream serialisation, this grid may start while the previous
  // kernel of the stream is still finishing: everything up to the waits below (barriers, tensor
  // memory, tensor-map prefetch) then overlaps that kernel's tail.  Let the next one do the same.
  if (!kProgram) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const TcProblem* probs = kProgram ? p.table : p.prob;
  const int nprob = p.nprob;
  for (int i = threadIdx.x; i < nprob; i += kThreadsTc) ub[i] = probs[i].unit_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&acc_full[s]), 1);
      // one arrival per epilogue warp (of both CTAs in the pair form)
      mbar_init(smem_u32(&acc_empty[s]), kEpiWarps * (kPair ? 2 : 1));
    }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2 && lane < 2 * nprob && lane < 2 * kTcMaxGroup) {
    // start fetching the tensor maps before the first copy needs them
    const TcProblem& P = probs[lane >> 1];
    const CUtensorMap* tm = (lane & 1) ? &P.tmB : &P.tmA;
    if (P.unit_count > 0)     // (a group entry of a program has no maps)
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tm)) : "memory");
  }
  if (warp == 1) {
    // pair form: the same warp of both CTAs allocates, and both get the same columns
    if (kPair) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                       smem_u32(&tmem_slot)),
                   "r"((uint32_t)kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                       smem_u32(&tmem_slot)),
                   "r"((uint32_t)kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  // pair form: no copy may complete on, and no warp may arrive at, a barrier of the other CTA
  // before that CTA has initialised it
  if (kPair) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  WaitCtx wc;
  wc.st = p.st;
  wc.abort_flag = &abort_flag;
  wc.limit_ns = p.wait_limit_ns;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      int q = 0, rr = 0;
      // operands may come from the previous kernel of the stream
      if (!kProgram) asm volatile("griddepcontrol.wait;" ::: "memory");
      for (;;) {
        if (!ok) break;
        const int u = next_unit<kProgram, kPair>(p, rr);
        if (u < 0) break;
        Unit w;
        decode_unit(probs, ub, nprob, u, q, w);
        const TcProblem& P = probs[w.q];
        if (kProgram && P.ndep) {
          // program launch: the operands are written by earlier products of this same launch
          for (int i = 0; i < P.ndep && ok; ++i) ok = wait_done(p.done + P.dep[i], P.dep_target[i], wc);
          if (!ok) break;
          asm volatile("fence.proxy.async;" ::: "memory");   // their stores, then our bulk copies
        }
        const int a_pl0 = w.z * P.a_batch_planes, b_pl0 = w.z * P.b_batch_planes;
        const int pa = P.pa, pb = P.pb;
        const bool a_mn = P.a_mn != 0, b_mn = P.b_mn != 0;
        const uint32_t b_tile_bytes = P.b_tile_bytes, tx = P.tx_bytes;
        // this CTA's rows of A and columns of B (pair form: its half of the tile)
        const int am0 = w.m0 + (kPair ? (int)rank * BM : 0);
        const int bcols = kPair ? (P.bn >> 1) : P.bn;
        const int bn_first = w.n0 + (kPair ? (int)rank * bcols : 0);
        const int nbox = bcols >> 6;
        const int conv = kPair ? (int)TC_CONV_NONE : P.conv_mode;
        // convolution: image, row and column of the first pixel of the unit's tile
        int cb = 0, cy0 = 0, cx0 = 0;
        if (conv == TC_CONV_PIXELS) {
          const int hw = P.cHo * P.cWo;
          cb = w.m0 / hw;
          const int rem = w.m0 - cb * hw;
          cy0 = rem / P.cWo;
          cx0 = rem - cy0 * P.cWo;
        }
        // weight vjp: the window of each half of the A tile (constant over the K blocks) and the
        // position of the unit's first K block; the divisions are kept out of the K loop, where
        // this single lane's integer work is what paces the copies
        int px_t = 0, px_c = 0;      // window and channel block of the next K block (TC_CONV_PIXELS)
        if (conv == TC_CONV_PIXELS) {
          px_t = w.kb0 / P.ccb;
          px_c = w.kb0 - px_t * P.ccb;
        }
        int wg_c0[2] = {0, 0}, wg_ox[2] = {0, 0}, wg_oy[2] = {0, 0};
        int wg_b = 0, wg_y = 0, wg_x = 0;
        if (conv == TC_CONV_WGRAD) {
          const int r0 = 2 * (w.m0 / BM);
          for (int hh = 0; hh < 2; ++hh) {
            int tap = (r0 + hh) / P.ccb;
            wg_c0[hh] = ((r0 + hh) - tap * P.ccb) * BK;
            if (tap >= P.cntaps) tap = P.cntaps - 1;   // rows past the last tap are never stored
            const int j0 = P.c1d ? 0 : tap / P.ck, j1 = tap - j0 * P.ck;
            wg_ox[hh] = j1 - P.cpad;
            wg_oy[hh] = P.c1d ? 0 : j0 - P.cpad;
          }
          const int pix = (w.z * P.num_kb + w.kb0) * BK;
          const int hw = P.cHo * P.cWo;
          wg_b = pix / hw;
          const int rem = pix - wg_b * hw;
          wg_y = rem / P.cWo;
          wg_x = rem - wg_y * P.cWo;
        }
        if (conv == TC_CONV_NONE) {
          // Lean loop of the plain products.  This lane runs alone: whatever it computes between
          // two copies delays the copies, so everything that does not change is hoisted and the
          // barrier of the NEXT stage is polled while this stage's copies are being issued.
          const CUtensorMap* tmA = &P.tmA;
          const CUtensorMap* tmB = &P.tmB;
          const uint32_t b_off = (uint32_t)pa * kATileBytes;
          const uint32_t txe = kPair ? 2u * tx : tx;
          const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
          // pair form: the bytes of both CTAs are counted on the even CTA's barrier, which expects them all
          const uint32_t full0_remote = kPair ? map_to_cta(full0, 0u) : full0;
          const uint32_t stages = (uint32_t)p.stages, stage_bytes = p.stage_bytes;
          uint32_t sbase = tiles + stage * stage_bytes;
          bool ready = mbar_try_wait<kPair>(empty0 + 8u * stage, phase ^ 1u);
          int k0 = w.kb0 * BK;
          for (int kb = w.kb0; kb < w.kb1; ++kb, k0 += BK) {
            if (!ready && !mbar_wait<kPair>(empty0 + 8u * stage, phase ^ 1u, wc, 1u)) { ok = false; break; }
            if (!kPair || rank == 0) mbar_expect_tx(full0 + 8u * stage, txe);
            const uint32_t fb = full0_remote + 8u * stage;
            if (a_mn) tma_load_4d<kPair>(sbase, tmA, fb, 0, k0, am0 >> 6, a_pl0);
            else tma_load_3d<kPair>(sbase, tmA, fb, k0, am0, a_pl0);
            if (b_mn) tma_load_4d<kPair>(sbase + b_off, tmB, fb, 0, k0, bn_first >> 6, b_pl0);
            else tma_load_3d<kPair>(sbase + b_off, tmB, fb, k0, bn_first, b_pl0);
            sbase += stage_bytes;
            if (++stage == stages) { stage = 0; phase ^= 1u; sbase = tiles; }
            ready = mbar_try_wait<kPair>(empty0 + 8u * stage, phase ^ 1u);
          }
          continue;
        }
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!mbar_wait<kPair>(smem_u32(&empty_bar[stage]), phase ^ 1u, wc, 1u)) { ok = false; break; }
          const uint32_t fb = smem_u32(&full_bar[stage]);
          mbar_expect_tx(fb, tx);
          const uint32_t sbase = tiles + stage * p.stage_bytes;
          int k0 = kb * BK;
          int bk0 = k0, bn0 = bn_first;       // B coordinates (K, N)
          if (conv == TC_CONV_PIXELS) {
            const int t = px_t, cblk = px_c;
            if (++px_c == P.ccb) { px_c = 0; ++px_t; }
            const int dy = P.tdy[t], dx = P.tdx[t], tb = P.ttb[t];
            for (int pl = 0; pl < pa; ++pl)
              tma_load_5d(sbase + (uint32_t)pl * kATileBytes, &P.tmA, fb, cblk * BK, P.cstride * cx0 + dx,
                          P.cstride * cy0 + dy, cb, a_pl0 + pl);
            bk0 = (tb * P.ccb + cblk) * BK;
            if (P.b_tap_rows) { bn0 = tb * P.N + w.n0; bk0 = cblk * BK; }
          } else {
            // K block = 64 pixels of slice z (one box: part of a row, rows, or images); the two
            // halves of the A tile are two blocks of 64 rows (tap, channel block)
            const int pix = (w.z * P.num_kb + kb) * BK;
            for (int hh = 0; hh < 2; ++hh)
              for (int pl = 0; pl < pa; ++pl)
                tma_load_5d(sbase + (uint32_t)pl * kATileBytes + (uint32_t)hh * 8192u, &P.tmA, fb, wg_c0[hh],
                            P.cstride * wg_x + wg_ox[hh], P.cstride * wg_y + wg_oy[hh], wg_b, pl);
            // next box
            wg_x += P.cbx;
            if (wg_x >= P.cWo) {
              wg_x = 0;
              wg_y += P.cby;
              if (wg_y >= P.cHo) { wg_y = 0; wg_b += P.cbi; }
            }
            bk0 = pix;
            k0 = pix;
          }
          const uint32_t bbase = sbase + (uint32_t)pa * kATileBytes;
          const int bz = conv == TC_CONV_WGRAD ? 0 : b_pl0;
          for (int pl = 0; pl < pb; ++pl) {
            const uint32_t dst = bbase + (uint32_t)pl * b_tile_bytes;
            if (b_mn) {
              for (int h = 0; h < nbox; ++h)
                tma_load_3d<false>(dst + (uint32_t)h * 8192u, &P.tmB, fb, bn0 + h * 64, bk0, bz + pl);
            } else {
              tma_load_3d<false>(dst, &P.tmB, fb, bk0, bn0, bz + pl);
            }
          }
          if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (pair form: of the even CTA only) ----------------
    if (lane == 0 && rank == 0) {
      MmaRing ring;
      ring.stage = 0; ring.phase = 0; ring.stages = (uint32_t)p.stages;
      ring.tiles16 = tiles >> 4; ring.stage16 = p.stage_bytes >> 4; ring.sb16 = ring.tiles16;
      ring.full0 = smem_u32(&full_bar[0]); ring.empty0 = smem_u32(&empty_bar[0]);
      ring.full = ring.full0; ring.empty = ring.empty0;
      int j = 0, q = 0, rr = 0;
      for (;;) {
        const int u = next_unit<kProgram, kPair>(p, rr);
        if (u < 0) break;
        Unit w;
        decode_unit(probs, ub, nprob, u, q, w);
        const TcProblem& P = probs[w.q];
        const uint32_t set = (uint32_t)j & 1u, aphase = ((uint32_t)j >> 1) & 1u;
        if (!mbar_wait<kPair>(smem_u32(&acc_empty[set]), aphase ^ 1u, wc, 2u)) break;
        tc_fence_after();
        const uint32_t d_set = tmem_base + set * (uint32_t)kSetCols;
        // K advance of 16 elements: 32 bytes along a K-major row, 16 rows of 128 bytes otherwise
        const uint32_t a_kadv = P.a_mn ? (2048u >> 4) : (32u >> 4);
        const uint32_t b_kadv = P.b_mn ? (2048u >> 4) : (32u >> 4);
        const int nkb = w.kb1 - w.kb0;
        bool ok;
        switch (P.nops) {
          case 1: ok = mma_unit<1, kPair>(ring, P.ops, d_set, P.a_desc_base, P.b_desc_base, a_kadv, b_kadv, nkb, wc); break;
          case 2: ok = mma_unit<2, kPair>(ring, P.ops, d_set, P.a_desc_base, P.b_desc_base, a_kadv, b_kadv, nkb, wc); break;
          case 3: ok = mma_unit<3, kPair>(ring, P.ops, d_set, P.a_desc_base, P.b_desc_base, a_kadv, b_kadv, nkb, wc); break;
          case 4: ok = mma_unit<4, kPair>(ring, P.ops, d_set, P.a_desc_base, P.b_desc_base, a_kadv, b_kadv, nkb, wc); break;
          case 5: ok = mma_unit<5, kPair>(ring, P.ops, d_set, P.a_desc_base, P.b_desc_base, a_kadv, b_kadv, nkb, wc); break;
          default: ok = mma_unit<6, kPair>(ring, P.ops, d_set, P.a_desc_base, P.b_desc_base, a_kadv, b_kadv, nkb, wc); break;
        }
        if (!ok) break;
        umma_commit<kPair>(smem_u32(&acc_full[set]));
        ++j;
      }
    }
  } else {
    // ---------------- epilogue (warps 2..5) ----------------
    const int quarter = warp & 3;                 // tensor-memory lane quarter this warp may read
    const int half = 0;
    // this warp's buffer for bulk stores (0: none, direct stores)
    // (pair form only: the one-CTA form serves the small fp32-accurate tiles and the convolution
    // windows, whose epilogues are at the register limit without it)
    const uint32_t epi_sbuf = (kPair && p.epi_stage_off) ? tiles + p.epi_stage_off + (uint32_t)quarter * kEpiStageBytes : 0u;
    bool bulk_used = false;
    int j = 0, q = 0, rr = 0;
    bool ok = true;
    // sign words, addends, fragments read here and everything stored here may be in use by the
    // previous kernel of the stream
    if (!kProgram) asm volatile("griddepcontrol.wait;" ::: "memory");
    for (;;) {
      if (!ok) break;
      const int u = next_unit<kProgram, kPair>(p, rr);
      if (u < 0) break;
      Unit w;
      decode_unit(probs, ub, nprob, u, q, w);
      const TcProblem& P = probs[w.q];
      const uint32_t set = (uint32_t)j & 1u, aphase = ((uint32_t)j >> 1) & 1u;
      // pair form: this CTA's tensor memory holds rows rank*128 .. rank*128+127 of the tile
      const int row = w.m0 + (kPair ? (int)rank * BM : 0) + quarter * 32 + lane;
      const int bn = P.bn, nblk = P.nblocks, N = P.N;
      TcEpilogue epi = P.epi;           // this batch item's view of the outputs
      int orow = row;                   // where the row's outputs live
      if (epi.remap_s) {
        const int hw = epi.remap_ho * epi.remap_wo;
        const int b = row / hw, rem = row - b * hw;
        const int y = rem / epi.remap_wo, x = rem - y * epi.remap_wo;
        orow = (b * epi.remap_ho * epi.remap_s + epi.remap_s * y + epi.remap_py) *
                   (epi.remap_wo * epi.remap_s) + epi.remap_s * x + epi.remap_px;
      }
      if (w.z) {
        const int64_t z = w.z;
        if (epi.addend) epi.addend += z * epi.bs_f32;
        if (epi.out_f32) epi.out_f32 += z * epi.bs_f32;
        if (epi.planes) epi.planes += z * epi.bs_planes;
        if (epi.planes2) epi.planes2 += z * epi.bs_planes2;
        if (epi.mask) epi.mask += z * epi.bs_mask;
        if (epi.sumsq) epi.sumsq += z * epi.bs_sumsq;
        if (epi.scale_dev) epi.scale_dev += z;
      }
      // The row's sign words of this tile are fetched now, while the products are still running:
      // read inside the chunk loop, each would put a trip to global memory on the epilogue's
      // critical path.  (Sign words are never written by the launch that reads them.)
      uint32_t mw[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) mw[i] = 0xffffffffu;
      const bool early_words = kPair;
      if (early_words && epi.mask && epi.act != MW_ACT_NONE && row < P.M &&
          ((epi.mode == TC_EPI_FWD && !epi.write_mask) || epi.mode == TC_EPI_BWD || epi.mode == TC_EPI_VIJP)) {
        const uint32_t* mrow = epi.mask + (int64_t)orow * (N >> 5) + (w.n0 >> 5);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (32 * i < bn && w.n0 + 32 * i < N) mw[i] = mrow[i];
      }
      // every lane observes the barrier itself; the warp then takes one common decision so the
      // warp-wide tensor-memory loads below are never executed by part of a warp
      ok = __all_sync(0xffffffffu, mbar_wait<kPair>(smem_u32(&acc_full[set]), aphase, wc, 4u));
      if (!ok) break;
      tc_fence_after();
      double sumsq_local = 0.0;
      EpiOut eo;
      if (epi_sbuf && P.out_tma) {
        // the copy engine must have read what the previous unit left in the buffer
        if (bulk_used) {
          if (lane == 0) bulk_wait_read_all();
          __syncwarp();
        }
        bulk_used = true;
        eo.sbuf = epi_sbuf;
        eo.m_f32 = (P.out_tma & 1) ? &P.tmO : nullptr;
        eo.m_pl = (P.out_tma & 2) ? &P.tmP : nullptr;
        eo.m_pl2 = (P.out_tma & 4) ? &P.tmP2 : nullptr;
        eo.row0 = row - lane;
        eo.z = w.z;
      }
      // symmetric product: a tile that lies wholly above the diagonal stands for its mirror image too
      eo.mirror = P.sym && w.n0 >= w.m0 + P.bm;
      const uint32_t t0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + set * (uint32_t)kSetCols;
      // sum of the column blocks of 32 accumulator columns starting at c
      auto load_chunk = [&](int c, float (&v)[32]) {
        uint32_t r0[32];
        tmem_ld32_issue(t0 + (uint32_t)c, r0);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r0[i]);
        for (int b = 1; b < nblk; ++b) {
          tmem_ld32_issue(t0 + (uint32_t)(b * bn + c), r0);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] += __uint_as_float(r0[i]);
        }
      };
      bool fused_step = true;
      if (!kPair && P.split > 1) {
        // K split: leave this piece of the tile in the meeting place, element (row, c + i) of
        // piece s at ((s * nchunk + c / 32) * 32 + i) * 128 + row so that a warp writes whole lines
        float* mine = P.split_partials + ((int64_t)w.tl * P.split + w.ks) * (int64_t)(BM * bn) +
                      quarter * 32 + lane;
#pragma unroll 1
        for (int c = half * 32; c < bn; c += 32 * (kEpiWarps / 4)) {
          if (w.n0 + c >= N) break;
          float v[32];
          load_chunk(c, v);
          float* dst = mine + (int64_t)c * BM;
#pragma unroll
          for (int i = 0; i < 32; ++i) dst[i * BM] = v[i];
        }
        __threadfence();
        __syncwarp();
        unsigned int* cnt = P.split_counters + (int64_t)w.tl * kEpiWarps + quarter * (kEpiWarps / 4) + half;
        unsigned int old = 0;
        if (lane == 0) old = atomicAdd(cnt, 1u);
        old = __shfl_sync(0xffffffffu, old, 0);
        // the warp that finds the other pieces of its 32 rows complete adds all pieces in fixed
        // order (its own straight from tensor memory) and applies the fused step
        fused_step = old == (unsigned)P.split - 1u;
        if (fused_step) {
          __threadfence();
          if (lane == 0) *cnt = 0u;     // ready for the next launch
        }
      }
      if (fused_step) {
        const bool split = !kPair && P.split > 1;
        const float* others = split ? P.split_partials + (int64_t)w.tl * P.split * (int64_t)(BM * bn) +
                                          quarter * 32 + lane
                                    : nullptr;
#pragma unroll 1
        for (int c = half * 32; c < bn; c += 32 * (kEpiWarps / 4)) {
          if (w.n0 + c >= N) break;
          float v[32];
          if (split) {
            float own[32];
            load_chunk(c, own);
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0.f;
            // two pieces per round trip (all loads of a pair are in flight together), added in
            // index order with this warp's own piece in its place
            for (int sp = 0; sp < P.split; sp += 2) {
              const bool has1 = sp + 1 < P.split;
              const float* s0 = others + (int64_t)sp * (BM * bn) + (int64_t)c * BM;
              const float* s1 = s0 + (int64_t)(BM * bn);
              float t0[32], t1[32];
              if (sp != w.ks) {
#pragma unroll
                for (int i = 0; i < 32; ++i) t0[i] = __ldcg(s0 + i * BM);
              }
              if (has1 && sp + 1 != w.ks) {
#pragma unroll
                for (int i = 0; i < 32; ++i) t1[i] = __ldcg(s1 + i * BM);
              }
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] += sp == w.ks ? own[i] : t0[i];
              if (has1) {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] += sp + 1 == w.ks ? own[i] : t1[i];
              }
            }
          } else {
            load_chunk(c, v);
          }
          if (row < P.M || eo.sbuf) {
            const int ci = c >> 5;      // the chunk's sign word, by selection (no indexed registers)
            const uint32_t lo = ci & 2 ? (ci & 1 ? mw[3] : mw[2]) : (ci & 1 ? mw[1] : mw[0]);
            const uint32_t hi = ci & 2 ? (ci & 1 ? mw[7] : mw[6]) : (ci & 1 ? mw[5] : mw[4]);
            uint32_t mword = ci & 4 ? hi : lo;
            if (!early_words && epi.mask && epi.act != MW_ACT_NONE && row < P.M &&
                ((epi.mode == TC_EPI_FWD && !epi.write_mask) || epi.mode == TC_EPI_BWD || epi.mode == TC_EPI_VIJP))
              mword = epi.mask[(int64_t)orow * (N >> 5) + ((w.n0 + c) >> 5)];
            epilogue_chunk(epi, N, row, orow, w.n0 + c, v, sumsq_local, row < P.M, eo, mword);
          }
        }
      }
      // this warp has read its part of the accumulator set: hand it back to the MMA issuer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (kPair && rank != 0) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[set]), 0u));
        else mbar_arrive(smem_u32(&acc_empty[set]));
      }
      ++j;
      if (epi.mode == TC_EPI_RESID && epi.sumsq && fused_step) {
        // this warp's share of ||v||_F^2 goes to a slot of its own (fixed-order sum by the reader)
        for (int o = 16; o; o >>= 1) sumsq_local += __shfl_xor_sync(0xffffffffu, sumsq_local, o);
        if (lane == 0) {
          epi.sumsq[((int64_t)(row >> 7) * P.tiles_n + w.n0 / bn) * kEpiWarps + quarter] = sumsq_local;
          // symmetric product: the tile below the diagonal that this one stands for has the same sum
          // (pair form: written to that tile's slots; one-CTA form: counted twice here, the slots of
          // the tiles that are left out stay as the caller zeroed them)
          if (eo.mirror) {
            if (kPair)
              epi.sumsq[((int64_t)(2 * (w.n0 / bn) + (int)rank) * P.tiles_n + w.m0 / P.bm) * kEpiWarps + quarter] =
                  sumsq_local;
            else
              epi.sumsq[((int64_t)(row >> 7) * P.tiles_n + w.n0 / bn) * kEpiWarps + quarter] = 2.0 * sumsq_local;
          }
        }
      }
      if (kProgram && fused_step) {
        // program launch: publish this warp's part of the tile to the products that wait for it
        // (bulk stores must have been written, not just read from the buffer)
        if (eo.sbuf) {
          if (lane == 0) bulk_wait_all();
          __syncwarp();
        }
        __threadfence();
        __syncwarp();
        if (lane == 0) {
          atomicAdd(p.done + w.q, 1u);
          if (P.done2 >= 0) atomicAdd(p.done + P.done2, 1u);
        }
      }
    }
  }
  // bulk stores of this thread complete before the CTA retires
  if (warp >= 2 && lane == 0) bulk_wait_all();
  tc_fence_before();
  __syncthreads();
  if (warp == 0 && lane == 0 && abort_flag) {
    // a wait ran out: give copies still in flight a bounded time to land before the CTA retires
    for (int s = 0; s < p.stages; ++s)
      for (uint32_t i = 0; i < 4096u && !mbar_try_wait<kPair>(smem_u32(&full_bar[s]), 0u); ++i) __nanosleep(256);
  }
  // pair form: neither CTA may retire (or give up its tensor memory) while the other may still
  // arrive at its barriers or have products running on both tensor memories; every role of both
  // CTAs gets here through bounded waits
  if (kPair) cluster_sync_all();
  tc_fence_after();
  if (warp == 1) {
    if (kPair)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                   : "memory");
  }
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  }
  return fn;
}

constexpr int kMaxDevices = 64;
int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
  return dev;
}

// SMs of the current device (cached per device)
int sm_count() {
  static int n[kMaxDevices] = {};
  const int dev = current_device();
  if (n[dev] == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    n[dev] = v;
  }
  return n[dev];
}

// tile width: as wide as the accumulator set allows for the number of term orders.  Narrower
// tiles would give a small product more CTAs, but instructions below 128 columns are issue bound
// (about 57 cycles each whatever their width); a product that needs more CTAs is cut along K.
int pick_bn(int pa, int pb, int M, int N, int batch, bool wide = false) {
  (void)M; (void)batch; (void)wide;
  const int t = pa > pb ? pa : pb;
  int bn = t == 1 ? 256 : (t == 2 ? 128 : 64);
  while (bn > 64 && N % bn != 0) bn >>= 1;
  return bn;
}

// Pair form, two-term operands: 1 = all kept cross products of a tile accumulate in ONE block of 256
// columns (three full-width instructions per K step, both accumulator sets in use); 0 = products of
// order 0 and order 1 in blocks of their own, which halves the tile (instructions of 128 columns
// run at two thirds of the tensor rate).
int g_merge_orders = 1;

// tile width in the pair form
int pair_bn(int pa, int pb, int N) {
  const int t = pa > pb ? pa : pb;
  int bn = (t == 1 || g_merge_orders) ? 256 : 128;
  while (bn > 128 && N % bn != 0) bn >>= 1;
  return bn;
}

// 0: never use the pair form, 1: wherever a launch qualifies (default)
int g_pair_mode = 1;
// 1: epilogues hand plain outputs to the copy engine (0: per-lane stores everywhere)
int g_bulk_epilogue = 1;

// Can this product run in the pair form?  Operands of at most two terms (the accumulator blocks
// of a 128-column tile then fit one set), tiles at least 128 columns wide (each CTA stages whole
// 64-column boxes of its half), whole 256-row tiles, no convolution window, no K split.
bool pair_capable(const TcGemm& d) {
  if (d.conv.mode != TC_CONV_NONE || d.split_k > 1) return false;
  if (d.A.planes > 2 || d.B.planes > 2) return false;
  if (d.M % 256 != 0 || d.N % 128 != 0) return false;
  return true;
}

}  // namespace

int tc_tile_n(int a_planes, int b_planes, int M, int N, int batch) {
  return pick_bn(a_planes, b_planes, M, N, batch);
}

size_t tc_split_scratch_bytes(int a_planes, int b_planes, int M, int N, int batch, int split_k) {
  if (split_k <= 1) return 0;
  const int bn = pick_bn(a_planes, b_planes, M, N, batch);
  const size_t tiles = (size_t)((M + BM - 1) / BM) * ((N + bn - 1) / bn) * batch;
  return kTcSplitCounterBytes + align_up(tiles * split_k * BM * bn * sizeof(float), 256);
}

int tc_auto_split(int a_planes, int b_planes, int M, int N, int K, int batch) {
  const int bn = pick_bn(a_planes, b_planes, M, N, batch);
  const int64_t units = (int64_t)((M + BM - 1) / BM) * ((N + bn - 1) / bn) * batch;
  // only 64-column tiles are cut: the pieces of a wider tile are too costly to add up
  if (bn > 64) return 1;
  // as many pieces as keep every piece on an SM of its own, each at least four K blocks deep
  int s = (int)(sm_count() / units);
  const int num_kb = (K + BK - 1) / BK;
  if (s > num_kb / 4) s = num_kb / 4;
  if (s > 4) s = 4;
  return s < 1 ? 1 : s;
}

// ---- optional per-launch timing of the product kernel (measurement hook) -----------------
struct TcProfile {
  bool on = false;
  std::vector<cudaEvent_t> pool;      // pairs: [2i] before, [2i+1] after
  size_t used = 0;
  double flops = 0.0, mma_flops = 0.0;
};
static TcProfile g_prof;

void tc_profile_begin() {
  g_prof.on = true;
  g_prof.used = 0;
  g_prof.flops = g_prof.mma_flops = 0.0;
}

mw_status tc_profile_end(double* total_ms, long long* launches, double* flops, double* mma_flops) {
  g_prof.on = false;
  double ms = 0.0;
  for (size_t i = 0; i + 1 < g_prof.used; i += 2) {
    if (cudaEventSynchronize(g_prof.pool[i + 1]) != cudaSuccess) return MW_ERR_CUDA;
    float t = 0.f;
    if (cudaEventElapsedTime(&t, g_prof.pool[i], g_prof.pool[i + 1]) != cudaSuccess) return MW_ERR_CUDA;
    ms += t;
  }
  if (total_ms) *total_ms = ms;
  if (launches) *launches = (long long)(g_prof.used / 2);
  if (flops) *flops = g_prof.flops;
  if (mma_flops) *mma_flops = g_prof.mma_flops;
  return MW_OK;
}

static cudaEvent_t prof_event() {
  if (g_prof.used == g_prof.pool.size()) {
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    g_prof.pool.push_back(e);
  }
  return g_prof.pool[g_prof.used++];
}

struct TcMapCache {
  std::map<std::tuple<const void*, int, int, int, int64_t, int64_t>, CUtensorMap> maps;
};
TcMapCache* tc_cache_create() { return new TcMapCache(); }
void tc_cache_destroy(TcMapCache* c) { delete c; }

static mw_status get_map(TcMapCache* cache, const TcOperand& op, int box_rows, int total_planes,
                         CUtensorMap* out, int box_planes = 1) {
  const int64_t ld = op.ld ? op.ld : op.cols;
  auto key = std::make_tuple(op.base, op.rows, op.cols, total_planes, op.plane_stride,
                             (int64_t)box_rows + ((int64_t)box_planes << 10) + (ld << 12));
  if (cache) {
    auto it = cache->maps.find(key);
    if (it != cache->maps.end()) { *out = it->second; return MW_OK; }
  }
  auto fn = encode_fn();
  if (!fn) return MW_ERR_CUDA;
  if (((uintptr_t)op.base & 15u) || (op.cols % 8) != 0 || (ld % 8) != 0 || ld < op.cols) return MW_ERR_INVALID_ARG;
  const int64_t ps = total_planes > 1 ? op.plane_stride : (int64_t)op.rows * ld;
  if (ps % 8 != 0) return MW_ERR_INVALID_ARG;
  cuuint64_t dims[3] = {(cuuint64_t)op.cols, (cuuint64_t)op.rows, (cuuint64_t)total_planes};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)ps * 2};
  cuuint32_t box[3] = {64u, (cuuint32_t)box_rows, (cuuint32_t)box_planes};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(op.base), dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return MW_ERR_CUDA;
  if (cache) cache->maps[key] = *out;
  return MW_OK;
}

// MN-major operand [rows = K][cols] per plane, seen as (column inside its group of 64, k, group,
// plane): one box {64, 64, groups, planes} lands as [plane][group][64 k][64], the layout the
// product's operand descriptors expect (groups 8 KB apart)
static mw_status get_map_mn(TcMapCache* cache, const TcOperand& op, int groups, int total_planes,
                            int box_planes, CUtensorMap* out) {
  const int64_t ld = op.ld ? op.ld : op.cols;
  auto key = std::make_tuple(op.base, op.rows, op.cols, total_planes, op.plane_stride,
                             ((int64_t)1 << 61) + groups + ((int64_t)box_planes << 10) + (ld << 12));
  if (cache) {
    auto it = cache->maps.find(key);
    if (it != cache->maps.end()) { *out = it->second; return MW_OK; }
  }
  auto fn = encode_fn();
  if (!fn) return MW_ERR_CUDA;
  if (((uintptr_t)op.base & 15u) || (op.cols % 64) != 0 || (ld % 8) != 0 || ld < op.cols) return MW_ERR_INVALID_ARG;
  const int64_t ps = total_planes > 1 ? op.plane_stride : (int64_t)op.rows * ld;
  if (ps % 8 != 0) return MW_ERR_INVALID_ARG;
  cuuint64_t dims[4] = {64u, (cuuint64_t)op.rows, (cuuint64_t)(op.cols / 64), (cuuint64_t)total_planes};
  cuuint64_t strides[3] = {(cuuint64_t)ld * 2, 128u, (cuuint64_t)ps * 2};
  cuuint32_t box[4] = {64u, 64u, (cuuint32_t)groups, (cuuint32_t)box_planes};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(op.base), dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return MW_ERR_CUDA;
  if (cache) cache->maps[key] = *out;
  return MW_OK;
}

// Output of a product for the epilogue's bulk stores: [rows][cols] with `ld` elements between rows,
// `planes` of them `plane_stride` apart, `batch` items `batch_stride` apart; blocks of 32 rows of 64
// bytes (32 bf16 or 16 fp32 columns) in the 64-byte swizzle, which makes the epilogue's 16-byte
// shared-memory stores conflict-free.  Returns false when the array does not qualify.
static bool get_out_map(TcMapCache* cache, const void* base, bool f32, int rows, int cols, int64_t ld,
                        int planes, int64_t plane_stride, int batch, int64_t batch_stride, CUtensorMap* out) {
  const int64_t es = f32 ? 4 : 2;
  if (!base || ((uintptr_t)base & 15u) || cols % 32 != 0 || (ld * es) % 16 != 0 || ld < cols) return false;
  if (planes < 1) planes = 1;
  if (batch < 1) batch = 1;
  if (planes > 1 && ((plane_stride * es) % 16 != 0 || plane_stride <= 0)) return false;
  if (batch > 1 && ((batch_stride * es) % 16 != 0 || batch_stride <= 0)) return false;
  auto key = std::make_tuple(base, rows, cols, planes * 4096 + batch, plane_stride,
                             ((int64_t)1 << 60) + (f32 ? 1 : 0) + (ld << 4) + (batch_stride << 34));
  if (cache) {
    auto it = cache->maps.find(key);
    if (it != cache->maps.end()) { *out = it->second; return true; }
  }
  auto fn = encode_fn();
  if (!fn) return false;
  // strides of dimensions of extent 1 are never used but must be valid
  const int64_t s_row = ld * es;
  const int64_t s_pl = planes > 1 ? plane_stride * es : s_row * rows;
  const int64_t s_b = batch > 1 ? batch_stride * es : s_pl * planes;
  CUresult r;
  if (f32) {
    if (planes != 1) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)batch};
    cuuint64_t strides[2] = {(cuuint64_t)s_row, (cuuint64_t)s_b};
    cuuint32_t box[3] = {16u, 32u, 1u};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    r = fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    cuuint64_t dims[4] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)planes, (cuuint64_t)batch};
    cuuint64_t strides[3] = {(cuuint64_t)s_row, (cuuint64_t)s_pl, (cuuint64_t)s_b};
    cuuint32_t box[4] = {32u, 32u, 1u, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) return false;
  if (cache) cache->maps[key] = *out;
  return true;
}

// channel-last pixel array [images][H][W][C] per plane, read in boxes of 64 channels of bx x by
// pixels (every `stride`-th one in both directions) of bi images
static mw_status get_map_conv(TcMapCache* cache, const TcOperand& op, int H, int W, int bx, int by,
                              int bi, int stride, int total_planes, CUtensorMap* out) {
  const int C = op.cols;
  auto key = std::make_tuple(op.base, op.rows, op.cols, total_planes, op.plane_stride,
                             ((int64_t)1 << 62) + (((((int64_t)W * 4096 + H) * 512 + bx) * 512 + by) * 512 + bi) * 8 + stride);
  if (cache) {
    auto it = cache->maps.find(key);
    if (it != cache->maps.end()) { *out = it->second; return MW_OK; }
  }
  auto fn = encode_fn();
  if (!fn) return MW_ERR_CUDA;
  if (((uintptr_t)op.base & 15u) || C % 64 != 0 || op.rows % (H * W) != 0) return MW_ERR_INVALID_ARG;
  const int64_t ps = total_planes > 1 ? op.plane_stride : (int64_t)op.rows * op.cols;
  if (ps % 8 != 0) return MW_ERR_INVALID_ARG;
  // a strided box spans stride * count pixels and loads every stride-th of them
  if (bx * stride > 256 || by * stride > 256 || bi > 256) return MW_ERR_UNSUPPORTED;
  const cuuint64_t images = (cuuint64_t)(op.rows / (H * W));
  const cuuint64_t pb = (cuuint64_t)C * 2;     // bytes of one pixel
  cuuint64_t dims[5] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, images, (cuuint64_t)total_planes};
  cuuint64_t strides[4] = {pb, (cuuint64_t)W * pb, (cuuint64_t)H * W * pb, (cuuint64_t)ps * 2};
  cuuint32_t box[5] = {64u, (cuuint32_t)(bx * stride), (cuuint32_t)(by * stride), (cuuint32_t)bi, 1u};
  cuuint32_t estr[5] = {1u, (cuuint32_t)stride, (cuuint32_t)stride, 1u, 1u};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(op.base), dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return MW_ERR_CUDA;
  if (cache) cache->maps[key] = *out;
  return MW_OK;
}

namespace {

uint32_t make_idesc(bool a_mn, bool b_mn, int n, int m = BM) {
  // fp32 accumulate, bf16 A and B, major-ness of A and B, N / 8, M / 16 (M = 256: both CTAs of a pair)
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// Pair form: one instruction per kept cross product (i, j), 256 rows x bn columns; the products
// of order i + j accumulate in column block i + j.  Each CTA's stage holds its half of every B
// plane, b_tile_bytes apart.  Returns the tensor-core cycles of one K block.
double build_ops_pair(TcProblem& P) {
  const int pa = P.pa, pb = P.pb, bn = P.bn;
  const int t = pa > pb ? pa : pb;
  const bool merge = t * bn > kSetCols;       // no room for a block per order: one block for all
  const uint32_t b0 = (uint32_t)pa * kATileBytes;
  bool init[4] = {false, false, false, false};
  int n = 0;
  double cycles = 0.0;
  for (int i = 0; i < pa; ++i)
    for (int j = 0; j < pb; ++j) {
      if (i + j >= t) continue;
      const int blk = merge ? 0 : i + j;
      TcOp& o = P.ops[n++];
      o.a_off16 = ((uint32_t)i * kATileBytes) >> 4;
      o.b_off16 = (b0 + (uint32_t)j * P.b_tile_bytes) >> 4;
      o.idesc = make_idesc(P.a_mn != 0, P.b_mn != 0, bn, 2 * BM);
      o.dcol = (uint16_t)(blk * bn);
      o.rot = 0;
      o.first_kbs = init[blk] ? 0u : 1u;
      init[blk] = true;
      cycles += 4.0 * std::max(bn / 2.0, 88.0);
    }
  P.nops = n;
  P.nblocks = merge ? 1 : t;
  return cycles;
}

// the instruction list of one K step: one instruction per A plane covering the B planes whose
// cross product with it is kept (i + j < max(pa, pb)); products of equal order i + j share a
// column block.  Returns the tensor-core cycles of one K block (for sorting).
double build_ops(TcProblem& P, bool rotate) {
  const int pa = P.pa, pb = P.pb, bn = P.bn;
  const int t = pa > pb ? pa : pb;
  const int lead = rotate ? 1 : 0;            // extra column block for the alternating leading term
  auto col = [&](int order) { return (order == 0 ? 0 : (order + lead)) * bn; };
  const uint32_t b0 = (uint32_t)pa * kATileBytes;
  bool init[8] = {false, false, false, false, false, false, false, false};
  int n = 0;
  double cycles = 0.0;
  auto add = [&](int i, int j0, int cnt, int rot, int first) {
    TcOp& o = P.ops[n++];
    o.a_off16 = ((uint32_t)i * kATileBytes) >> 4;
    o.b_off16 = (b0 + (uint32_t)j0 * P.b_tile_bytes) >> 4;
    o.idesc = make_idesc(P.a_mn != 0, P.b_mn != 0, cnt * bn);
    o.dcol = (uint16_t)col(i + j0);
    o.rot = (uint16_t)rot;
    o.first_kbs = (uint32_t)first;
    const double w = cnt * bn;
    cycles += 4.0 * std::max(w / 2.0, 88.0);   // an instruction takes at least 88 cycles whatever its width
  };
  for (int i = 0; i < pa; ++i) {
    int cnt = pb < t - i ? pb : t - i;
    if (cnt <= 0) continue;
    int j0 = 0;
    if (i == 0 && rotate) {
      add(0, 0, 1, bn, 2);
      init[0] = true;
      j0 = 1;
      --cnt;
      if (cnt <= 0) continue;
    }
    // blocks i+j0 .. i+j0+cnt-1: one instruction when they are all fresh or all started
    bool all_init = true, none_init = true;
    for (int b = i + j0; b < i + j0 + cnt; ++b) {
      if (init[b]) none_init = false; else all_init = false;
    }
    if (all_init || none_init) {
      add(i, j0, cnt, 0, none_init ? 1 : 0);
    } else {
      for (int b = 0; b < cnt; ++b) add(i, j0 + b, 1, 0, init[i + j0 + b] ? 0 : 1);
    }
    for (int b = i + j0; b < i + j0 + cnt; ++b) init[b] = true;
  }
  P.nops = n;
  P.nblocks = t + lead;
  return cycles;
}

}  // namespace

// fills P from d (everything but unit_begin); returns the tensor-core cycles of one unit
static mw_status setup_problem(TcMapCache* cache, const TcGemm& d, TcProblem& P, double* unit_cost,
                               double* flops, double* mma_flops, bool pair = false) {
  if (pair && !pair_capable(d)) return MW_ERR_UNSUPPORTED;
  if (d.N % 64 != 0) return MW_ERR_UNSUPPORTED;
  // a ragged K tail is zero-filled by the copies of MN-major operands (K counts their rows)
  if ((!d.A.mn_major || !d.B.mn_major) && d.K % 64 != 0) return MW_ERR_UNSUPPORTED;
  if (d.A.planes < 1 || d.A.planes > 3 || d.B.planes < 1 || d.B.planes > 3) return MW_ERR_INVALID_ARG;
  if (d.A.mn_major && (d.M % 64 != 0)) return MW_ERR_UNSUPPORTED;
  const TcConv& cv = d.conv;
  int cbx = 0, cby = 0, cbi = 0;          // pixels, rows, images of one A box
  P.conv_mode = cv.mode;
  P.c1d = 0;
  if (cv.mode != TC_CONV_NONE) {
    const int span = cv.mode == TC_CONV_PIXELS ? BM : BK;    // pixels per A box
    const int Ho = cv.Ho ? cv.Ho : cv.H, Wo = cv.Wo ? cv.Wo : cv.W;
    const int C = d.A.cols;
    if (cv.W < 1 || cv.H < 1 || Ho < 1 || Wo < 1 || cv.stride < 1 || cv.stride > 4 || C != cv.C ||
        C % 64 != 0 || cv.k < 0 || cv.k * cv.k > kTcMaxTaps || cv.ntaps < 0 || cv.ntaps > kTcMaxTaps)
      return MW_ERR_UNSUPPORTED;
    cbx = Wo < span ? Wo : span;
    if (span % cbx != 0 || Wo % cbx != 0) return MW_ERR_UNSUPPORTED;
    cby = span / cbx < Ho ? span / cbx : Ho;
    if (Ho % cby != 0) return MW_ERR_UNSUPPORTED;
    cbi = span / (cbx * cby);
    if (cbx * cby * cbi != span) return MW_ERR_UNSUPPORTED;
    P.cHo = Ho; P.cWo = Wo; P.cstride = cv.stride; P.ccb = C / 64;
    P.cbx = cbx; P.cby = cby; P.cbi = cbi;
    P.ck = cv.k; P.cpad = cv.pad; P.b_tap_rows = cv.b_tap_rows;
    if (cv.mode == TC_CONV_PIXELS) {
      int nt = 0;
      if (cv.ntaps > 0) {
        for (; nt < cv.ntaps; ++nt) { P.tdy[nt] = cv.dy[nt]; P.tdx[nt] = cv.dx[nt]; P.ttb[nt] = cv.tb[nt]; }
      } else {
        for (int tap = 0; tap < cv.k * cv.k; ++tap) {
          if (tap == cv.skip_tap) continue;
          const int j0 = tap / cv.k, j1 = tap - j0 * cv.k;
          P.tdy[nt] = (signed char)(cv.sgn * (j0 - cv.pad));
          P.tdx[nt] = (signed char)(cv.sgn * (j1 - cv.pad));
          P.ttb[nt] = (signed char)tap;
          ++nt;
        }
      }
      P.cntaps = nt;
      if (nt < 1 || d.A.mn_major || d.M % (Ho * Wo) != 0 || d.batch != 1 || d.K != nt * C)
        return MW_ERR_UNSUPPORTED;
    } else {
      P.cntaps = cv.one_d ? cv.k : cv.k * cv.k;
      P.c1d = cv.one_d;
      if (cv.k < 1 || !d.A.mn_major || !d.B.mn_major || d.M != P.cntaps * C || d.K % 64 != 0 ||
          d.split_k > 1)
        return MW_ERR_UNSUPPORTED;
    }
  }
  P.ndep = 0;
  P.done2 = -1;
  P.M = d.M; P.N = d.N; P.K = d.K;
  P.pa = d.A.planes; P.pb = d.B.planes;
  P.a_mn = d.A.mn_major ? 1 : 0;
  P.b_mn = d.B.mn_major ? 1 : 0;
  P.a_batch_planes = d.A.batch_planes ? d.A.batch_planes : d.A.planes;
  P.b_batch_planes = d.B.batch_planes ? d.B.batch_planes : d.B.planes;
  P.bn = pair ? pair_bn(P.pa, P.pb, d.N) : pick_bn(P.pa, P.pb, d.M, d.N, d.batch, d.wide_tiles != 0);
  P.num_kb = (d.K + BK - 1) / BK;
  int split = d.split_k > 1 ? d.split_k : 1;
  if (split > P.num_kb) split = P.num_kb;
  P.kb_per_split = (P.num_kb + split - 1) / split;
  split = (P.num_kb + P.kb_per_split - 1) / P.kb_per_split;
  P.split = split;
  P.bm = pair ? 2 * BM : BM;
  const int tiles_m = (d.M + P.bm - 1) / P.bm;
  P.tiles_n = (d.N + P.bn - 1) / P.bn;
  P.tiles_mn = tiles_m * P.tiles_n;
  // symmetric result (TcEpilogue::symmetric): square tiles of a square product, term planes only,
  // stored by the copy engine (checked below, once the output maps are known)
  P.sym = (d.epi.symmetric && d.epi.mode == TC_EPI_RESID && d.M == d.N && d.M % P.bm == 0 && d.N % P.bn == 0 &&
           (!pair || (P.bn == P.bm && g_bulk_epilogue)) && cv.mode == TC_CONV_NONE && split == 1 && d.batch == 1 &&
           !d.epi.out_f32 && d.epi.n_planes > 0 && d.epi.remap_s == 0 && !d.epi.ld)
              ? 1 : 0;
  if (P.sym) {
    P.tiles_mn = 0;
    for (int m = 0; m < tiles_m; ++m) P.tiles_mn += P.tiles_n - (m * P.bm) / P.bn;
  }
  const int64_t units = (int64_t)P.tiles_mn * d.batch * split;
  if (units > (1 << 30)) return MW_ERR_UNSUPPORTED;
  P.unit_count = (int)units;
  const int b_cols = pair ? P.bn / 2 : P.bn;     // columns of the B tile one CTA stages
  P.b_tile_bytes = (uint32_t)b_cols * BK * 2;
  P.tx_bytes = (uint32_t)P.pa * kATileBytes + (uint32_t)P.pb * P.b_tile_bytes;
  P.a_desc_base = (P.a_mn ? (8192u >> 4) : 1u) << 16;
  P.b_desc_base = (P.b_mn ? (8192u >> 4) : 1u) << 16;
  const int t = P.pa > P.pb ? P.pa : P.pb;
  // fp32-accurate products alternate the leading block (needs two K blocks per unit)
  const bool rotate = t == 3 && P.pa == 3 && P.pb == 3 && P.kb_per_split >= 2 &&
                      (P.num_kb - (split - 1) * P.kb_per_split) >= 2;
  const double kb_cycles = pair ? build_ops_pair(P) : build_ops(P, rotate);
  *unit_cost = kb_cycles * P.kb_per_split;
  P.epi = d.epi;
  // bulk stores for outputs that are plain [M][N] arrays (no row scatter, no sub-sampling)
  P.out_tma = 0;
  if (g_bulk_epilogue && d.epi.remap_s == 0) {
    const TcEpilogue& e = d.epi;
    const int64_t ldo = e.ld ? e.ld : (int64_t)d.N;
    if (e.out_f32 && get_out_map(cache, e.out_f32, true, d.M, d.N, ldo, 1, 0, d.batch, e.bs_f32, &P.tmO))
      P.out_tma |= 1;
    if (e.n_planes && get_out_map(cache, e.planes, false, d.M, d.N, ldo, e.n_planes, e.plane_stride, d.batch,
                                  e.bs_planes, &P.tmP))
      P.out_tma |= 2;
    if (e.n_planes2 && !e.compact2 && !e.sub2_s &&
        get_out_map(cache, e.planes2, false, d.M, d.N, ldo, e.n_planes2, e.plane_stride2, d.batch, e.bs_planes2,
                    &P.tmP2))
      P.out_tma |= 4;
  }
  if (P.sym && pair && !(P.out_tma & 2)) {     // pair form without a copy-engine path for the planes: the full product
    P.sym = 0;
    P.tiles_mn = tiles_m * P.tiles_n;
    P.unit_count = P.tiles_mn * d.batch * split;
  }
  P.epi.symmetric = P.sym;
  P.split_partials = nullptr;
  P.split_counters = nullptr;
  if (split > 1) {
    if (!d.split_scratch || ((uintptr_t)d.split_scratch & 255u)) return MW_ERR_WORKSPACE;
    const size_t tiles = (size_t)P.tiles_mn * d.batch;
    if (tiles * kEpiWarps * sizeof(unsigned) > kTcSplitCounterBytes) return MW_ERR_UNSUPPORTED;
    P.split_counters = static_cast<unsigned int*>(d.split_scratch);
    P.split_partials = reinterpret_cast<float*>(static_cast<char*>(d.split_scratch) + kTcSplitCounterBytes);
  }
  const int a_total = d.batch > 1 ? (d.batch - 1) * P.a_batch_planes + d.A.planes : d.A.planes;
  const int b_total = d.batch > 1 ? (d.batch - 1) * P.b_batch_planes + d.B.planes : d.B.planes;
  if (cv.mode == TC_CONV_PIXELS) {
    MW_TRY(get_map_conv(cache, d.A, cv.H, cv.W, cbx, cby, cbi, cv.stride, a_total, &P.tmA));
    MW_TRY(get_map(cache, d.B, d.B.mn_major ? 64 : P.bn, b_total, &P.tmB));
  } else if (cv.mode == TC_CONV_WGRAD) {
    MW_TRY(get_map_conv(cache, d.A, cv.H, cv.W, cbx, cby, cbi, cv.stride, d.A.planes, &P.tmA));
    MW_TRY(get_map(cache, d.B, 64, d.B.planes, &P.tmB));
  } else {
    // one box per operand and K block, spanning its planes (and, MN-major, its column groups)
    if (d.A.mn_major) MW_TRY(get_map_mn(cache, d.A, BM / 64, a_total, P.pa, &P.tmA));
    else MW_TRY(get_map(cache, d.A, BM, a_total, &P.tmA, P.pa));
    if (d.B.mn_major) MW_TRY(get_map_mn(cache, d.B, b_cols / 64, b_total, P.pb, &P.tmB));
    else MW_TRY(get_map(cache, d.B, b_cols, b_total, &P.tmB, P.pb));
  }
  int np = 0;
  for (int a = 0; a < P.pa; ++a)
    for (int b = 0; b < P.pb; ++b)
      if (a + b < t) ++np;
  *flops += 2.0 * d.M * d.N * d.K * d.batch;
  // (a symmetric product executes only its tiles on and above the diagonal)
  const double done_share = P.sym ? (double)P.tiles_mn / ((double)tiles_m * P.tiles_n) : 1.0;
  *mma_flops += 2.0 * d.M * d.N * d.K * np * d.batch * done_share;
  return MW_OK;
}

static int stages_for(uint32_t stage_bytes) {
  const uint32_t budget = 227u * 1024u - 8192u;   // static shared memory + alignment slack
  int stages = (int)(budget / stage_bytes);
  return stages > kMaxStages ? kMaxStages : stages;
}

constexpr int kMaxDynamicSmem = 227 * 1024 - 6144;

// the epilogue's transposition buffers go behind the stages when the ring leaves room for them
static uint32_t epi_stage_offset(int stages, uint32_t stage_bytes, size_t* smem) {
  const size_t need = (size_t)kEpiWarps * kEpiStageBytes;
  if (*smem + need > (size_t)kMaxDynamicSmem) return 0;
  const uint32_t off = (uint32_t)stages * stage_bytes;
  *smem += need;
  return off;
}

// the opt-in to large dynamic shared memory belongs to the device: once per device and kernel
static mw_status ensure_kernel_attr() {
  static bool attr_set[kMaxDevices] = {};
  const int dev = current_device();
  if (!attr_set[dev]) {
    const int bytes = kMaxDynamicSmem;
    MW_CUDA_OK(cudaFuncSetAttribute(tc_group_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    MW_CUDA_OK(cudaFuncSetAttribute(tc_group_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    MW_CUDA_OK(cudaFuncSetAttribute(tc_group_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    MW_CUDA_OK(cudaFuncSetAttribute(tc_group_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    attr_set[dev] = true;
  }
  return MW_OK;
}

// bound of the device-side waits of the launches that follow (test hook; 0 restores the default)
static uint64_t g_wait_limit_ns = kDefaultWaitLimitNs;
// 0: program launches go without the cooperative attribute (profilers that cannot replay a
// cooperative launch of clusters; residency is then the caller's business).  Default 1.
static int g_cooperative = 1;

// CTA pairs that can be resident at once (cached per device); 0 when clusters cannot be launched
static int max_pairs(size_t smem) {
  static int n[kMaxDevices] = {};
  const int dev = current_device();
  if (n[dev] == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)sm_count());
    cfg.blockDim = dim3(kThreadsTc);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int c = 0;
    if (cudaOccupancyMaxActiveClusters(&c, tc_group_kernel<true, true>, &cfg) != cudaSuccess || c < 1) {
      cudaGetLastError();
      c = -1;
    }
    if (c > sm_count() / 2) c = sm_count() / 2;
    n[dev] = c;
  }
  return n[dev] > 0 ? n[dev] : 0;
}

// launch of one of the four kernel forms; `coop`: every CTA must be resident (program launches)
static cudaError_t launch_kernel(bool program, bool pair, int grid, size_t smem, cudaStream_t s,
                                 const TcGroupParams& prm) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreadsTc);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (program) {
    attr[na].id = cudaLaunchAttributeCooperative;
    attr[na].val.cooperative = g_cooperative;
  } else {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
  }
  ++na;
  if (pair) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 2;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  if (program) return pair ? cudaLaunchKernelEx(&cfg, tc_group_kernel<true, true>, prm)
                           : cudaLaunchKernelEx(&cfg, tc_group_kernel<true, false>, prm);
  return pair ? cudaLaunchKernelEx(&cfg, tc_group_kernel<false, true>, prm)
              : cudaLaunchKernelEx(&cfg, tc_group_kernel<false, false>, prm);
}

mw_status tc_gemm_group(TcMapCache* cache, const TcGemm* g, int count, DeviceStatus* st,
                        cudaStream_t s) {
  if (count < 1 || count > kTcMaxGroup) return MW_ERR_INVALID_ARG;
  MW_TRY(ensure_kernel_attr());
  // the pair form when every product of the launch qualifies
  bool pair = g_pair_mode != 0 && max_pairs(200 * 1024) > 0;
  for (int i = 0; i < count && pair; ++i) {
    const TcGemm& d = g[i];
    if (d.M <= 0 || d.N <= 0 || d.K <= 0 || d.batch <= 0) continue;
    pair = pair_capable(d);
  }
  static thread_local TcGroupParams prm;
  prm.nprob = 0;
  prm.st = st;
  prm.table = nullptr;
  prm.done = nullptr;
  prm.wait_limit_ns = g_wait_limit_ns;
  double cost[kTcMaxGroup];
  double flops = 0.0, mma_flops = 0.0;
  uint32_t stage_bytes = 0;
  for (int i = 0; i < count; ++i) {
    const TcGemm& d = g[i];
    if (d.M <= 0 || d.N <= 0 || d.K <= 0 || d.batch <= 0) continue;
    TcProblem& P = prm.prob[prm.nprob];
    MW_TRY(setup_problem(cache, d, P, &cost[prm.nprob], &flops, &mma_flops, pair));
    if (P.tx_bytes > stage_bytes) stage_bytes = P.tx_bytes;
    ++prm.nprob;
  }
  if (prm.nprob == 0) return MW_OK;
  // costliest units first
  for (int i = 1; i < prm.nprob; ++i)
    for (int j = i; j > 0 && cost[j] > cost[j - 1]; --j) {
      std::swap(cost[j], cost[j - 1]);
      std::swap(prm.prob[j], prm.prob[j - 1]);
    }
  int total = 0;
  for (int i = 0; i < prm.nprob; ++i) {
    prm.prob[i].unit_begin = total;
    total += prm.prob[i].unit_count;
  }
  prm.total_units = total;
  prm.stage_bytes = stage_bytes;
  const int stages = stages_for(stage_bytes);
  if (stages < 2) return MW_ERR_UNSUPPORTED;
  prm.stages = stages;
  size_t smem = (size_t)stages * stage_bytes + 1024;
  prm.epi_stage_off = epi_stage_offset(stages, stage_bytes, &smem);
  // a symmetric product mirrors its tiles through the epilogue's staging buffers
  for (int i = 0; i < prm.nprob; ++i)
    if (pair && prm.prob[i].sym && !prm.epi_stage_off) return MW_ERR_UNSUPPORTED;
  const bool prof = g_prof.on;
  if (prof) {
    cudaEventRecord(prof_event(), s);
    g_prof.flops += flops;
    g_prof.mma_flops += mma_flops;
  }
  // persistent grid: one CTA (or one pair of CTAs) per unit, at most what the device holds at once
  const int slots = pair ? max_pairs(smem) : sm_count();
  const int grid = (total < slots ? total : slots) * (pair ? 2 : 1);
  const cudaError_t le = launch_kernel(false, pair, grid, smem, s, prm);
  ++g_launch_count;
  const mw_status rc = le == cudaSuccess ? MW_OK : MW_ERR_CUDA;
  if (prof) cudaEventRecord(prof_event(), s);
  return rc;
}

// ---- program launches ----------------------------------------------------------------------
struct TcProgram {
  std::vector<TcProblem> table;
  uint32_t stage_bytes = 0;
  int total_units = 0;
  double flops = 0.0, mma_flops = 0.0;
  void* table_dev = nullptr;
  unsigned int* done_dev = nullptr;
  bool uploaded = false;
  bool pair = false;          // every product in the pair form (clusters of two CTAs)
  std::vector<unsigned> target;   // arrivals that complete each table entry (product or group)
  std::vector<int> sched;         // units of every CTA (pair), see balance_units
  int sched_slots = 0, sched_len = 0;
  bool balance = false;           // hand the units out by the schedule instead of round-robin
};

TcProgram* tc_program_create() { return new TcProgram(); }
void tc_program_destroy(TcProgram* p) { delete p; }

void tc_program_begin(TcProgram* pr, void* table_dev, unsigned int* done_dev, bool pair) {
  pr->pair = pair && g_pair_mode != 0 && ensure_kernel_attr() == MW_OK && max_pairs(200 * 1024) > 0;
  pr->table.clear();
  pr->target.clear();
  pr->stage_bytes = 0;
  pr->total_units = 0;
  pr->flops = pr->mma_flops = 0.0;
  pr->table_dev = table_dev;
  pr->done_dev = done_dev;
  pr->uploaded = false;
  pr->sched.clear();
  pr->sched_slots = pr->sched_len = 0;
  pr->balance = false;
}

void tc_program_balance(TcProgram* pr, bool on) { pr->balance = on; }

int tc_program_add(TcProgram* pr, TcMapCache* cache, const TcGemm& d, const int* deps, int ndep,
                   mw_status* status, int group) {
  *status = MW_OK;
  if ((int)pr->table.size() >= kMaxProgram || ndep > kTcMaxDeps) { *status = MW_ERR_UNSUPPORTED; return -1; }
  pr->table.emplace_back();
  TcProblem& P = pr->table.back();
  double cost = 0.0;
  *status = setup_problem(cache, d, P, &cost, &pr->flops, &pr->mma_flops, pr->pair);
  if (*status != MW_OK) { pr->table.pop_back(); return -1; }
  P.unit_begin = pr->total_units;
  pr->total_units += P.unit_count;
  if (P.tx_bytes > pr->stage_bytes) pr->stage_bytes = P.tx_bytes;
  const int self = (int)pr->table.size() - 1;
  // one arrival per epilogue warp and tile (of both CTAs in the pair form)
  const unsigned arrivals = (unsigned)kEpiWarps * (pr->pair ? 2u : 1u) * (unsigned)(P.unit_count / P.split);
  pr->target.push_back(arrivals);
  if (group >= 0) {
    if (group >= self || pr->table[group].unit_count != 0) { *status = MW_ERR_INVALID_ARG; return -1; }
    P.done2 = group;
    pr->target[group] += arrivals;
  }
  for (int i = 0; i < ndep; ++i) {
    const int q = deps[i];
    if (q < 0) continue;
    if (q >= self) { *status = MW_ERR_INVALID_ARG; return -1; }   // only earlier entries
    P.dep[P.ndep] = q;
    P.dep_target[P.ndep] = 0;     // filled in at launch, when the groups are complete
    ++P.ndep;
  }
  return self;
}

int tc_program_add_group(TcProgram* pr);

// test hook: an entry that nothing ever completes (a group without members that claims one arrival)
int tc_program_add_unreachable(TcProgram* pr) {
  const int q = tc_program_add_group(pr);
  if (q >= 0) pr->target[(size_t)q] = 1u;
  return q;
}

int tc_program_add_group(TcProgram* pr) {
  if ((int)pr->table.size() >= kMaxProgram) return -1;
  pr->table.emplace_back();
  TcProblem& P = pr->table.back();
  P = TcProblem();
  P.unit_begin = pr->total_units;
  P.unit_count = 0;
  P.split = 1;
  P.tiles_mn = 1;
  P.tiles_n = 1;
  P.done2 = -1;
  pr->target.push_back(0u);
  return (int)pr->table.size() - 1;
}

// room for the unit schedule behind the table
constexpr size_t kSchedBytes = 256 * 1024;
size_t tc_program_table_bytes(int products) { return (size_t)products * sizeof(TcProblem) + kSchedBytes + 256; }

// Rough length of one unit in SM cycles: its tcgen05 instructions (128 cycles each at 256
// accumulator columns, a floor of 88 below) or its epilogue (fp32 tiles cost about twice the
// bf16 planes), whichever is longer.
static double unit_cycles(const TcProblem& P) {
  const int nkb = P.split > 1 ? P.kb_per_split : P.num_kb;
  const double main_loop = (double)nkb * P.nops * (BK / 16) * (P.bn >= 256 ? 128.0 : 88.0);
  const double per_elem = P.epi.out_f32 ? 0.25 : 0.12;
  const double epilogue = 3000.0 + per_elem * 128.0 * P.bn;
  return (main_loop > epilogue ? main_loop : epilogue) + 1000.0;
}

// Units of a program launch differ in length (a vijp tile of three-term operands against a
// weight vjp tile), and whatever waits for a product waits for its slowest tile.  For programs
// that ask for it (tc_program_balance: the chained sweep on single CTAs, where it measured 15 %
// faster; on CTA pairs and in the Newton-Schulz programs it measured slower than round-robin)
// the schedule gives each unit, in list order, to the CTA (pair) with the least work so far; every
// CTA still meets its units in list order, which is all the waiting needs (a unit's operands come
// from earlier units, each of which is the oldest unfinished one of some CTA or already done).
static void balance_units(TcProgram* pr, int slots) {
  std::vector<double> load((size_t)slots, 0.0);
  std::vector<std::vector<int>> mine((size_t)slots);
  for (const TcProblem& P : pr->table) {
    if (P.unit_count <= 0) continue;
    const double cyc = unit_cycles(P);
    for (int i = 0; i < P.unit_count; ++i) {
      int best = 0;
      for (int g = 1; g < slots; ++g)
        if (load[(size_t)g] < load[(size_t)best]) best = g;
      load[(size_t)best] += cyc;
      mine[(size_t)best].push_back(P.unit_begin + i);
    }
  }
  size_t len = 0;
  for (const auto& m : mine) len = m.size() > len ? m.size() : len;
  pr->sched_len = (int)len + 1;
  pr->sched_slots = slots;
  pr->sched.assign((size_t)slots * pr->sched_len, -1);
  for (int g = 0; g < slots; ++g)
    for (size_t k = 0; k < mine[(size_t)g].size(); ++k) pr->sched[(size_t)g * pr->sched_len + k] = mine[(size_t)g][k];
}

mw_status tc_program_launch(TcProgram* pr, DeviceStatus* st, cudaStream_t s) {
  const int nprob = (int)pr->table.size();
  if (nprob == 0) return MW_OK;
  if (!pr->table_dev || !pr->done_dev || ((uintptr_t)pr->table_dev & 63u)) return MW_ERR_WORKSPACE;
  for (TcProblem& P : pr->table)
    for (int i = 0; i < P.ndep; ++i) P.dep_target[i] = pr->target[P.dep[i]];
  // the table travels with every launch: the caller's workspace is only promised to keep its
  // contents between the calls of one step
  MW_CUDA_OK(cudaMemcpyAsync(pr->table_dev, pr->table.data(), nprob * sizeof(TcProblem),
                             cudaMemcpyHostToDevice, s));
  MW_CUDA_OK(cudaMemsetAsync(pr->done_dev, 0, sizeof(unsigned int) * nprob, s));
  static thread_local TcGroupParams prm;
  prm.nprob = nprob;
  prm.st = st;
  prm.table = static_cast<const TcProblem*>(pr->table_dev);
  prm.done = pr->done_dev;
  prm.total_units = pr->total_units;
  prm.stage_bytes = pr->stage_bytes;
  prm.wait_limit_ns = g_wait_limit_ns;
  const int stages = stages_for(pr->stage_bytes);
  if (stages < 2) return MW_ERR_UNSUPPORTED;
  prm.stages = stages;
  size_t smem = (size_t)stages * pr->stage_bytes + 1024;
  prm.epi_stage_off = epi_stage_offset(stages, pr->stage_bytes, &smem);
  if (pr->pair && !prm.epi_stage_off)
    for (const TcProblem& P : pr->table)
      if (P.sym) return MW_ERR_UNSUPPORTED;   // (mirrors its tiles through the staging buffers)
  MW_TRY(ensure_kernel_attr());
  const bool prof = g_prof.on;
  if (prof) {
    cudaEventRecord(prof_event(), s);
    g_prof.flops += pr->flops;
    g_prof.mma_flops += pr->mma_flops;
  }
  // products wait for one another inside the launch: every CTA must be resident (cooperative launch)
  const int slots = pr->pair ? max_pairs(smem) : sm_count();
  if (slots < 1) return MW_ERR_CUDA;
  const int used = pr->total_units < slots ? pr->total_units : slots;
  const int grid = used * (pr->pair ? 2 : 1);
  prm.sched = nullptr;
  prm.sched_len = 0;
  if (pr->balance && pr->total_units > used) {
    if (pr->sched_slots != used) balance_units(pr, used);
    const size_t bytes = pr->sched.size() * sizeof(int);
    if (bytes <= kSchedBytes) {
      char* dst = static_cast<char*>(pr->table_dev) + (((size_t)nprob * sizeof(TcProblem) + 255) & ~(size_t)255);
      MW_CUDA_OK(cudaMemcpyAsync(dst, pr->sched.data(), bytes, cudaMemcpyHostToDevice, s));
      prm.sched = reinterpret_cast<const int*>(dst);
      prm.sched_len = pr->sched_len;
    }
  }
  const cudaError_t e = launch_kernel(true, pr->pair, grid, smem, s, prm);
  ++g_launch_count;
  if (prof) cudaEventRecord(prof_event(), s);
  return e == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}

bool tc_pair_ok(int a_planes, int b_planes, int M, int N) {
  TcGemm d;
  d.A.planes = a_planes; d.B.planes = b_planes; d.M = M; d.N = N; d.K = 64;
  return g_pair_mode != 0 && pair_capable(d);
}
int tc_set_bulk_epilogue(int mode) {
  const int old = g_bulk_epilogue;
  g_bulk_epilogue = mode != 0;
  return old;
}
int tc_set_cooperative(int mode) {
  const int old = g_cooperative;
  g_cooperative = mode != 0;
  return old;
}
int tc_set_merge_orders(int mode) {
  const int old = g_merge_orders;
  g_merge_orders = mode != 0;
  return old;
}
int tc_set_pair_mode(int mode) {
  const int old = g_pair_mode;
  g_pair_mode = mode != 0;
  return old;
}
void tc_set_wait_limit_ns(uint64_t ns) { g_wait_limit_ns = ns ? ns : kDefaultWaitLimitNs; }
size_t tc_sumsq_slots(int a_planes, int b_planes, int M, int N, bool pair) {
  const int bn = pair ? pair_bn(a_planes, b_planes, N) : pick_bn(a_planes, b_planes, M, N, 1);
  return (size_t)((M + BM - 1) / BM) * ((N + bn - 1) / bn) * kEpiWarps;
}

mw_status tc_gemm(TcMapCache* cache, const TcOperand& A, const TcOperand& B, int M, int N, int K,
                  const TcEpilogue& epi, DeviceStatus* st, cudaStream_t s, int batch) {
  TcGemm g;
  g.A = A; g.B = B; g.M = M; g.N = N; g.K = K; g.batch = batch; g.epi = epi;
  return tc_gemm_group(cache, &g, 1, st, s);
}

// ---------------------------------------------------------------------------------------
// fp32 -> bf16 term planes
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
split_planes_batched_kernel(const float* __restrict__ in, int64_t n4, int64_t in_stride,
                            __nv_bfloat16* __restrict__ out, int planes, int64_t plane_stride,
                            int64_t out_stride) {
  const float* src = in + (int64_t)blockIdx.y * in_stride;
  __nv_bfloat16* dst = out + (int64_t)blockIdx.y * out_stride;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n4; i += (int64_t)gridDim.x * 256) {
    float4 v = reinterpret_cast<const float4*>(src)[i];
    float r[4] = {v.x, v.y, v.z, v.w};
    for (int p = 0; p < planes; ++p) {
      __nv_bfloat16 b[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b[j] = __float2bfloat16_rn(r[j]);
        r[j] -= __bfloat162float(b[j]);
      }
      uint2 pk;
      pk.x = (uint32_t)__bfloat16_as_ushort(b[0]) | ((uint32_t)__bfloat16_as_ushort(b[1]) << 16);
      pk.y = (uint32_t)__bfloat16_as_ushort(b[2]) | ((uint32_t)__bfloat16_as_ushort(b[3]) << 16);
      reinterpret_cast<uint2*>(dst + (int64_t)p * plane_stride)[i] = pk;
    }
  }
}

mw_status split_planes_batched(const float* in, int64_t n, int batch, int64_t in_stride,
                               __nv_bfloat16* out, int planes, int64_t plane_stride,
                               int64_t out_stride, cudaStream_t s) {
  if (n == 0 || batch == 0) return MW_OK;
  if (n % 4 != 0 || plane_stride % 4 != 0 || in_stride % 4 != 0 || out_stride % 4 != 0)
    return MW_ERR_UNSUPPORTED;
  int64_t bx = (n / 4 + 255) / 256;
  const int64_t cap = ((int64_t)sm_count() * 8 + batch - 1) / batch;
  if (bx > cap) bx = cap < 1 ? 1 : cap;
  split_planes_batched_kernel<<<dim3((unsigned)bx, (unsigned)batch), 256, 0, s>>>(
      in, n / 4, in_stride, out, planes, plane_stride, out_stride);
  return launch_ok();
}

mw_status split_planes(const float* in, int64_t n, __nv_bfloat16* out, int planes,
                       int64_t plane_stride, cudaStream_t s) {
  return split_planes_batched(in, n, 1, 0, out, planes, plane_stride, 0, s);
}

}  // namespace mw

// ---------------------------------------------------------------------------------------
// C ABI: the product, exposed for unit parity tests
// ---------------------------------------------------------------------------------------
extern "C" mw_status mw_gemm_split_bf16(const float* A, int32_t a_mn, const float* B, int32_t b_mn,
                                        float* D, int32_t M, int32_t N, int32_t K, int32_t terms,
                                        void* scratch, size_t scratch_bytes, void* stream) {
  using namespace mw;
  if (!A || !B || !D || !scratch) return MW_ERR_INVALID_ARG;
  if (terms < 1 || terms > 3 || M < 1 || N < 1 || K < 1) return MW_ERR_INVALID_ARG;
  if (M % 64 || N % 64 || K % 64) return MW_ERR_UNSUPPORTED;
  const size_t ea = (size_t)M * K, eb = (size_t)N * K;
  const size_t need = 256 + 2 * (size_t)terms * (ea + eb) + 512;
  if (((uintptr_t)scratch & 255u) || scratch_bytes < need) return MW_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  DeviceStatus* st = reinterpret_cast<DeviceStatus*>(scratch);
  MW_CUDA_OK(cudaMemsetAsync(st, 0, 256, s));
  __nv_bfloat16* pa = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(scratch) + 256);
  __nv_bfloat16* pb = pa + align_up((size_t)terms * ea, 128);
  MW_TRY(split_planes(A, (int64_t)ea, pa, terms, (int64_t)ea, s));
  MW_TRY(split_planes(B, (int64_t)eb, pb, terms, (int64_t)eb, s));
  TcOperand oa, ob;
  oa.base = pa; oa.planes = terms; oa.plane_stride = (int64_t)ea; oa.mn_major = a_mn != 0;
  oa.rows = a_mn ? K : M; oa.cols = a_mn ? M : K;
  ob.base = pb; ob.planes = terms; ob.plane_stride = (int64_t)eb; ob.mn_major = b_mn != 0;
  ob.rows = b_mn ? K : N; ob.cols = b_mn ? N : K;
  TcEpilogue e;
  e.mode = TC_EPI_PLAIN;
  e.out_f32 = D;
  MW_TRY(tc_gemm(nullptr, oa, ob, M, N, K, e, st, s));
  // surface a device-side timeout synchronously for this test entry point
  DeviceStatus host;
  MW_CUDA_OK(cudaMemcpyAsync(&host, st, sizeof(host), cudaMemcpyDeviceToHost, s));
  MW_CUDA_OK(cudaStreamSynchronize(s));
  return host.code == 0 ? MW_OK : (mw_status)host.code;
}

// ---------------------------------------------------------------------------------------
// Self-test of the bounded device-side waits
// ---------------------------------------------------------------------------------------
extern "C" mw_status mw_selftest_bounded_wait(void* scratch, size_t scratch_bytes, uint32_t limit_ms,
                                              int32_t* timed_out_status, void* stream) {
  using namespace mw;
  if (!scratch || !timed_out_status || limit_ms < 1 || limit_ms > 1000) return MW_ERR_INVALID_ARG;
  const int M = 128, N = 64, K = 128;
  const size_t table_off = 256, done_off = table_off + tc_program_table_bytes(4), op_off = align_up(done_off + 64, 256);
  const size_t need = op_off + 2 * (size_t)(M * K + N * K) + 4 * (size_t)M * N + 1024;
  if (((uintptr_t)scratch & 255u) || scratch_bytes < need) return MW_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  char* base = static_cast<char*>(scratch);
  DeviceStatus* st = reinterpret_cast<DeviceStatus*>(base);
  MW_CUDA_OK(cudaMemsetAsync(base, 0, need, s));        // status, counters, zero operands
  __nv_bfloat16* A = reinterpret_cast<__nv_bfloat16*>(base + op_off);
  __nv_bfloat16* B = A + (size_t)M * K;
  float* D = reinterpret_cast<float*>(B + (size_t)N * K);
  TcProgram* pr = tc_program_create();
  tc_program_begin(pr, base + table_off, reinterpret_cast<unsigned int*>(base + done_off), false);
  TcGemm g;
  g.A.base = A; g.A.rows = M; g.A.cols = K; g.A.planes = 1; g.A.plane_stride = (int64_t)M * K;
  g.B.base = B; g.B.rows = N; g.B.cols = K; g.B.planes = 1; g.B.plane_stride = (int64_t)N * K;
  g.M = M; g.N = N; g.K = K;
  g.epi.mode = TC_EPI_PLAIN;
  g.epi.out_f32 = D;
  mw_status rc = MW_OK;
  // a product that waits for an entry nothing will ever complete: its copy-issuing lane gives up
  // after the limit, records the timeout and raises the CTA's abort flag; the issuing lane and the
  // epilogue warps, waiting for data that will not come, see the flag and leave; tensor memory is
  // released and the kernel ends
  const int never = tc_program_add_unreachable(pr);
  const int deps[1] = {never};
  if (never < 0 || tc_program_add(pr, nullptr, g, deps, 1, &rc) < 0) {
    tc_program_destroy(pr);
    return rc != MW_OK ? rc : MW_ERR_UNSUPPORTED;
  }
  tc_set_wait_limit_ns((uint64_t)limit_ms * 1000000ull);
  rc = tc_program_launch(pr, st, s);
  tc_set_wait_limit_ns(0);
  tc_program_destroy(pr);
  if (rc != MW_OK) return rc;
  DeviceStatus host;
  MW_CUDA_OK(cudaMemcpyAsync(&host, st, sizeof(host), cudaMemcpyDeviceToHost, s));
  MW_CUDA_OK(cudaStreamSynchronize(s));
  *timed_out_status = (int32_t)host.code;
  MW_CUDA_OK(cudaMemsetAsync(st, 0, 256, s));
  return MW_OK;
}

// ---------------------------------------------------------------------------------------
// The same product for callers that cannot hand over scratch memory
// ---------------------------------------------------------------------------------------
namespace {

// Scratch of mw_gemm_split_bf16_static: the status block and the bf16 term planes of both
// operands.  One copy per GPU that loads the library, held until the process exits.
constexpr size_t kStaticScratchBytes = MW_GEMM_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kStaticMaxDevices = 64;
void* g_static_scratch_ptr[kStaticMaxDevices] = {};   // device address of the array, per device

}  // namespace

extern "C" mw_status mw_gemm_split_bf16_static(const float* A, int32_t a_mn, const float* B,
                                               int32_t b_mn, float* D, int32_t M, int32_t N,
                                               int32_t K, int32_t terms, void* stream) {
  using namespace mw;
  if (!A || !B || !D) return MW_ERR_INVALID_ARG;
  if (terms < 1 || terms > 3 || M < 1 || N < 1 || K < 1) return MW_ERR_INVALID_ARG;
  if (M % 64 || N % 64 || K % 64) return MW_ERR_UNSUPPORTED;
  const size_t ea = (size_t)M * K, eb = (size_t)N * K;
  const size_t need = 256 + 2 * (align_up((size_t)terms * ea, 128) + (size_t)terms * eb);
  if (need > kStaticScratchBytes) return MW_ERR_WORKSPACE;   // beyond the built-in scratch
  int dev = -1;
  MW_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kStaticMaxDevices) return MW_ERR_UNSUPPORTED;
  if (!g_static_scratch_ptr[dev]) {
    // In host code the array's name stands for the symbol, not for device memory: ask the
    // runtime for the address on the current device, once.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return MW_ERR_CUDA;
    g_static_scratch_ptr[dev] = p;
  }
  char* scratch = static_cast<char*>(g_static_scratch_ptr[dev]);
  cudaStream_t s = (cudaStream_t)stream;
  // the array keeps whatever the last call left: the status block has to start at zero, the
  // planes are overwritten in full before they are read
  DeviceStatus* st = reinterpret_cast<DeviceStatus*>(scratch);
  MW_CUDA_OK(cudaMemsetAsync(st, 0, 256, s));
  __nv_bfloat16* pa = reinterpret_cast<__nv_bfloat16*>(scratch + 256);
  __nv_bfloat16* pb = pa + align_up((size_t)terms * ea, 128);
  MW_TRY(split_planes(A, (int64_t)ea, pa, terms, (int64_t)ea, s));
  MW_TRY(split_planes(B, (int64_t)eb, pb, terms, (int64_t)eb, s));
  TcOperand oa, ob;
  oa.base = pa; oa.planes = terms; oa.plane_stride = (int64_t)ea; oa.mn_major = a_mn != 0;
  oa.rows = a_mn ? K : M; oa.cols = a_mn ? M : K;
  ob.base = pb; ob.planes = terms; ob.plane_stride = (int64_t)eb; ob.mn_major = b_mn != 0;
  ob.rows = b_mn ? K : N; ob.cols = b_mn ? N : K;
  TcEpilogue e;
  e.mode = TC_EPI_PLAIN;
  e.out_f32 = D;
  MW_TRY(tc_gemm(nullptr, oa, ob, M, N, K, e, st, s));
  DeviceStatus host;
  MW_CUDA_OK(cudaMemcpyAsync(&host, st, sizeof(host), cudaMemcpyDeviceToHost, s));
  MW_CUDA_OK(cudaStreamSynchronize(s));
  return host.code == 0 ? MW_OK : (mw_status)host.code;
}
