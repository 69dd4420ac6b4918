// Quantized GEMM of a configuration evaluation: int8 x int8 -> int32 (tcgen05 kind::i8) and
// bf16 x bf16 -> fp32 (kind::f16) for 16-bit layers, with the dequantize / shortcut /
// activation / re-quantize epilogue fused in (Eq. 1's rescale 2^-(b-1)*gamma for both operands;
// the "Evaluate f(x, w)" step of Algorithms 1 and 2).
//
// Structure (one persistent CTA per SM, 576 threads):
//   warp 0      TMA producer: 128-byte-swizzled K-major tiles of A [128 x 128 B] and
//               B [BN x 128 B] into a ring of shared-memory stages (mbarrier full/empty).
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M=128, N=BN, K=32 B per instruction)
//               from shared-memory descriptors into one of two TMEM accumulator buffers
//               (2 x 256 columns), and commits stage-release / accumulator-ready barriers.
//   warps 2..17 epilogue: tcgen05.ld of the accumulator (one row per thread, 16 or 32 columns per
//               load), rescale, shortcut add, activation, stores of fp32 and/or the consumer's
//               int8 / bf16 codes through shared-memory staging and TMA stores; overlaps the next
//               tile's main loop.
//   warps 18,19 (convolution launches only, 640 threads) gather the A tile of an implicit-GEMM
//               convolution from the NHWC codes of the layer's input with cp.async.
//   warps 18,19 (chained launches only, 640 threads) publish finished tiles (18) and clear tiles
//               whose input rows are complete (19): a chain runs up to 16 consecutive GEMMs of a
//               forward pass as one cooperative launch (see the kernel).
// Every wait (mbarrier, counter in shared or global memory) is bounded: after ~2 s it sets the
// context's error word and the CTA leaves through the normal teardown (TMEM is freed).
#include <cuda.h>

#include <cstring>
#include <mutex>
#include <new>
#include <unordered_map>

#include "common.cuh"

namespace qcfg {

namespace {

constexpr int BM = 128;               // rows per tile (UMMA M, cta_group::1)
constexpr int kStageKBytes = 128;     // bytes of K per stage row = one 128B swizzle atom
constexpr int kUmmaKBytes = 32;       // bytes of K per tcgen05.mma
constexpr int kEpiWarps = 16;
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;
constexpr int kGatherWarps = 2;       // convolution launches only: build the A tile from the NHWC source
constexpr int kGemmThreadsConv = kGemmThreads + 32 * kGatherWarps;
constexpr int kGatherDepth = 2;       // k-blocks a gather warp keeps in flight
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;         // columns per accumulator buffer
constexpr int kMaxStages = 8;
constexpr int kSmemHeader = 1024;     // barriers and bookkeeping
constexpr int kCsBytes = kEpiWarps * 64 * 4;   // per epilogue warp: rescale factors of its 64 columns
constexpr int kSmemMax = 232448;      // 227 KB
constexpr uint64_t kWaitLimitNs = 2000000000ull;

constexpr int kNumOuts = 2 + kMaxSlots;   // raw accumulators, fp32 output, consumer code slots

struct OutDesc {
  int32_t kind;       // 0 none, 1 int8 codes, 2 bf16 codes, 3 fp32, 4 int32
  int32_t tma;        // 1: staged through shared memory and written by a TMA store
  void* ptr;
  int64_t ld;         // elements
  float inv_scale, qmax;
};
// One launch runs up to kMaxGroups GEMMs of equal m, k, operand type and tile shape ("groups":
// layers that are ready at the same time, e.g. the three projections reading one input).  Their
// column tiles are numbered one after the other, so the persistent CTAs work through all of them
// and only the first tile's main loop and the last tile's epilogue stay unoverlapped.
constexpr int kMaxGroups = 3;
// Tensor maps of a record sit in a pool; per group an index row says where its A and B operand
// maps, the map of the output a fast epilogue body writes and the maps of its outputs are.
constexpr int kMapsPerGroup = 3 + kNumOuts;
enum : int { MAP_A = 0, MAP_B = 1, MAP_FAST = 2, MAP_OUT = 3 };
constexpr int kPoolAll = kMaxGroups * kMapsPerGroup;   // a launch of its own: every map has its place
constexpr int kPoolChain = 8;                          // a record of a chain: the (distinct) maps it really uses
// Epilogue bodies.  The general one handles any combination of outputs with run-time branches; the
// two common combinations have straight-line bodies (same arithmetic, same order).
enum : int32_t { EPI_GENERAL = 0, EPI_CODES1 = 1, EPI_Y = 2 };
// Fast bodies (256-column tiles only): EPI_CODES1 writes each warp's 32 x 64 int8 block with one
// TMA store (64-byte rows, 64B swizzle), EPI_Y each 32 x 32 fp32 block with one (128-byte rows,
// 128B swizzle).
struct GroupDesc {
  int32_t n, tn_begin;        // columns; first column-tile index of the group in the launch's numbering
  int32_t act;
  int32_t need_y;             // anything besides raw accumulators to produce
  int32_t mode;               // EPI_*: which epilogue body serves this group
  // chains number a record's tiles group by group (column tile fastest inside a group):
  int32_t gtiles_n, tile_first;   // column tiles of this group; record-local index of its first tile (unused: INT32_MAX)
  int32_t signal;             // a later record of the launch reads this group's output rows
  float scale_x;
  const float* scale_w;
  const float* residual; int64_t ldr;
  unsigned* amax;             // optional: bit pattern of max |output| over the whole matrix (general body only)
  OutDesc outs[kNumOuts];     // [0] raw accumulators, [1] fp32 output, [2..] consumer codes
};
// Implicit-GEMM convolution: the A operand is not a matrix in memory but the NHWC code tensor of the
// layer's input; row (b, oh, ow) of the k-block (tap, channel chunk) is gathered from pixel
// (b, oh*stride - pad + dy, ow*stride - pad + dx), zero outside the image.
struct ConvDesc {
  int32_t on, H, W, C, kh, kw, stride, pad, OH, OW, esz, K;
  int64_t img_bytes;          // bytes of one image (H * W * C * esz)
  const uint8_t* src;
};
constexpr int kMaxDeps = 4;
struct GemmParams {
  int32_t m, k_blocks, bn, tiles_m, tiles_n, stages, is_bf16;   // tiles_n: column tiles of all groups together
  int32_t epi_bytes;          // staging bytes per epilogue warp (2048 or 4096)
  uint32_t idesc;
  GroupDesc grp[kMaxGroups];  // unused groups have tn_begin = INT32_MAX
  unsigned* err;
  unsigned long long* stamp;  // optional [2]: earliest start / latest end of the launch's CTAs (%globaltimer, ns)
  ConvDesc conv;              // conv.on: A comes from the gather warps (single-group launches only)
  // chains: records of the same launch whose output rows this record reads (-1: none), and
  // whether a later record of the launch reads this one's
  uint8_t mi[kMaxGroups][kMapsPerGroup];   // pool indices of the groups' tensor maps
  int32_t deps[kMaxDeps];
  int32_t need;               // finished tiles per row tile and CTA rank that make this record's rows complete for its readers
};
// What one launch gets: one record, or a chain of them (see the kernel).
constexpr int kChainMax = 16;
template <int POOL> struct Rec { CUtensorMap m[POOL]; GemmParams p; };
template <bool CHAIN> struct LaunchArgs {
  Rec<CHAIN ? kPoolChain : kPoolAll> rec[CHAIN ? kChainMax : 1];
  int32_t n;             // records in use
  int32_t total_tiles;   // tiles of all records together
  int32_t flag_stride;   // counters per record (two per row tile: one per CTA of the pair)
  unsigned* flags;       // [n x flag_stride], zero when the launch starts
};
static_assert(sizeof(LaunchArgs<true>) <= 32764, "kernel parameters are limited to 32764 bytes");

// ---------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the CTA should give up (this or another wait timed out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* err,
                                          uint64_t limit_ns = kWaitLimitNs) {
  uint64_t t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 0) {
      if (*abort_flag) return false;
      uint64_t now = global_timer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) {
        atomicOr(err, ERR_TIMEOUT);
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// Chains: waits until a counter of finished tiles has reached `need`.  Bounded like every other wait.
__device__ __forceinline__ bool flag_wait(const unsigned* flag, uint32_t need, volatile int* abort_flag, unsigned* err,
                                          uint64_t limit_ns = kWaitLimitNs) {
  uint64_t t0 = 0;
  for (uint32_t it = 1;; ++it) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v >= need) return true;
    __nanosleep(100);        // the warp that polls is ahead of the producer; it need not spin at full rate
    if ((it & 63u) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) {
        atomicOr(err, ERR_TIMEOUT);
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// Chains: waits until the CTA's dependency warp has cleared `need` tiles (a counter in shared memory).
__device__ __forceinline__ bool cleared_wait(uint32_t addr, uint32_t need, volatile int* abort_flag, unsigned* err,
                                             uint64_t limit_ns = kWaitLimitNs) {
  uint64_t t0 = 0;
  for (uint32_t it = 1;; ++it) {
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    if (v >= need) return true;
    __nanosleep(40);
    if ((it & 1023u) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) {
        atomicOr(err, ERR_TIMEOUT);
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// Chains: waits (whole warp) until every epilogue warp has reported `need` tiles; lane w reads warp w's counter.
__device__ __forceinline__ bool reported_wait(uint32_t rep0, uint32_t need, int lane, volatile int* abort_flag, unsigned* err,
                                              uint64_t limit_ns = kWaitLimitNs) {
  uint64_t t0 = 0;
  for (uint32_t it = 1;; ++it) {
    uint32_t v = need;
    if (lane < kEpiWarps) asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(rep0 + 4 * lane) : "memory");
    if (__all_sync(0xffffffffu, v >= need)) return true;
    __nanosleep(40);
    if ((it & 1023u) == 0) {
      bool give_up = *abort_flag != 0;
      const uint64_t now = global_timer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) {
        if (lane == 0) { atomicOr(err, ERR_TIMEOUT); *abort_flag = 1; }
        give_up = true;
      }
      if (__any_sync(0xffffffffu, give_up)) return false;
    }
  }
}

// The same wait for a whole converged warp, written so that the compiler sees warp-uniform control
// flow (the spin is inside one asm statement, the outcome is a vote): the producer and the MMA
// issuer run their loops on all 32 lanes, which keeps their address and descriptor arithmetic on
// the uniform datapath, and elect one lane only for the TMA / MMA instructions themselves.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* err) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .u32 n;\n\t"
      "mov.u32 n, 64;\n\t"
      "SPIN:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "@p bra DONE;\n\t"
      "sub.u32 n, n, 1;\n\t"
      "setp.ne.u32 p, n, 0;\n\t"
      "@p bra SPIN;\n\t"
      "mov.u32 %0, 0;\n\t"
      "bra OUT;\n\t"
      "DONE:\n\t"
      "mov.u32 %0, 1;\n\t"
      "OUT:\n\t}"
      : "=r"(done) : "r"(bar), "r"(parity) : "memory");
  if (__all_sync(0xffffffffu, done != 0)) return true;
  const bool ok = mbar_wait(bar, parity, abort_flag, err);
  return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ bool elect_one() {
  uint32_t e;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(e));
  return e != 0;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

// Pair flavour (two CTAs of a cluster work on one 256-row tile, cta_group::2): the load of either
// CTA reports its bytes to the barrier of the pair's first CTA; shared-memory addresses of the
// two CTAs differ in bit 24 of the shared::cluster window.
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar & kPeerBitMask), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar) {   // arrive on the first CTA's copy of the barrier
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & kPeerBitMask) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {       // arrives on this barrier in both CTAs
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <bool BF16>
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  if (BF16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
  }
}

template <bool BF16>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  if (BF16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
  }
}

__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors used by the MMA issuer: K-major tile of 128-byte rows, 128B
// swizzle, groups of 8 rows 1024 bytes apart (the layout a 128B-swizzled TMA box produces).
// Bits 0-13 start address in 16-byte units, bit 16 leading byte offset (unused for swizzled
// K-major), bits 32-45 stride byte offset between 8-row groups (1024 >> 4), bit 46 descriptor
// version of sm_100, bits 61-63 layout type 2 = SWIZZLE_128B.

// ---------------------------------------------------------------------------- epilogue math

// int8 code of Eq. 1 in the low byte of the returned word: clamp, then add 1.5*2^23 (a
// round-half-even at integer granularity); the low mantissa byte is the two's-complement code.
__device__ __forceinline__ uint32_t code_word(float y, float inv_scale, float qmax) {
  const float t = __fmul_rn(y, inv_scale);
  // clamp to [-qmax, qmax] in one instruction: magnitude min(|t|, qmax), sign of t (qmax > 0)
  float c;
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c) : "f"(t), "f"(qmax));
  return __float_as_uint(__fadd_rn(c, 12582912.0f));
}
// low bytes of four words -> one word (byte i from word i)
__device__ __forceinline__ uint32_t pack4(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int32_t x, int32_t y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Writes one warp's 32-row x 32-column piece of an output.  Each thread holds its row's 32
// elements packed into WORDS 32-bit words (32: fp32 / int32, 16: bf16, 8: int8).
// Staged path: the warp lays the piece out in one of its two shared-memory slots and one lane
// issues a TMA store, which writes whole rows and clips at the matrix edge.  Direct path
// (outputs whose row pitch is not a multiple of 16 bytes): per-thread stores.
template <int WORDS>
__device__ __forceinline__ void store_piece(const OutDesc& o, const CUtensorMap* map, const uint32_t (&w)[WORDS],
                                            bool row_ok, int ncols, int64_t row, int row0, int col0,
                                            uint32_t stage, uint32_t stage_bytes, uint32_t& cursor, int lane) {
  constexpr int kRowBytes = WORDS * 4;
  constexpr int kElemBytes = kRowBytes / 32;
  if (o.tma) {
    // The warp's buffer holds two slots used alternately: before a slot is rewritten only the
    // store issued two pieces ago must have been read by the TMA engine (at most one store
    // stays pending).  4-byte outputs go out as two 16-column pieces of 64-byte rows (64B
    // swizzle: the 16-byte writes of eight lanes then cover all banks).
    const uint32_t slot_bytes = stage_bytes >> 1;
    constexpr int kHalves = (WORDS == 32) ? 2 : 1;
#pragma unroll
    for (int h = 0; h < kHalves; ++h) {
      if (h == 1 && ncols <= 16) break;                 // warp-uniform: the second half lies outside
      if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      __syncwarp();
      const uint32_t base = stage + (cursor & 1u) * slot_bytes;
      ++cursor;
      if (WORDS == 32) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int js = j ^ ((lane >> 1) & 3);
          st_shared_v4(base + lane * 64 + js * 16, w[16 * h + 4 * j], w[16 * h + 4 * j + 1], w[16 * h + 4 * j + 2], w[16 * h + 4 * j + 3]);
        }
      } else {
#pragma unroll
        for (int j = 0; j < WORDS / 4; ++j)
          st_shared_v4(base + lane * kRowBytes + j * 16, w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) tma_store_2d(map, base, col0 + 16 * h, row0);
    }
    return;
  }
  if (!row_ok) return;
  uint8_t* dst = reinterpret_cast<uint8_t*>(o.ptr) + (row * o.ld + col0) * kElemBytes;
  if (ncols >= 32 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
#pragma unroll
    for (int j = 0; j < WORDS / 4; ++j)
      reinterpret_cast<uint4*>(dst)[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      if (i < ncols) {
        if (kElemBytes == 4) reinterpret_cast<uint32_t*>(dst)[i] = w[i * WORDS / 32];
        else if (kElemBytes == 2) reinterpret_cast<uint16_t*>(dst)[i] = (uint16_t)(w[i >> 1] >> (16 * (i & 1)));
        else dst[i] = (uint8_t)(w[i >> 2] >> (8 * (i & 3)));
      }
    }
  }
}

// ---- fast epilogue bodies -------------------------------------------------------------------
// Two values at a time with packed fp32 instructions (same roundings as the scalar forms: each
// half is an independent round-to-nearest operation).
__device__ __forceinline__ float2 gelu_tanh2(float2 y) {
  const float2 c1 = make_float2(-2.302208198f, -2.302208198f), c3 = make_float2(-0.1029432396f, -0.1029432396f);
  const float2 y2 = __fmul2_rn(y, y);
  const float2 t = __fmul2_rn(y, __ffma2_rn(c3, y2, c1));
  float2 e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"(t.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"(t.y));
  const float2 d = __fadd2_rn(e, make_float2(1.0f, 1.0f));
  float2 r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r.x) : "f"(d.x));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r.y) : "f"(d.y));
  return __fmul2_rn(y, r);
}
// Rescaled and activated values of 16 accumulator columns of one row.  cs points to the 16
// rescale factors of these columns in shared memory (every lane reads the same addresses).
template <bool BF16>
__device__ __forceinline__ void sub_values(float2 (&y)[8], const uint32_t (&v)[16], const float* cs, int act) {
  if (BF16) {
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = make_float2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 c = *reinterpret_cast<const float4*>(cs + 4 * q);
      y[2 * q] = __fmul2_rn(make_float2((float)(int32_t)v[4 * q], (float)(int32_t)v[4 * q + 1]), make_float2(c.x, c.y));
      y[2 * q + 1] = __fmul2_rn(make_float2((float)(int32_t)v[4 * q + 2], (float)(int32_t)v[4 * q + 3]), make_float2(c.z, c.w));
    }
  }
  if (act == QCFG_ACT_RELU) {
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = make_float2(fmaxf(y[i].x, 0.0f), fmaxf(y[i].y, 0.0f));
  } else if (act == QCFG_ACT_GELU_TANH) {
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = gelu_tanh2(y[i]);
  }
}
// int8 codes of Eq. 1 for two values, each in the low byte of its word
__device__ __forceinline__ float2 code_words2(float2 y, float2 inv2, float qmax) {
  const float2 t = __fmul2_rn(y, inv2);
  float2 c;
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c.x) : "f"(t.x), "f"(qmax));
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c.y) : "f"(t.y), "f"(qmax));
  return __fadd2_rn(c, make_float2(12582912.0f, 12582912.0f));
}

// One warp's share of a 256-column tile (32 rows x 64 columns) in four pieces of 16 columns.
// The accumulator load of the next piece is in flight while the current one is processed; the
// accumulator buffer is released as soon as the last piece sits in registers.
// CODES: one int8 matrix, the warp's 32 x 64 block staged in 64-byte rows (64B swizzle) and
// written by one TMA store.  Otherwise the fp32 matrix, each 32 x 32 block staged in 128-byte
// rows (128B swizzle), one TMA store per block; the single staging slot is reused once the
// previous store has read it.
// rep_addr (chains, else 0): this warp's report counter in shared memory, set to rep_val once the
// stores the warp issued for its previous tile have completed; that is checked after this tile's
// first piece, a quarter of an epilogue after they were issued.
template <bool BF16, bool PAIR, bool CODES>
__device__ __forceinline__ void epilogue_tile_fast(const GroupDesc& G, const CUtensorMap* fmap, uint32_t tbase,
                                                   const float* cs, uint32_t stage, int row0, int col0, int lane,
                                                   uint32_t tempty_bar, uint32_t rep_addr, uint32_t rep_val) {
  const int act = G.act;
  const float qmax = G.outs[2].qmax;
  const float2 inv2 = make_float2(G.outs[2].inv_scale, G.outs[2].inv_scale);
  uint32_t va[16], vb[16];
  if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the slot's last store was a tile ago
  __syncwarp();
  tmem_ld16_issue(tbase, va);
  auto piece = [&](const uint32_t (&v)[16], int s) {
    float2 y[8];
    sub_values<BF16>(y, v, cs + 16 * s, act);
    if (CODES) {
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 a = code_words2(y[2 * j], inv2, qmax), b = code_words2(y[2 * j + 1], inv2, qmax);
        w[j] = pack4(__float_as_uint(a.x), __float_as_uint(a.y), __float_as_uint(b.x), __float_as_uint(b.y));
      }
      st_shared_v4(stage + lane * 64 + ((s ^ ((lane >> 1) & 3)) << 4), w[0], w[1], w[2], w[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int p16 = 4 * (s & 1) + j;
        st_shared_v4(stage + lane * 128 + ((p16 ^ (lane & 7)) << 4), __float_as_uint(y[2 * j].x), __float_as_uint(y[2 * j].y),
                     __float_as_uint(y[2 * j + 1].x), __float_as_uint(y[2 * j + 1].y));
      }
    }
  };
#pragma unroll 1
  for (int h = 0; h < 2; ++h) {
    tmem_ld_wait();
    tmem_ld16_issue(tbase + 32 * h + 16, vb);
    if (!CODES && h == 1) {   // the first block's store must have read the slot before it is refilled
      if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      __syncwarp();
    }
    piece(va, 2 * h);
    if (h == 0 && rep_addr && lane == 0) {    // a quarter of a tile after the previous tile's last store
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
      asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(rep_addr), "r"(rep_val) : "memory");
    }
    tmem_ld_wait();
    if (h == 0) {
      tmem_ld16_issue(tbase + 32, va);
    } else {          // every column of this warp is in registers: the accumulator buffer is free
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { if (PAIR) mbar_arrive_leader(tempty_bar); else mbar_arrive(tempty_bar); }
    }
    piece(vb, 2 * h + 1);
    if (!CODES) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0 && col0 + 32 * h < G.n) tma_store_2d(fmap, stage, col0 + 32 * h, row0);
    }
  }
  if (CODES) {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) tma_store_2d(fmap, stage, col0, row0);
  }
}

// One 32-column chunk of one accumulator row (all 32 lanes of the warp call this together).
template <bool BF16, bool CHAIN>
__device__ __forceinline__ void epilogue_chunk(const GroupDesc& p, const CUtensorMap* pool, const uint8_t* mi, int m, uint32_t epi_bytes,
                                               uint32_t (&v)[32], float cs_lane,
                                               int64_t row, int row0, int col0, uint32_t stage, uint32_t& cursor, int lane) {
  const int ncols = p.n - col0;                    // valid columns in this chunk (may be <= 0 or > 32)
  if (ncols <= 0 || row0 >= m) return;             // warp-uniform: the piece lies outside the matrix
  const bool row_ok = row < m;
  const bool full = ncols >= 32;

  if (!BF16 && p.outs[0].kind) store_piece<32>(p.outs[0], &pool[mi[MAP_OUT]], v, row_ok, ncols, row, row0, col0, stage, epi_bytes, cursor, lane);
  if (!p.need_y) return;

  float y[32];
  if (BF16) {
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = __uint_as_float(v[i]);
  } else {
    // lane i holds scale_x * scale_w[col0 + i] (loaded before the accumulator was ready)
#pragma unroll
    for (int i = 0; i < 32; ++i)
      y[i] = __fmul_rn((float)(int32_t)v[i], __shfl_sync(0xffffffffu, cs_lane, i));
  }
  if (p.residual && row_ok) {
    // In a chain another SM may have written the shortcut earlier in this launch, so it is read
    // with ordinary loads, not through the read-only path.  (A stale L1 line is impossible: within a
    // launch every address is written at most once and read only after that write has been seen.)
    const float* r = p.residual + row * p.ldr + col0;
    if (full && (p.ldr & 3) == 0 && (((uintptr_t)p.residual) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float4 r4 = CHAIN ? *(reinterpret_cast<const float4*>(r) + i) : __ldg(reinterpret_cast<const float4*>(r) + i);
        y[4 * i + 0] = __fadd_rn(y[4 * i + 0], r4.x);
        y[4 * i + 1] = __fadd_rn(y[4 * i + 1], r4.y);
        y[4 * i + 2] = __fadd_rn(y[4 * i + 2], r4.z);
        y[4 * i + 3] = __fadd_rn(y[4 * i + 3], r4.w);
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) if (i < ncols) y[i] = __fadd_rn(y[i], CHAIN ? r[i] : __ldg(r + i));
    }
  }
  if (p.act == QCFG_ACT_RELU) {
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = fmaxf(y[i], 0.0f);
  } else if (p.act == QCFG_ACT_GELU_TANH) {
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = gelu_tanh(y[i]);
  }
  if (p.amax) {     // calibration: the range of what the consumers will read (bit patterns, exact in any order)
    unsigned mx = 0;
    if (row_ok) {
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const unsigned a = __float_as_uint(y[i]) & 0x7fffffffu;
        if (i < ncols) mx = mx > a ? mx : a;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned other = __shfl_xor_sync(0xffffffffu, mx, o);
      mx = mx > other ? mx : other;
    }
    if (lane == 0 && mx) atomicMax(p.amax, mx);
  }
  if (p.outs[1].kind) {
    uint32_t w[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(y[i]);
    store_piece<32>(p.outs[1], &pool[mi[MAP_OUT + 1]], w, row_ok, ncols, row, row0, col0, stage, epi_bytes, cursor, lane);
  }
#pragma unroll
  for (int s = 0; s < kMaxSlots; ++s) {
    const OutDesc& o = p.outs[2 + s];
    if (o.kind == 1) {
      uint32_t w[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        w[i] = pack4(code_word(y[4 * i], o.inv_scale, o.qmax), code_word(y[4 * i + 1], o.inv_scale, o.qmax),
                     code_word(y[4 * i + 2], o.inv_scale, o.qmax), code_word(y[4 * i + 3], o.inv_scale, o.qmax));
      store_piece<8>(o, &pool[mi[MAP_OUT + 2 + s]], w, row_ok, ncols, row, row0, col0, stage, epi_bytes, cursor, lane);
    } else if (o.kind == 2) {
      uint32_t w[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(y[2 * i], y[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
      }
      store_piece<16>(o, &pool[mi[MAP_OUT + 2 + s]], w, row_ok, ncols, row, row0, col0, stage, epi_bytes, cursor, lane);
    }
  }
}

// ---------------------------------------------------------------------------- the kernel

// One launch runs one GEMM record or, in the CHAIN flavour, up to kChainMax records one after the
// other: consecutive layers of a model, each reading what an earlier one wrote.  The tiles of all
// records form one sequence (record after record, group after group, column tile fastest) that the
// CTA pairs deal out round-robin, so a pair that runs out of tiles of one record goes on with the
// next: no pipeline fill and drain, no idle last round and no kernel boundary between layers.
// A tile may start when the row tiles it reads are complete: every finished tile adds one to a
// counter of its (record, row tile, CTA rank) -- a warp of its own does that once the tile's stores
// have completed -- and another warp, ahead of the producer, waits for the counters of the records
// a tile's record names and clears the tile for loading.
// Waits only ever point at earlier tiles of the sequence and the launch is cooperative (all CTAs
// resident), so the first unfinished tile can always proceed.  The records of a chain share tile
// shape, operand type, stage count, staging size, rows and grid.
template <bool BF16, bool PAIR, bool GROUPED, bool CHAIN>
__global__ void __launch_bounds__(kGemmThreadsConv, 1)
gemm_kernel(const __grid_constant__ LaunchArgs<CHAIN> L) {
  const GemmParams& p = L.rec[0].p;        // what all records of the launch have in common is read here
  const GemmParams* q = &L.rec[0].p;       // the record this thread's role is working on
  const CUtensorMap* mp = L.rec[0].m;      // its pool of tensor maps
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment for the 128B swizzle atoms
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);           // full[8] empty[8] tfull[2] tempty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 260);
  const uint32_t cleared_addr = smem_u32(smem + 264);            // chains: tiles of this CTA whose inputs are complete
  float* cs_all = reinterpret_cast<float*>(smem + kSmemHeader);  // kEpiWarps x 64 rescale factors
  uint8_t* epi_stage = smem + kSmemHeader + kCsBytes;            // kEpiWarps x epi_bytes, 1024-aligned
  uint8_t* stage_base = epi_stage + kEpiWarps * p.epi_bytes;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // Pair flavour: the two CTAs of a cluster share one 256-row tile.  Each loads its own 128 rows
  // of A and its own half of the tile's B rows; the first CTA issues the MMAs for both
  // (cta_group::2), each CTA's TMEM receives the accumulators of its 128 rows.  p.tiles_m then
  // counts 256-row tiles.
  const int rank = PAIR ? (int)cluster_ctarank() : 0;
  const int b_rows = PAIR ? (p.bn >> 1) : p.bn;                  // B rows held per stage by this CTA
  const uint32_t stage_bytes = (uint32_t)(BM + b_rows) * kStageKBytes;
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kMaxStages;
  const uint32_t tfull0 = empty0 + 8 * kMaxStages, tempty0 = tfull0 + 16;
  // chains: per epilogue warp, the number of its tiles whose stores have completed (counters, not
  // phase barriers: the warp that reads them may fall any number of tiles behind)
  const uint32_t rep0 = smem_u32(smem + 320);
  const int tile0 = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // first tile of this CTA (pair)
  const int tile_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int rows_per_tile = PAIR ? 2 * BM : BM;
  // group of a column tile (a single-GEMM launch has only group 0, known at compile time)
  auto group_of = [&](int tn) -> int {
    return GROUPED ? (int)(tn >= q->grp[1].tn_begin) + (int)(tn >= q->grp[2].tn_begin) : 0;
  };
  auto tile_in_group = [&](int tn, int g) -> int { return GROUPED ? tn - q->grp[g].tn_begin : tn; };
  // Tiles are numbered with the row-tile index fastest.  Each role walks its tiles by adding the
  // stride split into (row tiles, column tiles) once here: a division per tile would sit on the
  // epilogue's and the producer's path.
  int num_tiles, step_tn, step_tm, tm0, tn0;
  auto set_record = [&](int li) {
    q = &L.rec[CHAIN ? li : 0].p;
    mp = L.rec[CHAIN ? li : 0].m;
    num_tiles = q->tiles_m * q->tiles_n;
    step_tn = tile_step / q->tiles_m; step_tm = tile_step - step_tn * q->tiles_m;
    tm0 = tile0 % q->tiles_m; tn0 = tile0 / q->tiles_m;
  };
  set_record(0);
  // chains: position in the launch's tile sequence
  struct Cur { int li, first, ntiles; const GemmParams* q; const CUtensorMap* mp; };
  auto cur_seek = [&](Cur& c, int g) {       // g < L.total_tiles
    while (g >= c.first + c.ntiles) {
      c.first += c.ntiles; ++c.li;
      c.q = &L.rec[CHAIN ? c.li : 0].p; c.mp = L.rec[CHAIN ? c.li : 0].m;
      c.ntiles = c.q->tiles_m * c.q->tiles_n;
    }
  };
  Cur cur{0, 0, num_tiles, q, mp};
  // record-local tile index -> group, row tile, column tile (column tiles numbered over all groups)
  auto locate = [&](const GemmParams* qq, int T, int& gi, int& tm, int& tn) {
    gi = (int)(T >= qq->grp[1].tile_first) + (int)(T >= qq->grp[2].tile_first);
    const GroupDesc& G = qq->grp[gi];
    const int Tl = T - G.tile_first;
    tm = Tl / G.gtiles_n;
    tn = G.tn_begin + (Tl - tm * G.gtiles_n);
  };
  const int total_tiles = CHAIN ? L.total_tiles : num_tiles;

  // producer state (thread 0 only): next k-block to load
  // The producer and the MMA issuer share their scheduler with four epilogue warps that almost
  // always have an instruction ready, so every instruction these two threads need per k-block
  // costs them many cycles of waiting for an issue slot: their loops keep all addresses and
  // coordinates in registers and update them incrementally.
  int ld_tile = tile0, ld_kb = 0, ld_s = 0;
  uint32_t ld_ph = 0;
  const int k_elems = BF16 ? kStageKBytes / 2 : kStageKBytes;
  const uint32_t stage0 = smem_u32(stage_base);
  uint32_t ld_dst = stage0, ld_bar = full0;      // stage address and its full barrier
  int ld_x = 0, ld_ya = 0, ld_yb = 0;            // TMA coordinates of the next k-block
  int ld_tm = tm0, ld_tn = tn0;
  const CUtensorMap* ld_map_a = &mp[q->mi[0][MAP_A]];
  const CUtensorMap* ld_map_b = &mp[q->mi[0][MAP_B]];
  auto set_tile_coords = [&]() {
    const int g = group_of(ld_tn);
    if (GROUPED) { ld_map_a = &mp[q->mi[g][MAP_A]]; ld_map_b = &mp[q->mi[g][MAP_B]]; }
    ld_ya = ld_tm * rows_per_tile + rank * BM;
    ld_yb = tile_in_group(ld_tn, g) * p.bn + rank * b_rows;
  };
  set_tile_coords();
  const bool elected = elect_one();    // the lane of a converged warp that issues TMA / MMA instructions
  const bool conv_on = p.conv.on != 0;
  // bytes the TMA loads of one CTA put into a stage (the A tile is gathered in convolution launches)
  const uint32_t tma_bytes = conv_on ? (uint32_t)b_rows * kStageKBytes : stage_bytes;
  auto issue_load = [&]() {   // whole warp 0; the stage's empty barrier must already have been passed
    if (elected) {
    if (PAIR) {
      // the first CTA's barrier collects the bytes of both CTAs' loads
      if (rank == 0) mbar_expect_tx(ld_bar, 2 * tma_bytes);
      if (!conv_on) tma_load_2d_pair(ld_dst, ld_map_a, ld_bar, ld_x, ld_ya);
      tma_load_2d_pair(ld_dst + BM * kStageKBytes, ld_map_b, ld_bar, ld_x, ld_yb);
    } else {
      mbar_expect_tx(ld_bar, tma_bytes);
      if (!conv_on) tma_load_2d(ld_dst, ld_map_a, ld_bar, ld_x, ld_ya);
      tma_load_2d(ld_dst + BM * kStageKBytes, ld_map_b, ld_bar, ld_x, ld_yb);
    }
    }
    ld_dst += stage_bytes; ld_bar += 8; ld_x += k_elems;
    if (++ld_s == p.stages) { ld_s = 0; ld_ph ^= 1; ld_dst = stage0; ld_bar = full0; }
    if (++ld_kb == q->k_blocks) {
      ld_kb = 0; ld_x = 0; ld_tile += tile_step;
      ld_tm += step_tm; ld_tn += step_tn;
      if (ld_tm >= q->tiles_m) { ld_tm -= q->tiles_m; ++ld_tn; }
      set_tile_coords();
    }
  };

  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&mp[q->mi[0][MAP_A]]) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&mp[q->mi[0][MAP_B]]) : "memory");
    const uint32_t full_count = 1 + (p.conv.on ? kGatherWarps * (PAIR ? 2 : 1) : 0);   // the TMA thread, plus one arrival per gather warp
    for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, full_count); mbar_init(empty0 + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, PAIR ? 2 * kEpiWarps : kEpiWarps); }
    if (CHAIN) for (int a = 0; a < kEpiWarps; ++a) *reinterpret_cast<volatile uint32_t*>(smem + 320 + 4 * a) = 0u;
    *abort_flag = 0;
    *reinterpret_cast<volatile uint32_t*>(smem + 264) = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (PAIR) {   // the same warp of both CTAs allocates for the pair
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  if (PAIR) {     // both CTAs' barriers exist before either one's loads or arrivals can reach them
    __syncthreads();
    cluster_sync_all();
  }
  // Everything above touches no global memory, so under programmatic dependent launch it
  // overlaps the tail of the previous kernel in the stream; from here on its results are needed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (p.stamp && threadIdx.x == 32) atomicMin(p.stamp, (unsigned long long)global_timer());
  if (warp == 0) {
    // the ring is empty: fill it before the block-wide barrier so the first tiles are in flight
    if (!CHAIN) for (int i = 0; i < p.stages && ld_tile < num_tiles; ++i) issue_load();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    bool ok = true;
    if (CHAIN) {
      // The dependency warp clears tiles ahead of time (see there); here only a counter in shared
      // memory is read, so no device-scope fence sits between two tiles' loads.
      uint32_t t_ld = 0;
      for (int g = tile0; g < total_tiles && ok; g += tile_step) {
        cur_seek(cur, g);
        const GemmParams* cq = cur.q;
        int gi, tm, tn;
        locate(cq, g - cur.first, gi, tm, tn);
        if (!cleared_wait(cleared_addr, ++t_ld, abort_flag, p.err)) { ok = false; break; }
        const CUtensorMap* ma = &cur.mp[cq->mi[gi][MAP_A]];
        const CUtensorMap* mb = &cur.mp[cq->mi[gi][MAP_B]];
        const int ya = tm * rows_per_tile + rank * BM;
        const int yb = (tn - cq->grp[gi].tn_begin) * p.bn + rank * b_rows;
        int x = 0;
        for (int kb = 0; kb < cq->k_blocks; ++kb) {
          if (!mbar_wait_warp(ld_bar + 8 * kMaxStages, ld_ph ^ 1, abort_flag, p.err)) { ok = false; break; }
          if (elected) {
            if (rank == 0) mbar_expect_tx(ld_bar, 2 * stage_bytes);
            tma_load_2d_pair(ld_dst, ma, ld_bar, x, ya);
            tma_load_2d_pair(ld_dst + BM * kStageKBytes, mb, ld_bar, x, yb);
          }
          ld_dst += stage_bytes; ld_bar += 8; x += k_elems;
          if (++ld_s == p.stages) { ld_s = 0; ld_ph ^= 1; ld_dst = stage0; ld_bar = full0; }
        }
      }
    } else {
      while (ld_tile < num_tiles) {
        if (!mbar_wait_warp(ld_bar + 8 * kMaxStages, ld_ph ^ 1, abort_flag, p.err)) { ok = false; break; }
        issue_load();
      }
    }
    if (PAIR && ok) {
      // the peer's MMA completions still arrive on this CTA's stage barriers: drain them all
      // before this CTA may exit (a stage never filled passes at once)
      for (int i = 0; i < p.stages && ok; ++i) {
        if (!mbar_wait_warp(empty0 + 8 * ld_s, ld_ph ^ 1, abort_flag, p.err)) ok = false;
        if (++ld_s == p.stages) { ld_s = 0; ld_ph ^= 1; }
      }
    }
    if (!ok) {
      // give copies already in flight a bounded time to land before the CTA exits
      const uint64_t t0 = global_timer();
      while (global_timer() - t0 < 200000ull) {}
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (rank == 0) {
      // Descriptor low words (start address field, 16-byte units) of the four K steps of the
      // current stage's A and B tiles; the high word is the same for all.
      constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
      const uint32_t lo0 = ((stage0 >> 4) & 0x3FFFu) | (1u << 16);
      const uint32_t lo_step = stage_bytes >> 4;
      constexpr uint32_t kBOff = (uint32_t)(BM * kStageKBytes) >> 4;
      uint32_t lo = lo0, fb = full0;
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      int t = 0;
      auto mma4 = [&](uint32_t d_tmem, uint32_t first_acc) {
        if (!elected) return;
#pragma unroll
        for (int k4 = 0; k4 < kStageKBytes / kUmmaKBytes; ++k4) {
          // advancing the start address by 32 bytes (2 units) steps along K inside the swizzle atom
          const uint64_t da = ((uint64_t)kDescHi << 32) | (uint64_t)(lo + 2u * k4);
          const uint64_t db = ((uint64_t)kDescHi << 32) | (uint64_t)(lo + kBOff + 2u * k4);
          const uint32_t acc = k4 == 0 ? first_acc : 1u;
          if (PAIR) tc_mma_pair<BF16>(d_tmem, da, db, p.idesc, acc);
          else tc_mma<BF16>(d_tmem, da, db, p.idesc, acc);
        }
      };
      for (int tile = tile0; tile < total_tiles && ok; tile += tile_step, ++t) {
        if (CHAIN) { cur_seek(cur, tile); q = cur.q; }
        const int a = t & 1;
        if (!mbar_wait_warp(tempty0 + 8 * a, ((t >> 1) & 1) ^ 1, abort_flag, p.err)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)a * kAccCols;
        for (int kb = 0; kb < q->k_blocks; ++kb) {
          if (!mbar_wait_warp(fb, ph, abort_flag, p.err)) { ok = false; break; }
          tc_fence_after();
          mma4(d_tmem, kb != 0);
          // stage reusable once these MMAs have read it
          if (elected) { if (PAIR) tc_commit_pair(fb + 8 * kMaxStages); else tc_commit(fb + 8 * kMaxStages); }
          lo += lo_step; fb += 8;
          if (++s == p.stages) { s = 0; ph ^= 1; lo = lo0; fb = full0; }
        }
        if (ok && elected) { if (PAIR) tc_commit_pair(tfull0 + 8 * a); else tc_commit(tfull0 + 8 * a); }   // accumulator complete
      }
    }
  } else if (CHAIN && warp >= 2 + kEpiWarps) {
    // ------------------------------------------------------------------ signal warp (chains)
    // For each of this CTA's tiles in order: once all epilogue warps have seen their stores of
    // the tile complete (the bulk-group wait makes the TMA writes visible to the waiting thread,
    // whose barrier arrival this warp has acquired), publish it with a release at device scope:
    // one is added to the counter of its record, row tile and CTA rank.
    if (warp == 2 + kEpiWarps) {
      int t = 0;
      for (int g = tile0; g < total_tiles; g += tile_step, ++t) {
        cur_seek(cur, g);
        if (!reported_wait(rep0, (uint32_t)t + 1u, lane, abort_flag, p.err)) break;
        int gi, tm, tn;
        locate(cur.q, g - cur.first, gi, tm, tn);
        if (elected && cur.q->grp[gi].signal) {
          asm volatile("red.release.gpu.global.add.u32 [%0], 1;"
                       ::"l"(L.flags + (size_t)cur.li * L.flag_stride + 2 * tm + rank) : "memory");
        }
      }
    } else if (warp == 3 + kEpiWarps) {
      // ---------------------------------------------------------------- dependency warp (chains)
      // Walks this CTA's tiles ahead of the producer.  For each, lane d waits (acquire at device
      // scope, bounded) until the counter of dependency d says the rows the tile reads are
      // complete; then one lane orders the asynchronous proxy after that and publishes the tile
      // count in shared memory, which is all the producer looks at.  The two device-scope fences
      // cost about a microsecond each under load, and here they delay nobody.
      uint32_t t_clear = 0;
      for (int g = tile0; g < total_tiles; g += tile_step) {
        cur_seek(cur, g);
        int gi, tm, tn;
        locate(cur.q, g - cur.first, gi, tm, tn);
        const int dep = lane < kMaxDeps ? cur.q->deps[lane] : -1;
        bool failed = false;
        if (dep >= 0)
          failed = !flag_wait(L.flags + (size_t)dep * L.flag_stride + 2 * tm + rank, (uint32_t)L.rec[dep].p.need, abort_flag, p.err);
        const bool had = __any_sync(0xffffffffu, dep >= 0);
        if (__any_sync(0xffffffffu, failed)) break;
        ++t_clear;
        __syncwarp();
        if (elected) {
          if (had) asm volatile("fence.proxy.async;" ::: "memory");
          asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(cleared_addr), "r"(t_clear) : "memory");
        }
      }
    }
  } else if (warp >= 2 + kEpiWarps) {
    // ------------------------------------------------------------------ gather warps (convolutions)
    // Each lane owns two rows of the CTA's 128-row A tile.  Per k-block it copies the rows' eight
    // 16-byte chunks from the NHWC source (cp.async with zero fill outside the image, beyond the
    // reduction length and past the last row) to where a 128B-swizzled TMA box would have put them.
    // kGatherDepth k-blocks stay in flight; when the oldest has landed the lane makes its writes
    // visible to the tensor core (fence.proxy.async) and one lane per warp arrives on the stage's
    // full barrier (the pair's first CTA's).
    const ConvDesc& cv = p.conv;
    const int gw = warp - (2 + kEpiWarps);
    const int epc = 16 / cv.esz;                       // elements per 16-byte chunk
    const int opix = cv.OH * cv.OW;
    int s = 0, as = 0, inflight = 0;
    uint32_t ph = 0;
    int tm = tm0, tn = tn0;
    bool ok = true;
    auto landed = [&]() {                              // the oldest group in flight has landed
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) { if (PAIR) mbar_arrive_leader(full0 + 8 * as); else mbar_arrive(full0 + 8 * as); }
      if (++as == p.stages) as = 0;
      --inflight;
    };
    for (int tile = tile0; tile < num_tiles && ok; tile += tile_step) {
      int ih0[2], iw0[2];
      const uint8_t* img[2];
      bool rv[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int64_t pm = (int64_t)tm * rows_per_tile + rank * BM + gw * 64 + i * 32 + lane;
        rv[i] = pm < p.m;
        const int q = rv[i] ? (int)pm : 0;
        const int b = q / opix, pix = q - b * opix;
        const int oh = pix / cv.OW, ow = pix - oh * cv.OW;
        ih0[i] = oh * cv.stride - cv.pad;
        iw0[i] = ow * cv.stride - cv.pad;
        img[i] = cv.src + (int64_t)b * cv.img_bytes;
      }
      int dy = 0, dx = 0, c = 0, ke = 0;
      for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
        if (!mbar_wait_warp(empty0 + 8 * s, ph ^ 1, abort_flag, p.err)) { ok = false; break; }
        const uint32_t a_dst = stage0 + (uint32_t)s * stage_bytes + (uint32_t)(gw * 64 + lane) * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const bool kin = ke < cv.K;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const int ih = ih0[i] + dy, iw = iw0[i] + dx;
            const bool valid = rv[i] && kin && (unsigned)ih < (unsigned)cv.H && (unsigned)iw < (unsigned)cv.W;
            const uint8_t* src = valid ? img[i] + ((int64_t)(ih * cv.W + iw) * cv.C + c) * cv.esz : cv.src;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                         ::"r"(a_dst + i * 32 * 128 + ((j ^ (lane & 7)) << 4)), "l"(src), "r"(valid ? 16 : 0) : "memory");
          }
          ke += epc; c += epc;
          if (c >= cv.C) { c = 0; if (++dx == cv.kw) { dx = 0; ++dy; } }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (++s == p.stages) { s = 0; ph ^= 1; }
        if (++inflight > kGatherDepth) {
          asm volatile("cp.async.wait_group %0;" ::"n"(kGatherDepth) : "memory");
          landed();
        }
      }
      tm += step_tm; tn += step_tn;
      if (tm >= p.tiles_m) { tm -= p.tiles_m; ++tn; }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    while (inflight > 0) landed();
  } else {
    // ------------------------------------------------------------------ epilogue
    const int ew = warp - 2;
    const int quad = warp & 3;                 // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
    const int colgrp = ew >> 2;                // four warp sets share the tile's columns
    const int chunks = p.bn >> 5;
    const int cpg = chunks >= 4 ? (chunks >> 2) : 1;
    const int c_begin = colgrp * cpg;
    const int c_end = c_begin < chunks ? c_begin + cpg : c_begin;
    const uint32_t stage = smem_u32(epi_stage + ew * p.epi_bytes);
    float* cs_tab = cs_all + ew * 64;
    uint32_t cursor = 0;
    bool prev_fast = false;
    bool ok = true;
    int t = 0;
    // Weight scales of this warp's chunks, one column per lane and chunk.  They are fetched one
    // tile ahead: when the epilogue is the longer phase the accumulator is already waiting at
    // the top of the loop, and a load issued there would put its whole latency on the tile.
    auto load_scales = [&](const GemmParams* qq, bool valid, int tile_tn, float (&w)[2]) {
      w[0] = 0.f; w[1] = 0.f;
      if (BF16 || !valid) return;
      const int gi = GROUPED ? (int)(tile_tn >= qq->grp[1].tn_begin) + (int)(tile_tn >= qq->grp[2].tn_begin) : 0;
      const GroupDesc& G = qq->grp[gi];
      if (!G.need_y) return;
      const int cb = (GROUPED ? tile_tn - G.tn_begin : tile_tn) * p.bn + c_begin * 32;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int col = cb + j * 32 + lane;
        if (c_begin + j < c_end && col < G.n) w[j] = __ldg(G.scale_w + col);
      }
    };
    float sw_next[2];
    int tm = tm0, tn = tn0;
    if (CHAIN) {
      if (tile0 < total_tiles) {
        cur_seek(cur, tile0);
        int gi0, tm_0, tn_0;
        locate(cur.q, tile0 - cur.first, gi0, tm_0, tn_0);
        load_scales(cur.q, true, tn_0, sw_next);
      }
    } else {
      load_scales(q, tile0 < num_tiles, tn0, sw_next);
    }
    for (int tile = tile0; tile < total_tiles && ok; tile += tile_step, ++t) {
      if (CHAIN) {     // record of this tile, column tile fastest inside it
        cur_seek(cur, tile); q = cur.q; mp = cur.mp;
        int gi_;
        locate(q, tile - cur.first, gi_, tm, tn);
      }
      const int a = t & 1;
      const int row0 = tm * rows_per_tile + rank * BM + quad * 32;
      const int g = group_of(tn);
      const GroupDesc& G = q->grp[g];
      const int col_base = tile_in_group(tn, g) * p.bn + c_begin * 32;
      const float cs[2] = {__fmul_rn(G.scale_x, sw_next[0]), __fmul_rn(G.scale_x, sw_next[1])};
      int tm_next = tm + step_tm, tn_next = tn + step_tn;
      if (CHAIN) {
        const int nt = tile + tile_step;
        Cur c2 = cur;
        if (nt < total_tiles) cur_seek(c2, nt);
        int gi2 = 0, tm2 = 0, tn2 = 0;
        if (nt < total_tiles) locate(c2.q, nt - c2.first, gi2, tm2, tn2);
        load_scales(c2.q, nt < total_tiles, tn2, sw_next);
      } else {
        if (tm_next >= q->tiles_m) { tm_next -= q->tiles_m; ++tn_next; }
        load_scales(q, tile + tile_step < num_tiles, tn_next, sw_next);
      }
      // Chains: the previous tile is reported once its stores have completed.  When this tile's
      // accumulator is already there the check is left to the body (after its first piece, when
      // the old stores have landed); when it is not, this tile may itself be waiting for
      // rows other CTAs produce, and they for the report, so the report goes out now.
      uint32_t rep_addr = (CHAIN && t > 0) ? rep0 + 4 * ew : 0u;
      const bool fast_inside = G.mode != EPI_GENERAL && !(row0 >= q->m || col_base >= G.n);
      if (rep_addr && !(fast_inside && __all_sync(0xffffffffu, mbar_try_wait(tfull0 + 8 * a, (t >> 1) & 1)))) {
        if (lane == 0) {
          asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
          asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(rep_addr), "r"((uint32_t)t) : "memory");
        }
        __syncwarp();
        rep_addr = 0;
      }
      if (!mbar_wait(tfull0 + 8 * a, (t >> 1) & 1, abort_flag, p.err)) { ok = false; break; }
      tc_fence_after();
      const uint32_t tbase = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(a * kAccCols + c_begin * 32);
      const int nch = c_end - c_begin;           // 0, 1 or 2
      const int64_t row = (int64_t)row0 + lane;
      const uint32_t tempty_bar = tempty0 + 8 * a;
      if (G.mode != EPI_GENERAL) {
        // fast bodies: 256-column tiles, so this warp owns 64 columns starting at col_base
        if (!fast_inside) {
          __syncwarp();
          if (lane == 0) { if (PAIR) mbar_arrive_leader(tempty_bar); else mbar_arrive(tempty_bar); }
        } else {
          if (!BF16) {   // rescale factors of the 64 columns, read back by every lane
            cs_tab[lane] = cs[0];
            cs_tab[32 + lane] = cs[1];
            __syncwarp();
          }
          if (G.mode == EPI_CODES1)
            epilogue_tile_fast<BF16, PAIR, true>(G, &mp[q->mi[g][MAP_FAST]], tbase, cs_tab, stage, row0, col_base, lane, tempty_bar, rep_addr, (uint32_t)t);
          else
            epilogue_tile_fast<BF16, PAIR, false>(G, &mp[q->mi[g][MAP_FAST]], tbase, cs_tab, stage, row0, col_base, lane, tempty_bar, rep_addr, (uint32_t)t);
        }
        prev_fast = true;
      } else {
        if (prev_fast) {    // a fast body's last store reads the whole staging buffer: let it finish
          if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          __syncwarp();
          prev_fast = false;
        }
        uint32_t v[32];
        // one copy of the chunk code, looped: keeps the instruction footprint small
#pragma unroll 1
        for (int c = 0; c < nch; ++c) {
          tmem_ld32_issue(tbase + 32 * c, v);
          tmem_ld_wait();
          if (c == nch - 1) {   // the accumulator buffer is free again once this warp's columns sit in registers
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { if (PAIR) mbar_arrive_leader(tempty_bar); else mbar_arrive(tempty_bar); }
          }
          const float csl = c ? cs[1] : cs[0];
          epilogue_chunk<BF16, CHAIN>(G, mp, q->mi[g], q->m, (uint32_t)p.epi_bytes, v, csl, row, row0, col_base + 32 * c, stage, cursor, lane);
        }
        if (nch == 0) {
          __syncwarp();
          if (lane == 0) { if (PAIR) mbar_arrive_leader(tempty_bar); else mbar_arrive(tempty_bar); }
        }
      }
      if (!CHAIN) { tm = tm_next; tn = tn_next; }
    }
    if (CHAIN && t > 0 && ok) {       // the last tile: report it as soon as its stores have completed
      if (lane == 0) {
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(rep0 + 4 * ew), "r"((uint32_t)t) : "memory");
      }
    }
    // all TMA stores of this warp must have completed before the CTA's shared memory goes away
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  tc_fence_before();
  __syncthreads();
  if (p.stamp && threadIdx.x == 32) atomicMax(p.stamp + 1, (unsigned long long)global_timer());
  if (PAIR) cluster_sync_all();     // the peer no longer signals this CTA's barriers nor uses its TMEM
  if (warp == 1) {
    tc_fence_after();
    if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------- host side

// Host state of the chain being collected (one per context).
struct Span { const uint8_t* lo; const uint8_t* hi; };      // byte range [lo, hi) of a matrix
struct ChainRecInfo { Span in[2 * kMaxGroups]; int n_in; Span out[kNumOuts * kMaxGroups]; int out_grp[kNumOuts * kMaxGroups]; int n_out; };
constexpr size_t kFlagRingBytes = 8u << 20;
constexpr int kChainMaxTilesM = 2048;
struct ChainState {
  LaunchArgs<true> args;          // args.n records collected so far
  // the first record once more, set up as a launch of its own: a chain that ends with one record
  // goes out that way (the cooperative launch only pays when tiles of several GEMMs can overlap)
  LaunchArgs<false> solo;
  int solo_grid = 0, solo_grouped = 0;
  size_t solo_smem = 0;
  ChainRecInfo info[kChainMax];
  double ops = 0.0;
  unsigned* ring = nullptr;       // device counters, handed out front to back and cleared when used up
  unsigned* zero = nullptr;       // a device word that stays zero (self-test of the bounded waits)
  size_t ring_used = 0;           // bytes
  bool open = false;              // a forward pass is running: eligible launches may be deferred
  bool bf16 = false;
  int grid = 0;
  int64_t m = 0;
  size_t smem = 0;
  cudaStream_t st = nullptr;
  ChainState() { memset(&args, 0, sizeof(args)); memset(&solo, 0, sizeof(solo)); }
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// A two-dimensional tiled tensor map.  Encoding one costs a driver call of a microsecond or two and
// an evaluation needs a couple of hundred, always the same ones (a map depends only on address,
// shape, pitch, box, type and swizzle), so encoded maps are kept in a process-wide table.
struct MapKey {
  const void* ptr; uint64_t d0, d1, pitch; uint32_t b0, b1, dt, swz, promo;
  bool operator==(const MapKey& o) const {
    return ptr == o.ptr && d0 == o.d0 && d1 == o.d1 && pitch == o.pitch && b0 == o.b0 && b1 == o.b1 && dt == o.dt &&
           swz == o.swz && promo == o.promo;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    uint64_t h = (uint64_t)(uintptr_t)k.ptr * 0x9E3779B97F4A7C15ull;
    auto mix = [&](uint64_t v) { h ^= v + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2); };
    mix(k.d0); mix(k.d1); mix(k.pitch); mix(((uint64_t)k.b0 << 32) | k.b1); mix(((uint64_t)k.dt << 40) | ((uint64_t)k.swz << 20) | k.promo);
    return (size_t)h;
  }
};
std::mutex g_map_mutex;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_map_cache;
constexpr size_t kMapCacheMax = 16384;

bool encode_2d(CUtensorMap* map, CUtensorMapDataType dt, const void* ptr, uint64_t d0, uint64_t d1, uint64_t pitch_bytes,
               uint32_t b0, uint32_t b1, CUtensorMapSwizzle swz, CUtensorMapL2promotion promo) {
  const MapKey key{ptr, d0, d1, pitch_bytes, b0, b1, (uint32_t)dt, (uint32_t)swz, (uint32_t)promo};
  {
    std::lock_guard<std::mutex> lock(g_map_mutex);
    auto it = g_map_cache.find(key);
    if (it != g_map_cache.end()) { *map = it->second; return true; }
  }
  cuuint64_t dims[2] = {d0, d1};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {b0, b1};
  cuuint32_t estr[2] = {1, 1};
  const CUresult r = g_encode(map, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, promo,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  std::lock_guard<std::mutex> lock(g_map_mutex);
  if (g_map_cache.size() >= kMapCacheMax) g_map_cache.clear();
  g_map_cache.emplace(key, *map);
  return true;
}

int make_map(Ctx* ctx, CUtensorMap* map, const void* ptr, int is_bf16, int64_t k, int64_t rows, int64_t ld, int box_rows) {
  const int esz = is_bf16 ? 2 : 1;
  if (!encode_2d(map, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, ptr, (uint64_t)k, (uint64_t)rows,
                 (uint64_t)(ld * esz), (uint32_t)(kStageKBytes / esz), (uint32_t)box_rows, CU_TENSOR_MAP_SWIZZLE_128B,
                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
    return set_error(ctx, QCFG_ECUDA, "cuTensorMapEncodeTiled failed");
  return QCFG_OK;
}

// Tensor map of an output matrix [m x n] for stores of 32-row pieces (32 columns, or 16 for 4-byte elements).  Returns false
// (direct stores are used instead) when the pointer or the row pitch is not 16-byte aligned.
bool make_out_map(CUtensorMap* map, const OutDesc& o, int64_t m, int64_t n) {
  int esz; CUtensorMapDataType dt;
  switch (o.kind) {
    case 1: esz = 1; dt = CU_TENSOR_MAP_DATA_TYPE_UINT8; break;
    case 2: esz = 2; dt = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16; break;
    case 3: esz = 4; dt = CU_TENSOR_MAP_DATA_TYPE_FLOAT32; break;
    default: esz = 4; dt = CU_TENSOR_MAP_DATA_TYPE_INT32; break;
  }
  if (((uintptr_t)o.ptr & 15) || ((o.ld * esz) & 15)) return false;
  return encode_2d(map, dt, o.ptr, (uint64_t)n, (uint64_t)m, (uint64_t)(o.ld * esz), esz == 4 ? 16u : 32u, 32u,
                   esz == 4 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// Tensor map of the output a fast epilogue body writes: 32-row boxes of 64 int8 columns (64B
// swizzle) or of 32 fp32 columns (128B swizzle).
bool make_fast_map(CUtensorMap* map, const OutDesc& o, int64_t m, int64_t n) {
  const bool codes = o.kind == 1;
  const int esz = codes ? 1 : 4;
  if (((uintptr_t)o.ptr & 15) || ((o.ld * esz) & 15)) return false;
  return encode_2d(map, codes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, o.ptr, (uint64_t)n, (uint64_t)m,
                   (uint64_t)(o.ld * esz), codes ? 64u : 32u, 32u, codes ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

// Self-test of the bounded waits: the kernel waits on a barrier nothing ever arrives on and on
// counters (global and shared) nothing ever advances, each with a caller-chosen limit.  Every wait
// has to give up; only then does the last one set the time-out bit of the error word.  The kernel
// ends normally either way.
__global__ void wait_timeout_kernel(uint64_t limit_ns, unsigned* err, const unsigned* zero_word) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  __shared__ unsigned local_err;
  __shared__ uint32_t counters[kEpiWarps + 1];
  if (threadIdx.x == 0) {
    abort_flag = 0;
    local_err = 0;
    for (int i = 0; i <= kEpiWarps; ++i) counters[i] = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const int lane = threadIdx.x & 31;
  // whole-warp wait on the per-warp report counters
  const bool gave_up_rep = !reported_wait(smem_u32(&counters[0]), 1u, lane, &abort_flag, &local_err, limit_ns);
  bool all = gave_up_rep;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    all = all && !cleared_wait(smem_u32(&counters[kEpiWarps]), 1u, &abort_flag, &local_err, limit_ns);
    abort_flag = 0;
    all = all && !flag_wait(zero_word, 1u, &abort_flag, &local_err, limit_ns);
    abort_flag = 0;
    if (all) (void)mbar_wait(smem_u32(&bar), 0, &abort_flag, err, limit_ns);
  }
}

}  // namespace

int launch_wait_timeout(Ctx* ctx, uint64_t limit_ns, cudaStream_t st) {
  ChainState* cs = static_cast<ChainState*>(chain_slot(ctx));
  if (!cs) return set_error(ctx, QCFG_ESTATE, "wait self-test: context not initialised");
  wait_timeout_kernel<<<1, 32, 0, st>>>(limit_ns, err_word(ctx), cs->zero);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "wait self-test launch");
}

int gemm_init(Ctx* ctx) {
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
      return set_error(ctx, QCFG_ECUDA, "cuTensorMapEncodeTiled entry point not found");
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  cudaError_t e = cudaSuccess;
  const void* kernels[10] = {
      (const void*)gemm_kernel<false, false, false, false>, (const void*)gemm_kernel<false, false, true, false>,
      (const void*)gemm_kernel<false, true, false, false>,  (const void*)gemm_kernel<false, true, true, false>,
      (const void*)gemm_kernel<true, false, false, false>,  (const void*)gemm_kernel<true, false, true, false>,
      (const void*)gemm_kernel<true, true, false, false>,   (const void*)gemm_kernel<true, true, true, false>,
      (const void*)gemm_kernel<false, true, true, true>,    (const void*)gemm_kernel<true, true, true, true>};
  for (int i = 0; i < 10 && e == cudaSuccess; ++i)
    e = cudaFuncSetAttribute(kernels[i], cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
  if (e != cudaSuccess) return check_cuda(ctx, e, "gemm smem attribute");
  ChainState* cs = new (std::nothrow) ChainState();
  if (!cs) return set_error(ctx, QCFG_ENOMEM, "gemm: host allocation failed");
  e = cudaMalloc(&cs->ring, kFlagRingBytes);
  if (e == cudaSuccess) e = cudaMemset(cs->ring, 0, kFlagRingBytes);
  if (e == cudaSuccess) e = cudaMalloc(&cs->zero, sizeof(unsigned));
  if (e == cudaSuccess) e = cudaMemset(cs->zero, 0, sizeof(unsigned));
  if (e != cudaSuccess) {
    if (cs->ring) cudaFree(cs->ring);
    if (cs->zero) cudaFree(cs->zero);
    delete cs;
    return check_cuda(ctx, e, "gemm chain counters");
  }
  chain_slot(ctx) = cs;
  return QCFG_OK;
}

void gemm_destroy(Ctx* ctx) {
  ChainState* cs = static_cast<ChainState*>(chain_slot(ctx));
  if (!cs) return;
  if (cs->ring) cudaFree(cs->ring);
  if (cs->zero) cudaFree(cs->zero);
  delete cs;
  chain_slot(ctx) = nullptr;
}

// ----- chains: consecutive GEMM launches of a forward pass folded into one cooperative launch

void gemm_chain_open(Ctx* ctx) {
  ChainState* cs = static_cast<ChainState*>(chain_slot(ctx));
  if (cs && ctx_chain_enabled(ctx)) cs->open = true;
}

int gemm_chain_flush(Ctx* ctx) {
  ChainState* cs = static_cast<ChainState*>(chain_slot(ctx));
  if (!cs || cs->args.n == 0) return QCFG_OK;
  const int n = cs->args.n;
  cs->args.n = 0;
  LaunchArgs<true>& A = cs->args;
  if (n == 1) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cs->solo_grid);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = cs->solo_smem;
    cfg.stream = cs->st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cs->solo.rec[0].p.stamp = prof_stamp(ctx, cs->bf16 ? 1 : 0, cs->ops);
    cs->ops = 0.0;
    cudaError_t le;
    if (cs->bf16) le = cs->solo_grouped ? cudaLaunchKernelEx(&cfg, gemm_kernel<true, true, true, false>, cs->solo)
                                        : cudaLaunchKernelEx(&cfg, gemm_kernel<true, true, false, false>, cs->solo);
    else le = cs->solo_grouped ? cudaLaunchKernelEx(&cfg, gemm_kernel<false, true, true, false>, cs->solo)
                               : cudaLaunchKernelEx(&cfg, gemm_kernel<false, true, false, false>, cs->solo);
    if (le != cudaSuccess) return check_cuda(ctx, le, "gemm launch");
    count_launch(ctx);
    return check_cuda(ctx, cudaGetLastError(), "gemm launch");
  }
  // counters: two per row tile and record, from a region nobody has used since it was cleared
  const int stride = 2 * A.rec[0].p.tiles_m;
  const size_t need = (size_t)n * stride * sizeof(unsigned);
  if (cs->ring_used + need > kFlagRingBytes) {
    // used up (once in a few thousand launches): wait for every launch that may still read it
    cudaError_t me = cudaDeviceSynchronize();
    if (me == cudaSuccess) me = cudaMemsetAsync(cs->ring, 0, kFlagRingBytes, cs->st);
    if (me != cudaSuccess) return check_cuda(ctx, me, "gemm chain counters");
    cs->ring_used = 0;
  }
  A.flags = cs->ring + cs->ring_used / sizeof(unsigned);
  cs->ring_used += need;
  A.flag_stride = stride;
  A.n = n;
  int total = 0;
  for (int i = 0; i < n; ++i) {
    GemmParams& rp = A.rec[i].p;
    total += rp.tiles_m * rp.tiles_n;
    rp.need = 0;
    for (int gi = 0; gi < kMaxGroups; ++gi)
      if (rp.grp[gi].tn_begin != 0x7fffffff && rp.grp[gi].signal) rp.need += rp.grp[gi].gtiles_n;
  }
  A.total_tiles = total;
  A.rec[0].p.stamp = prof_stamp(ctx, cs->bf16 ? 1 : 0, cs->ops);
  cs->ops = 0.0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)cs->grid);
  cfg.blockDim = dim3(kGemmThreads + 64);      // two more warps: one publishes finished tiles, one clears tiles whose inputs are complete
  cfg.dynamicSmemBytes = cs->smem;
  cfg.stream = cs->st;
  cudaLaunchAttribute attr[3];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  attr[2].id = cudaLaunchAttributeCooperative;      // CTAs wait for tiles of other CTAs
  attr[2].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 3;
  const cudaError_t le = cs->bf16 ? cudaLaunchKernelEx(&cfg, gemm_kernel<true, true, true, true>, A)
                                  : cudaLaunchKernelEx(&cfg, gemm_kernel<false, true, true, true>, A);
  A.n = 0;
  if (le == cudaErrorCooperativeLaunchTooLarge || le == cudaErrorNotSupported) {
    // The device cannot keep the whole grid resident right now (or does not take cooperative
    // launches): nothing ran.  The records go out one by one through the ordinary flavour, in
    // their order, and this context stops chaining.
    (void)cudaGetLastError();
    ctx_disable_chains(ctx);
    cudaLaunchConfig_t one = cfg;
    one.blockDim = dim3(kGemmThreads);
    one.numAttrs = 2;
    for (int i = 0; i < n; ++i) {
      memset(&cs->solo, 0, sizeof(cs->solo));
      memcpy(cs->solo.rec[0].m, A.rec[i].m, sizeof(A.rec[i].m));     // pool indices stay valid in the larger pool
      cs->solo.rec[0].p = A.rec[i].p;
      for (int d = 0; d < kMaxDeps; ++d) cs->solo.rec[0].p.deps[d] = -1;
      cs->solo.n = 1;
      cs->solo.total_tiles = A.rec[i].p.tiles_m * A.rec[i].p.tiles_n;
      const cudaError_t se = cs->bf16 ? cudaLaunchKernelEx(&one, gemm_kernel<true, true, true, false>, cs->solo)
                                      : cudaLaunchKernelEx(&one, gemm_kernel<false, true, true, false>, cs->solo);
      if (se != cudaSuccess) return check_cuda(ctx, se, "gemm launch");
      count_launch(ctx);
    }
    return check_cuda(ctx, cudaGetLastError(), "gemm launch");
  }
  if (le != cudaSuccess) return check_cuda(ctx, le, "gemm chain launch");
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "gemm chain launch");
}

int gemm_chain_close(Ctx* ctx) {
  ChainState* cs = static_cast<ChainState*>(chain_slot(ctx));
  if (!cs) return QCFG_OK;
  cs->open = false;
  return gemm_chain_flush(ctx);
}

// After a device-side wait gave up, counters of unfinished launches may be left behind.
int gemm_chain_reset(Ctx* ctx) {
  ChainState* cs = static_cast<ChainState*>(chain_slot(ctx));
  if (!cs) return QCFG_OK;
  cs->args.n = 0;
  cs->ops = 0.0;
  cs->ring_used = 0;
  return check_cuda(ctx, cudaMemset(cs->ring, 0, kFlagRingBytes), "gemm chain counters reset");
}

// Tile width a GEMM of n columns gets.
static int tile_n_of(int64_t n) { return n <= 32 ? 32 : n <= 64 ? 64 : n <= 128 ? 128 : 256; }

bool gemm_groupable(const GemmArgs& a, const GemmArgs& b) {
  if (a.conv_kh > 0 || b.conv_kh > 0) return false;
  return a.m == b.m && a.k == b.k && a.is_bf16 == b.is_bf16 && tile_n_of(a.n) == tile_n_of(b.n);
}

int launch_gemm_group(Ctx* ctx, const GemmArgs* gs_in, int count, cudaStream_t st) {
  if (count < 1 || count > kMaxGroups) return set_error(ctx, QCFG_EINVAL, "gemm: %d groups", count);
  // While launches are being chained a record's tiles run group after group.  Of three groups,
  // those that write operand codes for later layers go in the middle: the group before them gives
  // the previous record time to complete the rows they read, the group after them gives their own
  // rows time to complete before the next record asks for them.  Of two, they go first.
  GemmArgs ordered[kMaxGroups];
  {
    ChainState* st_ = static_cast<ChainState*>(chain_slot(ctx));
    if (st_ && st_->open && count > 1) {
      int feed[kMaxGroups], n_feed = 0, rest[kMaxGroups], n_rest = 0;
      for (int i = 0; i < count; ++i) {
        bool feeds = false;
        for (int s = 0; s < kMaxSlots; ++s) feeds = feeds || gs_in[i].slots[s].kind != 0;
        if (feeds) feed[n_feed++] = i; else rest[n_rest++] = i;
      }
      int k = 0;
      const int before = count == 3 ? (n_rest + 1) / 2 : 0;   // two groups: the feeder first, the other one is the buffer
      for (int i = 0; i < before; ++i) ordered[k++] = gs_in[rest[i]];
      for (int i = 0; i < n_feed; ++i) ordered[k++] = gs_in[feed[i]];
      for (int i = before; i < n_rest; ++i) ordered[k++] = gs_in[rest[i]];
    } else {
      for (int i = 0; i < count; ++i) ordered[i] = gs_in[i];
    }
  }
  const GemmArgs* gs = ordered;
  const GemmArgs& g0 = gs[0];
  const int esz = g0.is_bf16 ? 2 : 1;
  const int bn = tile_n_of(g0.n);
  for (int i = 0; i < count; ++i) {
    const GemmArgs& g = gs[i];
    if (g.m <= 0 || g.n <= 0 || g.k <= 0) return set_error(ctx, QCFG_ESHAPE, "gemm: m, n, k must be positive");
    if (((uintptr_t)g.a & 15) || ((uintptr_t)g.b & 15) || (g.lda * esz) % 16 || (g.ldb * esz) % 16)
      return set_error(ctx, QCFG_EALIGN, "gemm: operands need 16-byte aligned pointers and row strides");
    if (g.conv_kh > 0) {
      if (count > 1) return set_error(ctx, QCFG_EINVAL, "gemm: convolutions are launched alone");
      if ((g.conv_c * esz) % 16 || g.lda != g.conv_c || g.k != (int64_t)g.conv_kh * g.conv_kw * g.conv_c || g.conv_stride < 1)
        return set_error(ctx, QCFG_ESHAPE, "gemm: convolution needs channels in whole 16-byte chunks and k = kh*kw*c");
      if (g.ldb < g.k) return set_error(ctx, QCFG_ESHAPE, "gemm: leading dimension below k");
    } else if (g.lda < g.k || g.ldb < g.k) return set_error(ctx, QCFG_ESHAPE, "gemm: leading dimension below k");
    if (g.m > 0x7fffffff || g.n > 0x7fffffff) return set_error(ctx, QCFG_ESHAPE, "gemm: dimension too large");
    if (i && !gemm_groupable(g0, g)) return set_error(ctx, QCFG_EINVAL, "gemm: grouped launches need equal m, k, type and tile width");
  }

  GemmParams p{};
  p.m = (int32_t)g0.m;
  const int64_t kbytes = g0.k * esz;
  p.k_blocks = (int32_t)((kbytes + kStageKBytes - 1) / kStageKBytes);
  p.bn = bn;
  // pair flavour (two CTAs per 256-row tile, cta_group::2) for wide outputs with at least two
  // row tiles: it halves the B bytes each SM stages per k-block
  const bool pair = ctx_pair_enabled(ctx) && bn == 256 && g0.m > BM && sm_count(ctx) >= 2;
  const int tile_rows = pair ? 2 * BM : BM;
  p.tiles_m = (int32_t)((g0.m + tile_rows - 1) / tile_rows);
  const int stage_bytes = (BM + (pair ? bn / 2 : bn)) * kStageKBytes;
  p.is_bf16 = g0.is_bf16;
  // instruction descriptor: D format (F32 = 1, S32 = 2) at bit 4, A/B format (BF16 = 1, S8 = 1)
  // at bits 7 and 10, both operands K-major, N/8 at bit 17, M/16 at bit 24
  p.idesc = ((g0.is_bf16 ? 1u : 2u) << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(tile_rows >> 4) << 24);
  p.err = err_word(ctx);

  CUtensorMap maps[kPoolAll];      // group i's maps at i * kMapsPerGroup + MAP_*
  memset(maps, 0, sizeof(maps));
  for (int i = 0; i < kMaxGroups; ++i)
    for (int j = 0; j < kMapsPerGroup; ++j) p.mi[i][j] = (uint8_t)(i * kMapsPerGroup + j);
  bool wide = false;
  int32_t tn_total = 0;
  double ops = 0.0;
  for (int i = 0; i < kMaxGroups; ++i) { p.grp[i].tn_begin = 0x7fffffff; p.grp[i].tile_first = 0x7fffffff; p.grp[i].gtiles_n = 1; }
  for (int i = 0; i < count; ++i) {
    const GemmArgs& g = gs[i];
    GroupDesc& G = p.grp[i];
    G.n = (int32_t)g.n;
    G.tn_begin = tn_total;
    G.gtiles_n = (int32_t)((g.n + bn - 1) / bn);
    G.tile_first = p.tiles_m * tn_total;
    tn_total += (int32_t)((g.n + bn - 1) / bn);
    G.scale_x = g.scale_x; G.scale_w = g.scale_w; G.act = g.act;
    G.residual = g.residual; G.ldr = g.ldr;
    G.amax = reinterpret_cast<unsigned*>(g.amax);
    if (g.acc && !g.is_bf16) { G.outs[0].kind = 4; G.outs[0].ptr = g.acc; G.outs[0].ld = g.n; }
    if (g.y) { G.outs[1].kind = 3; G.outs[1].ptr = g.y; G.outs[1].ld = g.ldy; }
    G.need_y = g.y != nullptr || g.amax != nullptr;
    for (int s = 0; s < kMaxSlots; ++s) {
      if (!g.slots[s].kind) continue;
      OutDesc& o = G.outs[2 + s];
      o.kind = g.slots[s].kind; o.ptr = g.slots[s].ptr; o.ld = g.slots[s].ld;
      o.inv_scale = g.slots[s].inv_scale; o.qmax = g.slots[s].qmax;
      G.need_y = 1;
    }
    if (!G.need_y && !G.outs[0].kind) return set_error(ctx, QCFG_EINVAL, "gemm: no output requested");
    if (G.need_y && !g.is_bf16 && !g.scale_w) return set_error(ctx, QCFG_EINVAL, "gemm: scale_w is null");
    for (int j = 0; j < kNumOuts; ++j)
      if (G.outs[j].kind) G.outs[j].tma = make_out_map(&maps[i * kMapsPerGroup + MAP_OUT + j], G.outs[j], g.m, g.n) ? 1 : 0;
    // staging per epilogue warp: two slots of 1 KB when only int8 codes are written, else of 2 KB
    for (int j = 0; j < kNumOuts; ++j) if (G.outs[j].kind >= 2 && G.outs[j].tma) wide = true;
    G.mode = EPI_GENERAL;
    if (bn == 256 && !G.residual && !G.amax && !G.outs[0].kind && !G.outs[3].kind && !G.outs[4].kind) {
      if (!G.outs[1].kind && G.outs[2].kind == 1 && make_fast_map(&maps[i * kMapsPerGroup + MAP_FAST], G.outs[2], g.m, g.n)) G.mode = EPI_CODES1;
      else if (G.outs[1].kind && !G.outs[2].kind && make_fast_map(&maps[i * kMapsPerGroup + MAP_FAST], G.outs[1], g.m, g.n)) { G.mode = EPI_Y; wide = true; }
    }
    int rc = g.conv_kh > 0 ? QCFG_OK : make_map(ctx, &maps[i * kMapsPerGroup + MAP_A], g.a, g.is_bf16, g.k, g.m, g.lda, BM);
    if (rc == QCFG_OK) rc = make_map(ctx, &maps[i * kMapsPerGroup + MAP_B], g.b, g.is_bf16, g.k, g.n, g.ldb, pair ? bn / 2 : bn);
    if (rc != QCFG_OK) return rc;
    ops += 2.0 * (double)g.m * (double)g.n * (double)g.k;
  }
  p.tiles_n = tn_total;
  const bool conv = g0.conv_kh > 0;
  if (conv) {
    ConvDesc& cv = p.conv;
    cv.on = 1; cv.H = g0.conv_h; cv.W = g0.conv_w; cv.C = g0.conv_c; cv.kh = g0.conv_kh; cv.kw = g0.conv_kw;
    cv.stride = g0.conv_stride; cv.pad = g0.conv_pad; cv.esz = esz; cv.K = (int32_t)g0.k;
    cv.OH = (cv.H + 2 * cv.pad - cv.kh) / cv.stride + 1;
    cv.OW = (cv.W + 2 * cv.pad - cv.kw) / cv.stride + 1;
    cv.img_bytes = (int64_t)cv.H * cv.W * cv.C * esz;
    cv.src = reinterpret_cast<const uint8_t*>(g0.a);
    if (cv.OH < 1 || cv.OW < 1 || g0.m % ((int64_t)cv.OH * cv.OW))
      return set_error(ctx, QCFG_ESHAPE, "gemm: convolution rows are not a whole number of images");
  }
  // Launches that may join a chain all take the larger staging size, so any sequence of them
  // shares one shared-memory layout.
  ChainState* cs = static_cast<ChainState*>(chain_slot(ctx));
  // (a GEMM with fewer tiles than CTA pairs has nothing to overlap with: the wait for its
  // producer's rows would cost more than the launch boundary it saves)
  const bool chainable = cs && cs->open && ctx_chain_enabled(ctx) && pair && !conv && bn == 256 && prof_mode(ctx) != 1 && p.tiles_m <= kChainMaxTilesM &&
                         2 * p.tiles_m * p.tiles_n >= sm_count(ctx);
  p.epi_bytes = (wide || chainable) ? 4096 : 2048;
  int stages = (kSmemMax - kSmemHeader - kCsBytes - 1024 - kEpiWarps * p.epi_bytes) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages <= kGatherDepth) return set_error(ctx, QCFG_ESHAPE, "gemm: too few pipeline stages");
  p.stages = stages;

  const int num_tiles = p.tiles_m * p.tiles_n;
  int grid = sm_count(ctx);
  if (pair) {
    int* cached = pair_cluster_cache(ctx) + (g0.is_bf16 ? 1 : 0);
    if (*cached == 0) {     // how many CTA pairs the device keeps resident at once
      cudaLaunchConfig_t q = {};
      q.gridDim = dim3((unsigned)(grid & ~1));
      q.blockDim = dim3(kGemmThreads);
      q.dynamicSmemBytes = kSmemMax;
      cudaLaunchAttribute qa[1];
      qa[0].id = cudaLaunchAttributeClusterDimension;
      qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
      q.attrs = qa; q.numAttrs = 1;
      int n = 0;
      cudaError_t oe = g0.is_bf16 ? cudaOccupancyMaxActiveClusters(&n, gemm_kernel<true, true, true, true>, &q)
                                  : cudaOccupancyMaxActiveClusters(&n, gemm_kernel<false, true, true, true>, &q);
      if (oe != cudaSuccess || n < 1) { (void)cudaGetLastError(); n = grid / 2; }
      if (n > grid / 2) n = grid / 2;
      *cached = n;
    }
    grid = 2 * (*cached);
    if (grid > 2 * num_tiles && !chainable) grid = 2 * num_tiles;
  } else if (grid > num_tiles) grid = num_tiles;
  const size_t smem = (size_t)kSmemHeader + kCsBytes + 1024 + (size_t)kEpiWarps * p.epi_bytes + (size_t)stages * stage_bytes;
  // a chain record carries only the distinct maps it uses; one that needs more runs on its own
  CUtensorMap pool[kPoolChain];
  bool fits = true;
  if (chainable) {
    memset(pool, 0, sizeof(pool));
    int used = 0;
    auto place = [&](int i, int j) {
      const CUtensorMap& mm = maps[i * kMapsPerGroup + j];
      int at = -1;
      for (int u = 0; u < used && at < 0; ++u) if (memcmp(&pool[u], &mm, sizeof(CUtensorMap)) == 0) at = u;
      if (at < 0) {
        if (used == kPoolChain) { fits = false; return; }
        pool[used] = mm; at = used++;
      }
      p.mi[i][j] = (uint8_t)at;
    };
    for (int i = 0; i < kMaxGroups; ++i)
      for (int j = 0; j < kMapsPerGroup; ++j) p.mi[i][j] = 0;
    for (int i = 0; i < count && fits; ++i) {
      place(i, MAP_A);
      place(i, MAP_B);
      if (p.grp[i].mode != EPI_GENERAL) {       // a fast body writes through this one map only
        place(i, MAP_FAST);
        continue;
      }
      for (int j = 0; j < kNumOuts && fits; ++j)
        if (p.grp[i].outs[j].kind && p.grp[i].outs[j].tma) place(i, MAP_OUT + j);
    }
    if (!fits)
      for (int i = 0; i < kMaxGroups; ++i)
        for (int j = 0; j < kMapsPerGroup; ++j) p.mi[i][j] = (uint8_t)(i * kMapsPerGroup + j);
  }
  const bool chained = chainable && fits;
  if (cs && cs->args.n > 0 &&
      (!chained || cs->args.n == kChainMax || cs->st != st || cs->bf16 != (g0.is_bf16 != 0) || cs->grid != grid ||
       cs->smem != smem || cs->m != g0.m)) {
    const int rc = gemm_chain_flush(ctx);
    if (rc != QCFG_OK) return rc;
  }
  if (chained) {
    // What the record reads and writes, as byte ranges.  Reading rows an earlier record of the
    // chain writes is a dependency the kernel waits for; any other overlap ends the chain first.
    ChainRecInfo info{};
    bool b_clash = false;
    auto overlap = [](const Span& x, const Span& y) { return x.lo < y.hi && y.lo < x.hi; };
    auto span_of = [&](const void* ptr, int64_t ld, int64_t cols, int esz_) {
      const uint8_t* lo = static_cast<const uint8_t*>(ptr);
      return Span{lo, lo + ((g0.m - 1) * ld + cols) * esz_};
    };
    for (int i = 0; i < count; ++i) {
      const GemmArgs& g = gs[i];
      info.in[info.n_in++] = span_of(g.a, g.lda, g.k, esz);
      if (g.residual) info.in[info.n_in++] = span_of(g.residual, g.ldr, g.n, 4);
      for (int j = 0; j < kNumOuts; ++j) {
        const OutDesc& o = p.grp[i].outs[j];
        if (o.kind) { info.out_grp[info.n_out] = i; info.out[info.n_out++] = span_of(o.ptr, o.ld, g.n, o.kind == 1 ? 1 : o.kind == 2 ? 2 : 4); }
      }
      // weights and their scales are never chain outputs in a forward pass; if they were, run apart
      const uint8_t* blo = static_cast<const uint8_t*>(g.b);
      const Span bs{blo, blo + ((g.n - 1) * g.ldb + g.k) * esz};
      for (int r = 0; r < cs->args.n; ++r)
        for (int o = 0; o < cs->info[r].n_out; ++o) b_clash = b_clash || overlap(bs, cs->info[r].out[o]);
    }
    int deps[kMaxDeps], n_deps = 0;
    bool read_grp[kChainMax][kMaxGroups] = {};
    bool clash = b_clash;
    for (int r = 0; r < cs->args.n && !clash; ++r) {
      const ChainRecInfo& E = cs->info[r];
      for (int o = 0; o < info.n_out && !clash; ++o) {
        for (int x = 0; x < E.n_in; ++x) clash = clash || overlap(info.out[o], E.in[x]);
        for (int x = 0; x < E.n_out; ++x) clash = clash || overlap(info.out[o], E.out[x]);
      }
      bool reads = false;
      for (int x = 0; x < info.n_in; ++x)
        for (int o = 0; o < E.n_out; ++o)
          if (overlap(info.in[x], E.out[o])) { reads = true; read_grp[r][E.out_grp[o]] = true; }
      if (reads) {
        if (n_deps == kMaxDeps) clash = true;
        else deps[n_deps++] = r;
      }
    }
    if (clash) {
      const int rc = gemm_chain_flush(ctx);
      if (rc != QCFG_OK) return rc;
      n_deps = 0;
    }
    for (int d = 0; d < kMaxDeps; ++d) p.deps[d] = d < n_deps ? deps[d] : -1;
    for (int d = 0; d < n_deps; ++d)
      for (int i = 0; i < kMaxGroups; ++i)
        if (read_grp[deps[d]][i]) cs->args.rec[deps[d]].p.grp[i].signal = 1;
    for (int i = 0; i < kMaxGroups; ++i) p.grp[i].signal = 0;
    p.need = 0;
    p.stamp = nullptr;
    const int slot = cs->args.n++;
    if (slot == 0) {
      GemmParams ps = p;
      for (int i = 0; i < kMaxGroups; ++i)
        for (int j = 0; j < kMapsPerGroup; ++j) ps.mi[i][j] = (uint8_t)(i * kMapsPerGroup + j);
      ps.epi_bytes = wide ? 4096 : 2048;
      int st_solo = (kSmemMax - kSmemHeader - kCsBytes - 1024 - kEpiWarps * ps.epi_bytes) / stage_bytes;
      if (st_solo > kMaxStages) st_solo = kMaxStages;
      ps.stages = st_solo;
      memcpy(cs->solo.rec[0].m, maps, sizeof(maps));
      cs->solo.rec[0].p = ps;
      cs->solo.n = 1; cs->solo.total_tiles = num_tiles; cs->solo.flag_stride = 0; cs->solo.flags = nullptr;
      cs->solo_grid = grid > 2 * num_tiles ? 2 * num_tiles : grid;
      cs->solo_grouped = count > 1 ? 1 : 0;
      cs->solo_smem = (size_t)kSmemHeader + kCsBytes + 1024 + (size_t)kEpiWarps * ps.epi_bytes + (size_t)st_solo * stage_bytes;
    }
    memcpy(cs->args.rec[slot].m, pool, sizeof(pool));
    cs->args.rec[slot].p = p;
    cs->info[slot] = info;
    cs->ops += ops;
    cs->st = st; cs->bf16 = g0.is_bf16 != 0; cs->grid = grid; cs->smem = smem; cs->m = g0.m;
    return QCFG_OK;
  }
  for (int d = 0; d < kMaxDeps; ++d) p.deps[d] = -1;
  // Programmatic dependent launch: the kernel's prologue (barrier set-up, TMEM allocation) may
  // start while the previous kernel in the stream drains; it waits (griddepcontrol.wait) before
  // touching global memory.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(conv ? kGemmThreadsConv : kGemmThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pair ? 2 : 1;
  using Kern = void (*)(const LaunchArgs<false>);
  static const Kern kernels[8] = {
      gemm_kernel<false, false, false, false>, gemm_kernel<false, false, true, false>, gemm_kernel<false, true, false, false>,
      gemm_kernel<false, true, true, false>,   gemm_kernel<true, false, false, false>,  gemm_kernel<true, false, true, false>,
      gemm_kernel<true, true, false, false>,   gemm_kernel<true, true, true, false>};
  const Kern kern = kernels[(g0.is_bf16 ? 4 : 0) + (pair ? 2 : 0) + (count > 1 ? 1 : 0)];
  p.stamp = prof_stamp(ctx, g0.is_bf16 ? 1 : 0, ops);
  static thread_local LaunchArgs<false> one;
  memcpy(one.rec[0].m, maps, sizeof(maps));
  one.rec[0].p = p;
  one.n = 1; one.total_tiles = num_tiles; one.flag_stride = 0; one.flags = nullptr;
  prof_begin(ctx, g0.is_bf16 ? 1 : 0, st);
  const cudaError_t le = cudaLaunchKernelEx(&cfg, kern, one);
  prof_end(ctx, g0.is_bf16 ? 1 : 0, ops, st);
  if (le != cudaSuccess) return check_cuda(ctx, le, "gemm launch");
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "gemm launch");
}

int launch_gemm(Ctx* ctx, const GemmArgs& g, cudaStream_t st) { return launch_gemm_group(ctx, &g, 1, st); }

}  // namespace qcfg
