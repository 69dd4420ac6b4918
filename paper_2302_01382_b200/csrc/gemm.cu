// Quantized GEMM of a configuration evaluation: int8 x int8 -> int32 (tcgen05 kind::i8) and
// bf16 x bf16 -> fp32 (kind::f16) for 16-bit layers, with the dequantize / shortcut /
// activation / re-quantize epilogue fused in (Eq. 1's rescale 2^-(b-1)*gamma for both operands;
// the "Evaluate f(x, w)" step of Algorithms 1 and 2).
//
// Structure (one persistent CTA per SM, 320 threads):
//   warp 0      TMA producer: 128-byte-swizzled K-major tiles of A [128 x 128 B] and
//               B [BN x 128 B] into a ring of shared-memory stages (mbarrier full/empty).
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M=128, N=BN, K=32 B per instruction)
//               from shared-memory descriptors into one of two TMEM accumulator buffers
//               (2 x 256 columns), and commits stage-release / accumulator-ready barriers.
//   warps 2..9  epilogue: tcgen05.ld of the accumulator (one row per thread, 32 columns per
//               load), rescale, shortcut add, activation, stores of fp32 and/or the consumer's
//               int8 / bf16 codes; overlaps the next tile's main loop.
// Every mbarrier wait is bounded: after ~2 s it sets the context's error word and the CTA
// leaves through the normal teardown (TMEM is freed).
#include <cuda.h>

#include "common.cuh"

namespace qcfg {

namespace {

constexpr int BM = 128;               // rows per tile (UMMA M, cta_group::1)
constexpr int kStageKBytes = 128;     // bytes of K per stage row = one 128B swizzle atom
constexpr int kUmmaKBytes = 32;       // bytes of K per tcgen05.mma
constexpr int kEpiWarps = 8;
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;         // columns per accumulator buffer
constexpr int kMaxStages = 8;
constexpr int kSmemHeader = 1024;     // barriers and bookkeeping
constexpr int kSmemMax = 232448;      // 227 KB
constexpr uint64_t kWaitLimitNs = 2000000000ull;

struct GemmParams {
  int32_t m, n, k_blocks, bn, tiles_m, tiles_n, stages, is_bf16;
  uint32_t idesc;
  float scale_x;
  const float* scale_w;
  int32_t act;
  float* y; int64_t ldy;
  const float* residual; int64_t ldr;
  int32_t* acc;
  int32_t need_y;             // anything besides raw accumulators to produce
  CodeSlot slots[kMaxSlots];
  unsigned* err;
};

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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* err) {
  uint64_t t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 0) {
      if (*abort_flag) return false;
      uint64_t now = global_timer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) {
        atomicOr(err, ERR_TIMEOUT);
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
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

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128B swizzle, groups of 8
// rows 1024 bytes apart (the layout a 128B-swizzled TMA box produces).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);          // start address, 16-byte units
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                         // descriptor version for sm_100
  d |= (uint64_t)2 << 61;                         // SWIZZLE_128B
  return d;
}

// ---------------------------------------------------------------------------- epilogue math

__device__ __forceinline__ float gelu_tanh(float y) {
  // y / (1 + exp(-2u)), u = sqrt(2/pi) (y + 0.044715 y^3): equals 0.5 y (1 + tanh u)
  float y2 = y * y;
  float u = 0.7978845608028654f * fmaf(0.044715f * y2, y, y);
  float e = expf(-2.0f * u);
  return y / (1.0f + e);
}
__device__ __forceinline__ float apply_act(float y, int act) {
  if (act == QCFG_ACT_RELU) return fmaxf(y, 0.0f);
  if (act == QCFG_ACT_GELU_TANH) return gelu_tanh(y);
  return y;
}
// int8 code of Eq. 1 in the low byte: clamp, then add 1.5*2^23 (round-half-even at integer
// granularity); the low mantissa byte is the two's-complement code.
__device__ __forceinline__ uint32_t code_byte(float y, float inv_scale, float qmax) {
  float t = __fmul_rn(y, inv_scale);
  t = fminf(fmaxf(t, -qmax), qmax);
  return __float_as_uint(__fadd_rn(t, 12582912.0f)) & 0xffu;
}

// One 32-column chunk of one accumulator row.
template <bool BF16>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& p, uint32_t (&v)[32], int64_t row, int col0) {
  const bool row_ok = row < p.m;
  const int ncols = p.n - col0;                    // valid columns in this chunk (may be <= 0 or > 32)
  if (!row_ok || ncols <= 0) return;
  const bool full = ncols >= 32;

  if (!BF16 && p.acc) {
    int32_t* dst = p.acc + row * (int64_t)p.n + col0;
    if (full && (p.n & 3) == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        reinterpret_cast<uint4*>(dst)[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) if (i < ncols) dst[i] = (int32_t)v[i];
    }
  }

  if (!p.need_y) return;
  float y[32];
  if (BF16) {
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = __uint_as_float(v[i]);
  } else {
    const float* sw = p.scale_w + col0;
    if (full && (((uintptr_t)sw) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float4 s4 = __ldg(reinterpret_cast<const float4*>(sw) + i);
        y[4 * i + 0] = __fmul_rn((float)(int32_t)v[4 * i + 0], __fmul_rn(p.scale_x, s4.x));
        y[4 * i + 1] = __fmul_rn((float)(int32_t)v[4 * i + 1], __fmul_rn(p.scale_x, s4.y));
        y[4 * i + 2] = __fmul_rn((float)(int32_t)v[4 * i + 2], __fmul_rn(p.scale_x, s4.z));
        y[4 * i + 3] = __fmul_rn((float)(int32_t)v[4 * i + 3], __fmul_rn(p.scale_x, s4.w));
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        float s = (i < ncols) ? __ldg(sw + i) : 0.0f;
        y[i] = __fmul_rn((float)(int32_t)v[i], __fmul_rn(p.scale_x, s));
      }
    }
  }
  if (p.residual) {
    const float* r = p.residual + row * p.ldr + col0;
    if (full && (p.ldr & 3) == 0 && (((uintptr_t)p.residual) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float4 r4 = __ldg(reinterpret_cast<const float4*>(r) + i);
        y[4 * i + 0] = __fadd_rn(y[4 * i + 0], r4.x);
        y[4 * i + 1] = __fadd_rn(y[4 * i + 1], r4.y);
        y[4 * i + 2] = __fadd_rn(y[4 * i + 2], r4.z);
        y[4 * i + 3] = __fadd_rn(y[4 * i + 3], r4.w);
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) if (i < ncols) y[i] = __fadd_rn(y[i], __ldg(r + i));
    }
  }
  if (p.act != QCFG_ACT_NONE) {
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = apply_act(y[i], p.act);
  }
  if (p.y) {
    float* dst = p.y + row * p.ldy + col0;
    if (full && (p.ldy & 3) == 0 && (((uintptr_t)p.y) & 15) == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        reinterpret_cast<float4*>(dst)[i] = make_float4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) if (i < ncols) dst[i] = y[i];
    }
  }
#pragma unroll
  for (int s = 0; s < kMaxSlots; ++s) {
    const CodeSlot& sl = p.slots[s];
    if (sl.kind == 1) {
      int8_t* dst = reinterpret_cast<int8_t*>(sl.ptr) + row * sl.ld + col0;
      uint32_t w[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        w[i] = code_byte(y[4 * i], sl.inv_scale, sl.qmax) | (code_byte(y[4 * i + 1], sl.inv_scale, sl.qmax) << 8) |
               (code_byte(y[4 * i + 2], sl.inv_scale, sl.qmax) << 16) | (code_byte(y[4 * i + 3], sl.inv_scale, sl.qmax) << 24);
      }
      if (full) {   // ld is a multiple of 16 and col0 of 32: 16-byte aligned
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
        reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) if (i < ncols) dst[i] = (int8_t)((w[i >> 2] >> (8 * (i & 3))) & 0xff);
      }
    } else if (sl.kind == 2) {
      __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(sl.ptr) + row * sl.ld + col0;
      uint32_t w[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(y[2 * i], y[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
      }
      if (full) {   // ld is a multiple of 8 elements and col0 of 32: 16-byte aligned
#pragma unroll
        for (int i = 0; i < 4; ++i)
          reinterpret_cast<uint4*>(dst)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (i < ncols) reinterpret_cast<uint16_t*>(dst)[i] = (uint16_t)((w[i >> 1] >> (16 * (i & 1))) & 0xffff);
      }
    }
  }
}

// ---------------------------------------------------------------------------- the kernel

template <bool BF16>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment for the 128B swizzle atoms
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);           // full[8] empty[8] tfull[2] tempty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 260);
  uint8_t* stage_base = smem + kSmemHeader;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t stage_bytes = (uint32_t)(BM + p.bn) * kStageKBytes;
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kMaxStages;
  const uint32_t tfull0 = empty0 + 8 * kMaxStages, tempty0 = tfull0 + 16;
  const int num_tiles = p.tiles_m * p.tiles_n;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, kEpiWarps); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
      const int k_elems = BF16 ? kStageKBytes / 2 : kStageKBytes;
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(empty0 + 8 * s, ph ^ 1, abort_flag, p.err)) { ok = false; break; }
          const uint32_t a_dst = smem_u32(stage_base + (size_t)s * stage_bytes);
          const uint32_t b_dst = a_dst + BM * kStageKBytes;
          mbar_expect_tx(full0 + 8 * s, stage_bytes);
          tma_load_2d(a_dst, &map_a, full0 + 8 * s, kb * k_elems, tm * BM);
          tma_load_2d(b_dst, &map_b, full0 + 8 * s, kb * k_elems, tn * p.bn);
          if (++s == p.stages) { s = 0; ph ^= 1; }
        }
      }
      if (!ok) {
        // give copies already in flight a bounded time to land before the CTA exits
        const uint64_t t0 = global_timer();
        while (global_timer() - t0 < 200000ull) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      int t = 0;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
        const int a = t & 1;
        if (!mbar_wait(tempty0 + 8 * a, ((t >> 1) & 1) ^ 1, abort_flag, p.err)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)a * kAccCols;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(full0 + 8 * s, ph, abort_flag, p.err)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(stage_base + (size_t)s * stage_bytes);
          const uint64_t da = smem_desc(a_addr), db = smem_desc(a_addr + BM * kStageKBytes);
#pragma unroll
          for (int k4 = 0; k4 < kStageKBytes / kUmmaKBytes; ++k4) {
            // advancing the start address by 32 bytes (2 units) steps along K inside the swizzle atom
            tc_mma<BF16>(d_tmem, da + (uint64_t)(2 * k4), db + (uint64_t)(2 * k4), p.idesc, (kb | k4) != 0);
          }
          tc_commit(empty0 + 8 * s);          // stage reusable once these MMAs have read it
          if (++s == p.stages) { s = 0; ph ^= 1; }
        }
        if (ok) tc_commit(tfull0 + 8 * a);    // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int ew = warp - 2;
    const int quad = warp & 3;                 // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
    const int half = ew >> 2;                  // interleave 32-column chunks between the two warp sets
    const int chunks = p.bn >> 5;
    bool ok = true;
    int t = 0;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
      const int a = t & 1;
      const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
      if (!mbar_wait(tfull0 + 8 * a, (t >> 1) & 1, abort_flag, p.err)) { ok = false; break; }
      tc_fence_after();
      const int64_t row = (int64_t)tm * BM + quad * 32 + lane;
      for (int c = half; c < chunks; c += 2) {
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(a * kAccCols + c * 32), v);
        epilogue_chunk<BF16>(p, v, row, tn * p.bn + c * 32);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8 * a);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int make_map(Ctx* ctx, CUtensorMap* map, const void* ptr, int is_bf16, int64_t k, int64_t rows, int64_t ld, int box_rows) {
  const int esz = is_bf16 ? 2 : 1;
  cuuint64_t dims[2] = {(cuuint64_t)k, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)(ld * esz)};
  cuuint32_t box[2] = {(cuuint32_t)(kStageKBytes / esz), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
                        const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return set_error(ctx, QCFG_ECUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return QCFG_OK;
}

}  // namespace

int gemm_init(Ctx* ctx) {
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
      return set_error(ctx, QCFG_ECUDA, "cuTensorMapEncodeTiled entry point not found");
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  cudaError_t e = cudaFuncSetAttribute(gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
  return check_cuda(ctx, e, "gemm smem attribute");
}

int launch_gemm(Ctx* ctx, const GemmArgs& g, cudaStream_t st) {
  if (g.m <= 0 || g.n <= 0 || g.k <= 0) return set_error(ctx, QCFG_ESHAPE, "gemm: m, n, k must be positive");
  const int esz = g.is_bf16 ? 2 : 1;
  if (((uintptr_t)g.a & 15) || ((uintptr_t)g.b & 15) || (g.lda * esz) % 16 || (g.ldb * esz) % 16)
    return set_error(ctx, QCFG_EALIGN, "gemm: operands need 16-byte aligned pointers and row strides");
  if (g.lda < g.k || g.ldb < g.k) return set_error(ctx, QCFG_ESHAPE, "gemm: leading dimension below k");
  if (g.m > 0x7fffffff || g.n > 0x7fffffff) return set_error(ctx, QCFG_ESHAPE, "gemm: dimension too large");

  GemmParams p{};
  p.m = (int32_t)g.m; p.n = (int32_t)g.n;
  const int64_t kbytes = g.k * esz;
  p.k_blocks = (int32_t)((kbytes + kStageKBytes - 1) / kStageKBytes);
  int bn = 256;
  if (g.n <= 32) bn = 32; else if (g.n <= 64) bn = 64; else if (g.n <= 128) bn = 128;
  p.bn = bn;
  p.tiles_m = (int32_t)((g.m + BM - 1) / BM);
  p.tiles_n = (int32_t)((g.n + bn - 1) / bn);
  const int stage_bytes = (BM + bn) * kStageKBytes;
  int stages = (kSmemMax - kSmemHeader - 1024) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  p.stages = stages;
  p.is_bf16 = g.is_bf16;
  // instruction descriptor: D format (F32 = 1, S32 = 2) at bit 4, A/B format (BF16 = 1, S8 = 1)
  // at bits 7 and 10, both operands K-major, N/8 at bit 17, M/16 at bit 24
  p.idesc = ((g.is_bf16 ? 1u : 2u) << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
  p.scale_x = g.scale_x; p.scale_w = g.scale_w; p.act = g.act;
  p.y = g.y; p.ldy = g.ldy; p.residual = g.residual; p.ldr = g.ldr; p.acc = g.acc;
  p.need_y = g.y != nullptr;
  for (int s = 0; s < kMaxSlots; ++s) { p.slots[s] = g.slots[s]; if (g.slots[s].kind) p.need_y = 1; }
  if (!p.need_y && !g.acc) return set_error(ctx, QCFG_EINVAL, "gemm: no output requested");
  if (p.need_y && !g.is_bf16 && !g.scale_w) return set_error(ctx, QCFG_EINVAL, "gemm: scale_w is null");
  p.err = err_word(ctx);

  CUtensorMap ma, mb;
  int rc = make_map(ctx, &ma, g.a, g.is_bf16, g.k, g.m, g.lda, BM);
  if (rc == QCFG_OK) rc = make_map(ctx, &mb, g.b, g.is_bf16, g.k, g.n, g.ldb, bn);
  if (rc != QCFG_OK) return rc;

  const int num_tiles = p.tiles_m * p.tiles_n;
  int grid = sm_count(ctx);
  if (grid > num_tiles) grid = num_tiles;
  const size_t smem = (size_t)kSmemHeader + 1024 + (size_t)stages * stage_bytes;
  prof_begin(ctx, g.is_bf16 ? 1 : 0, st);
  if (g.is_bf16) gemm_kernel<true><<<grid, kGemmThreads, smem, st>>>(ma, mb, p);
  else gemm_kernel<false><<<grid, kGemmThreads, smem, st>>>(ma, mb, p);
  prof_end(ctx, g.is_bf16 ? 1 : 0, 2.0 * (double)g.m * (double)g.n * (double)g.k, st);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "gemm launch");
}

}  // namespace qcfg
