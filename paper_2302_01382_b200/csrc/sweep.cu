// Quantization-error sensitivity sweep (Eq. 2 of the paper): for every tensor and every bit
// width b in 2..8 the sum of squared differences between x and Q_b(x), in ONE pass over HBM.
//
// A row (output channel) is held in registers by a team of 32..256 threads: the row maximum,
// the 7 scale pairs and the 7 error sums all come from those registers, so every weight is
// read from HBM exactly once.  Per element and bit width the work is four FMA-pipe ops:
//   u = fma(x, inv_scale, 1.5*2^23)   (round-half-even of x*inv_scale in the low mantissa bits)
//   r = u - 1.5*2^23                  (the code as a float)
//   e = fma(-scale, r, x)             (x - Q(x))
//   acc = fma(e, e, acc)
// The clip of Eq. 1 is a no-op here because the scale comes from the row's own maximum.
//
// Work distribution: the tensors of one kernel variant form one flat sequence of rows, cut into as
// many equal pieces as blocks stay resident on the device (three per SM); a piece that crosses a
// tensor boundary becomes several segments.  Every block therefore starts once, streams the same
// amount of data and ends with the others: no per-item start-up cost and no ragged last wave.
// Each segment writes its 7 sums and its maximum to its own slot; one finalize block per tensor
// adds the tensor's slots in a fixed order, so the result does not depend on timing.
//
// Sums: fp32 in three short stages, then fp64.  A thread's packed accumulators take at most
// kChainTerms squared errors each; they are then added into a second fp32 accumulator per bit width,
// which takes at most kChainTerms such sums; that one is reduced over the warp by five pairwise
// steps and added to the warp's fp64 sum in shared memory.  A sequential fp32 sum of n non-negative
// terms is within (n-1)*2^-24 relative of the exact sum, so the three stages together stay within
// (31 + 1 + 31 + 5) * 2^-24 = 4.1e-6, inside the sweep's 1e-5 tolerance; no thread keeps fp64
// accumulators in registers.
#include <cstring>

#include "common.cuh"

namespace qcfg {

namespace {

constexpr int kThreads = 256;
constexpr int kNB = 7;                       // bit widths 2..8
constexpr float kMagic = 12582912.0f;        // 1.5 * 2^23
constexpr int kRing = 3;                     // shared-memory row stages per thread
constexpr int kBlocksPerSM = 3;
constexpr int kChainTerms = 32;              // terms per fp32 accumulator at each of the two stages
constexpr int64_t kMinBlockElems = 16 * 1024;   // do not cut the work of a variant finer than this

// One run of whole rows of one tensor, processed by one block.
struct SweepSeg {
  const float* w;         // first row of the run
  int32_t rows;
  int32_t cols;
  int32_t tensor;         // index into the caller's tensor list
  int32_t team_log2;      // team size = 32 << team_log2 (row variants)
  int32_t slot;           // partial-result slot
  int32_t pad;
};
struct SweepBlock { int32_t seg0, nseg; };
struct TensorSlots { int32_t slot0, slot1; };

__device__ __forceinline__ void scales_for_lane(float A, int lane, float& s, float& inv) {
  int b = 2 + (lane % kNB);
  float qm = (float)((1 << (b - 1)) - 1);
  s = 1.0f; inv = 1.0f;
  if (A != 0.0f) { s = __fdiv_rn(A, qm); inv = __fdiv_rn(qm, A); }
}

__device__ __forceinline__ void err4(float x, float s, float inv, float& acc) {
  float u = fmaf(x, inv, kMagic);
  float r = u - kMagic;
  float e = fmaf(-s, r, x);
  acc = fmaf(e, e, acc);
}

// Writes the block's 7 sums and its maximum to out[0..7].  Ends with a barrier, so the shared
// buffer may be reused at once.
__device__ __forceinline__ void block_reduce_store(double (&dacc)[kNB], float amax, double* __restrict__ out) {
  __shared__ double sred[kThreads / 32][8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int j = 0; j < kNB; ++j) {
    double v = warp_sum(dacc[j]);
    if (lane == 0) sred[warp][j] = v;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if (lane == 0) sred[warp][7] = (double)amax;
  __syncthreads();
  if (threadIdx.x < 8) {
    double v = sred[0][threadIdx.x];
    for (int w = 1; w < kThreads / 32; ++w)
      v = (threadIdx.x == 7) ? fmax(v, sred[w][7]) : v + sred[w][threadIdx.x];
    out[threadIdx.x] = v;
  }
  __syncthreads();
}

// Two elements per instruction: the four operations of one (element, b) evaluation as packed
// fp32 arithmetic (sm_100 fma.rn.f32x2 / add.rn.f32x2), which halves the issue slots they need.
// ns holds the negated scale in both halves.
__device__ __forceinline__ void err8(float2 x, float2 ns, float2 inv, float2& acc) {
  const float2 magic = make_float2(kMagic, kMagic), nmagic = make_float2(-kMagic, -kMagic);
  float2 u = __ffma2_rn(x, inv, magic);
  float2 r = __fadd2_rn(u, nmagic);
  float2 e = __ffma2_rn(ns, r, x);
  acc = __ffma2_rn(e, e, acc);
}

// Rows of up to 32*V*team float4; cols % 4 == 0 and 16-byte aligned rows.  All 7 bit widths are
// always evaluated (a narrower request only selects columns in the finalize kernel).
template <int V>
__global__ void __launch_bounds__(kThreads, kBlocksPerSM)
sweep_rows_kernel(const SweepSeg* __restrict__ segs, const SweepBlock* __restrict__ blocks, int per_tensor,
                  const float* __restrict__ tensor_absmax, double* __restrict__ partial) {
  // rows between two first-stage flushes: every row adds 2*V terms to each half of a packed accumulator
  constexpr int kFlushRows = (kChainTerms / (2 * V)) > 0 ? (kChainTerms / (2 * V)) : 1;
  // Programmatic dependent launch: the block is scheduled while the previous kernel of the stream
  // drains and waits here for that kernel's results (result slots, per-tensor maxima, and whatever
  // produced the weights).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const SweepBlock blk = blocks[blockIdx.x];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __shared__ float smax2[2][kThreads / 32];
  __shared__ double swarp[kThreads / 32][8];             // per warp: 7 fp64 sums and the maximum
  extern __shared__ float4 ring[];                       // [kRing][V][kThreads]

  for (int si = blk.seg0; si < blk.seg0 + blk.nseg; ++si) {
    const SweepSeg d = segs[si];
    const int T = 32 << d.team_log2;
    const int nteams = kThreads / T;
    const int team = threadIdx.x / T;
    const int tl = threadIdx.x % T;
    const int c4 = d.cols >> 2;
    const int n_iter = (d.rows + nteams - 1) / nteams;
    const float A_tensor = per_tensor ? tensor_absmax[d.tensor] : 0.0f;
    int row_parity = 0;

    float2 facc[kNB];
    float f2[kNB];
#pragma unroll
    for (int j = 0; j < kNB; ++j) { facc[j] = make_float2(0.0f, 0.0f); f2[j] = 0.0f; }
    if (lane < 8) swarp[warp][lane] = 0.0;
    float amax_blk = 0.0f;

    auto process_row = [&](const float4 (&cur)[V]) {
      float m = 0.0f;
#pragma unroll
      for (int v = 0; v < V; ++v)
        m = fmaxf(fmaxf(fmaxf(m, fabsf(cur[v].x)), fmaxf(fabsf(cur[v].y), fabsf(cur[v].z))), fabsf(cur[v].w));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (T > 32) {
        // the team's warps exchange their maxima through shared memory; a named barrier per team
        // keeps other teams running, and alternating slots make one barrier per row enough
        float* slot = smax2[row_parity];
        if (lane == 0) slot[warp] = m;
        asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(T) : "memory");
        const int w0 = team * (T >> 5);
        m = slot[w0];
        for (int w = 1; w < (T >> 5); ++w) m = fmaxf(m, slot[w0 + w]);
        row_parity ^= 1;
      }
      amax_blk = fmaxf(amax_blk, m);
      if (per_tensor) m = A_tensor;

      // the 7 scale pairs: two IEEE divisions in lanes 0..6, broadcast by shuffles
      float s_l, inv_l;
      scales_for_lane(m, lane, s_l, inv_l);
      float2 ns[kNB], inv[kNB];
#pragma unroll
      for (int j = 0; j < kNB; ++j) {
        const float sj = -__shfl_sync(0xffffffffu, s_l, j), ij = __shfl_sync(0xffffffffu, inv_l, j);
        ns[j] = make_float2(sj, sj);
        inv[j] = make_float2(ij, ij);
      }
#pragma unroll
      for (int v = 0; v < V; ++v) {
        const float2 lo = make_float2(cur[v].x, cur[v].y), hi = make_float2(cur[v].z, cur[v].w);
#pragma unroll
        for (int j = 0; j < kNB; ++j) {
          err8(lo, ns[j], inv[j], facc[j]);
          err8(hi, ns[j], inv[j], facc[j]);
        }
      }
    };
    // second stage -> the warp's fp64 sums
    auto flush2 = [&]() {
#pragma unroll
      for (int j = 0; j < kNB; ++j) {
        float v = f2[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) swarp[warp][j] += (double)v;
        f2[j] = 0.0f;
      }
    };

    // Rows stream through a three-stage ring in shared memory filled by cp.async, two rows ahead
    // of the one being processed: enough loads in flight to cover HBM latency without holding
    // future rows in registers.  Every thread copies and reads back only its own 16-byte slots, so
    // no barrier is needed between the copy and the read.
    // rowp: this thread's first float4 of the next row its team fetches; fetch_row: that row's index
    const float4* rowp = reinterpret_cast<const float4*>(d.w + (int64_t)team * d.cols) + tl;
    const int64_t row_step4 = (int64_t)nteams * c4;
    int fetch_row = team;
    const uint32_t ring0 = (uint32_t)__cvta_generic_to_shared(ring + threadIdx.x);
    auto issue_row = [&](int stage) {
      const uint32_t dst0 = ring0 + (uint32_t)(stage * V) * (kThreads * 16);
      const bool row_ok = fetch_row < d.rows;
#pragma unroll
      for (int v = 0; v < V; ++v) {
        const uint32_t dst = dst0 + v * (kThreads * 16);
        if (row_ok && tl + v * T < c4) {
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(rowp + v * T) : "memory");
        } else {
          asm volatile("st.shared.v4.f32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "f"(0.0f) : "memory");
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      rowp += row_step4;
      fetch_row += nteams;
    };
    issue_row(0);
    issue_row(1);
    int stage = 0, n1 = 0, n2 = 0;
    for (int it = 0; it < n_iter; ++it) {
      int nxt = stage + 2; if (nxt >= kRing) nxt -= kRing;
      issue_row(nxt);                                                 // zeros past the end
      asm volatile("cp.async.wait_group 2;" ::: "memory");            // the row of this iteration has landed
      float4 cur[V];
#pragma unroll
      for (int v = 0; v < V; ++v) cur[v] = ring[(stage * V + v) * kThreads + threadIdx.x];
      process_row(cur);
      if (++n1 == kFlushRows) {
#pragma unroll
        for (int j = 0; j < kNB; ++j) { f2[j] += facc[j].x + facc[j].y; facc[j] = make_float2(0.0f, 0.0f); }
        n1 = 0;
        if (++n2 == kChainTerms - 1) { flush2(); n2 = 0; }
      }
      if (++stage == kRing) stage = 0;
    }
#pragma unroll
    for (int j = 0; j < kNB; ++j) f2[j] += facc[j].x + facc[j].y;
    flush2();
    asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax_blk = fmaxf(amax_blk, __shfl_xor_sync(0xffffffffu, amax_blk, o));
    if (lane == 0) swarp[warp][7] = (double)amax_blk;
    __syncthreads();
    if (threadIdx.x < 8) {                  // the warps' sums in a fixed order
      double v = swarp[0][threadIdx.x];
      for (int w = 1; w < kThreads / 32; ++w)
        v = (threadIdx.x == 7) ? fmax(v, swarp[w][7]) : v + swarp[w][threadIdx.x];
      partial[(int64_t)d.slot * 8 + threadIdx.x] = v;
    }
    __syncthreads();
  }
}

// Any shape or alignment: the whole block works on one row at a time and reads it twice
// (the second read hits L1/L2).
__global__ void __launch_bounds__(kThreads)
sweep_generic_kernel(const SweepSeg* __restrict__ segs, const SweepBlock* __restrict__ blocks, int per_tensor,
                     const float* __restrict__ tensor_absmax, int jlo, int jhi, double* __restrict__ partial) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const SweepBlock blk = blocks[blockIdx.x];
  const int lane = threadIdx.x & 31;
  __shared__ float smax[kThreads / 32];
  for (int si = blk.seg0; si < blk.seg0 + blk.nseg; ++si) {
    const SweepSeg d = segs[si];
    const float A_tensor = per_tensor ? tensor_absmax[d.tensor] : 0.0f;
    double dacc[kNB];
#pragma unroll
    for (int j = 0; j < kNB; ++j) dacc[j] = 0.0;
    float amax_blk = 0.0f;
    for (int row = 0; row < d.rows; ++row) {
      const float* p = d.w + (int64_t)row * d.cols;
      float m = 0.0f;
      for (int c = threadIdx.x; c < d.cols; c += kThreads) m = fmaxf(m, fabsf(__ldg(p + c)));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (lane == 0) smax[threadIdx.x >> 5] = m;
      __syncthreads();
      m = smax[0];
      for (int w = 1; w < kThreads / 32; ++w) m = fmaxf(m, smax[w]);
      __syncthreads();
      amax_blk = fmaxf(amax_blk, m);
      if (per_tensor) m = A_tensor;
      float s_l, inv_l;
      scales_for_lane(m, lane, s_l, inv_l);
      float s[kNB], inv[kNB], facc[kNB];
#pragma unroll
      for (int j = 0; j < kNB; ++j) {
        s[j] = __shfl_sync(0xffffffffu, s_l, j);
        inv[j] = __shfl_sync(0xffffffffu, inv_l, j);
        facc[j] = 0.0f;
      }
      int terms = 0;
      for (int c = threadIdx.x; c < d.cols; c += kThreads) {
        float x = __ldg(p + c);
#pragma unroll
        for (int j = 0; j < kNB; ++j)
          if (j >= jlo && j <= jhi) err4(x, s[j], inv[j], facc[j]);
        if (++terms == kChainTerms) {            // very long rows: keep the fp32 chains short
#pragma unroll
          for (int j = 0; j < kNB; ++j) { dacc[j] += (double)facc[j]; facc[j] = 0.0f; }
          terms = 0;
        }
      }
#pragma unroll
      for (int j = 0; j < kNB; ++j) dacc[j] += (double)facc[j];
    }
    block_reduce_store(dacc, amax_blk, partial + (int64_t)d.slot * 8);
  }
}

// One block per tensor: 32 groups of 8 threads stride over the tensor's slots (thread j of a group
// owns column j: 7 sums and the maximum), then thread j < 8 combines the 32 group results in a
// fixed order.
__global__ void __launch_bounds__(256)
sweep_finalize_kernel(const double* __restrict__ partial, const TensorSlots* __restrict__ ts, int jlo, int nb,
                      double* __restrict__ sse, float* __restrict__ absmax, int write_absmax) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the slots come from the kernels before
  __shared__ double sm[32][8];
  const int t = blockIdx.x;
  const int j = threadIdx.x & 7, g = threadIdx.x >> 3;
  const TensorSlots r = ts[t];
  double v = 0.0;
  for (int i = r.slot0 + g; i < r.slot1; i += 32) {
    const double x = partial[(int64_t)i * 8 + j];
    v = (j == 7) ? fmax(v, x) : v + x;
  }
  sm[g][j] = v;
  __syncthreads();
  if (threadIdx.x < 8) {
    double a = sm[0][j];
    for (int k = 1; k < 32; ++k) a = (j == 7) ? fmax(a, sm[k][j]) : a + sm[k][j];
    if (j == 7) {
      if (write_absmax) absmax[t] = (float)a;
    } else if (j >= jlo && j < jlo + nb) {
      sse[(int64_t)t * nb + (j - jlo)] = a;
    }
  }
}

// Launch configuration with programmatic stream serialization: the kernel may start while its
// predecessor in the stream drains; it orders itself with griddepcontrol.wait.
cudaLaunchAttribute g_pdl_attr;
inline cudaLaunchConfig_t pdl_config(int blocks, int threads, size_t smem, cudaStream_t st) {
  g_pdl_attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  g_pdl_attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = &g_pdl_attr;
  cfg.numAttrs = 1;
  return cfg;
}

template <int V>
void launch_rows(const SweepSeg* segs, const SweepBlock* blocks, int n_blocks, int per_tensor, const float* amax,
                 double* partial, cudaStream_t st) {
  constexpr size_t smem = (size_t)kRing * V * kThreads * sizeof(float4);
  cudaLaunchConfig_t cfg = pdl_config(n_blocks, kThreads, smem, st);
  cudaLaunchKernelEx(&cfg, sweep_rows_kernel<V>, segs, blocks, per_tensor, amax, partial);
}

template <int V>
cudaError_t set_rows_smem() {
  return cudaFuncSetAttribute(sweep_rows_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)((size_t)kRing * V * kThreads * sizeof(float4)));
}

// ------------------------------------------------------------------ planning (host)

constexpr int kClasses = 9;                  // 0 = generic kernel, V = 1..8 = row kernel variants

// Capacity of the tables a plan is written into.  Segments never exceed blocks + tensors.
struct PlanTables {
  SweepSeg* segs; int max_segs;
  SweepBlock* blocks; int max_blocks;
  TensorSlots* slots; int max_tensors;
};
struct Plan {
  int n_segs = 0, n_blocks = 0;
  int class_block0[kClasses], class_blocks[kClasses];
};

// Kernel variant and team size of a tensor.
inline int classify(const float* w, int64_t cols, int* team_log2) {
  *team_log2 = 0;
  const bool vec = ((uintptr_t)w % 16 == 0) && (cols % 4 == 0) && cols <= 8192 && cols > 0;
  if (!vec) return 0;
  const int64_t c4 = cols / 4;
  int tl = 0;
  while (tl < 3 && c4 > (int64_t)(32 << tl) * 8) ++tl;
  *team_log2 = tl;
  return (int)((c4 + (32 << tl) - 1) / (32 << tl));     // float4 per thread, 1..8
}

// Cuts every variant's rows into equal pieces, one per block.  Returns false when a table is too
// small.  Segments of one tensor get consecutive slots.
bool plan_sweep(const float* const* w, const int64_t* rows, const int64_t* cols, int32_t n_tensors, int sms,
                const PlanTables& T, Plan* P) {
  if (n_tensors > T.max_tensors) return false;
  const int resident = sms * kBlocksPerSM;
  for (int t = 0; t < n_tensors; ++t)      // tensors without elements keep an empty slot range
    T.slots[t].slot0 = T.slots[t].slot1 = 0;
  for (int c = 0; c < kClasses; ++c) {
    P->class_block0[c] = P->n_blocks;
    P->class_blocks[c] = 0;
    int64_t total = 0;
    int tl;
    for (int t = 0; t < n_tensors; ++t)
      if (classify(w[t], cols[t], &tl) == c) total += rows[t] * cols[t];
    if (total == 0) continue;
    int64_t nblk = (total + kMinBlockElems - 1) / kMinBlockElems;
    if (nblk > resident) nblk = resident;
    if (P->n_blocks + nblk > T.max_blocks) return false;
    const int64_t quota = (total + nblk - 1) / nblk;           // elements per block
    int blk = P->n_blocks;
    const int blk_last = P->n_blocks + (int)nblk - 1;
    int64_t room = quota;
    T.blocks[blk].seg0 = P->n_segs; T.blocks[blk].nseg = 0;
    for (int t = 0; t < n_tensors; ++t) {
      if (rows[t] * cols[t] == 0 || classify(w[t], cols[t], &tl) != c) continue;
      T.slots[t].slot0 = P->n_segs;
      int64_t row = 0;
      while (row < rows[t]) {
        int64_t take = (room + cols[t] - 1) / cols[t];         // whole rows filling the block's quota
        if (c > 0) {                                            // whole rounds of the block's teams
          const int64_t nt = kThreads / (32 << tl);
          take = (take + nt - 1) / nt * nt;
        }
        if (blk == blk_last) take = rows[t] - row;              // the last block takes what is left
        if (take < 1) take = 1;
        if (take > rows[t] - row) take = rows[t] - row;
        if (take > 0x7fffffff) take = 0x7fffffff;
        if (P->n_segs >= T.max_segs) return false;
        SweepSeg& s = T.segs[P->n_segs];
        s.w = w[t] + row * cols[t]; s.rows = (int32_t)take; s.cols = (int32_t)cols[t]; s.tensor = t;
        s.team_log2 = tl; s.slot = P->n_segs; s.pad = 0;
        P->n_segs++;
        T.blocks[blk].nseg++;
        row += take;
        room -= take * cols[t];
        if (room <= 0 && blk < blk_last) {
          ++blk;
          T.blocks[blk].seg0 = P->n_segs; T.blocks[blk].nseg = 0;
          room = quota;
        }
      }
      T.slots[t].slot1 = P->n_segs;
    }
    // blocks left without a segment are not launched
    const int used = blk - P->n_blocks + (T.blocks[blk].nseg > 0 ? 1 : 0);
    P->class_blocks[c] = used;
    P->n_blocks += used;
  }
  return true;
}

// Enqueues the sweep's kernels for a plan whose tables are on the device already.
int run_plan(Ctx* ctx, const Plan& P, const SweepSeg* segs, const SweepBlock* blocks, const TensorSlots* slots,
             double* partial, const float* const* w, const int64_t* rows, const int64_t* cols, int32_t n_tensors,
             int per_tensor, int b_lo, int b_hi, double* sse, float* absmax, cudaStream_t st) {
  if (per_tensor) {
    for (int t = 0; t < n_tensors; ++t) {
      int rc = launch_absmax(ctx, w[t], rows[t], cols[t], cols[t], QCFG_PER_TENSOR, absmax + t, st);
      if (rc != QCFG_OK) return rc;
    }
  }
  const int jlo = b_lo - 2, jhi = b_hi - 2, nb = b_hi - b_lo + 1;
  for (int c = 0; c < kClasses; ++c) {
    const int n = P.class_blocks[c];
    if (n == 0) continue;
    const SweepBlock* b = blocks + P.class_block0[c];
    prof_begin(ctx, 2, st);
    switch (c) {
      case 0: {
        cudaLaunchConfig_t cfg = pdl_config(n, kThreads, 0, st);
        cudaLaunchKernelEx(&cfg, sweep_generic_kernel, segs, b, per_tensor, (const float*)absmax, jlo, jhi, partial);
        break;
      }
      case 1: launch_rows<1>(segs, b, n, per_tensor, absmax, partial, st); break;
      case 2: launch_rows<2>(segs, b, n, per_tensor, absmax, partial, st); break;
      case 3: launch_rows<3>(segs, b, n, per_tensor, absmax, partial, st); break;
      case 4: launch_rows<4>(segs, b, n, per_tensor, absmax, partial, st); break;
      case 5: launch_rows<5>(segs, b, n, per_tensor, absmax, partial, st); break;
      case 6: launch_rows<6>(segs, b, n, per_tensor, absmax, partial, st); break;
      case 7: launch_rows<7>(segs, b, n, per_tensor, absmax, partial, st); break;
      default: launch_rows<8>(segs, b, n, per_tensor, absmax, partial, st); break;
    }
    prof_end(ctx, 2, 0.0, st);
    count_launch(ctx);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return check_cuda(ctx, e, "sweep launch");
  }
  {
    cudaLaunchConfig_t cfg = pdl_config(n_tensors, 256, 0, st);
    cudaLaunchKernelEx(&cfg, sweep_finalize_kernel, (const double*)partial, slots, jlo, nb, sse, absmax, per_tensor ? 0 : 1);
  }
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "sweep finalize launch");
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

// The shared-memory opt-in of a kernel is a per-device attribute: set for every variant whenever a
// context is created (the context's device is current then).
int sweep_init(Ctx* ctx) {
  cudaError_t e = set_rows_smem<1>();
  if (e == cudaSuccess) e = set_rows_smem<2>();
  if (e == cudaSuccess) e = set_rows_smem<3>();
  if (e == cudaSuccess) e = set_rows_smem<4>();
  if (e == cudaSuccess) e = set_rows_smem<5>();
  if (e == cudaSuccess) e = set_rows_smem<6>();
  if (e == cudaSuccess) e = set_rows_smem<7>();
  if (e == cudaSuccess) e = set_rows_smem<8>();
  return check_cuda(ctx, e, "sweep smem attribute");
}

int launch_sweep(Ctx* ctx, const float* const* w, const int64_t* rows, const int64_t* cols, int32_t n_tensors,
                 int granularity, int b_lo, int b_hi, double* sse, float* absmax, cudaStream_t st) {
  if (n_tensors == 0) return QCFG_OK;
  const int resident = sm_count(ctx) * kBlocksPerSM;
  const int max_blocks = kClasses * resident, max_segs = max_blocks + n_tensors;
  // host tables in one context-owned buffer: segments | blocks | tensor slot ranges
  const size_t seg_bytes = align_up((size_t)max_segs * sizeof(SweepSeg), 16);
  const size_t blk_bytes = align_up((size_t)max_blocks * sizeof(SweepBlock), 16);
  const size_t slot_bytes = align_up((size_t)n_tensors * sizeof(TensorSlots), 16);
  const size_t table_bytes = seg_bytes + blk_bytes + slot_bytes;
  char* host = static_cast<char*>(host_scratch(ctx, table_bytes));
  if (!host) return set_error(ctx, QCFG_ENOMEM, "sweep: host tables");
  memset(host, 0, table_bytes);
  PlanTables T{reinterpret_cast<SweepSeg*>(host), max_segs, reinterpret_cast<SweepBlock*>(host + seg_bytes), max_blocks,
               reinterpret_cast<TensorSlots*>(host + seg_bytes + blk_bytes), n_tensors};
  Plan P;
  if (!plan_sweep(w, rows, cols, n_tensors, sm_count(ctx), T, &P)) return set_error(ctx, QCFG_EINVAL, "sweep: planning failed");

  // device scratch: partials | the same three tables
  const size_t partial_bytes = align_up((size_t)(max_segs > 0 ? max_segs : 1) * 8 * sizeof(double), 256);
  char* base = static_cast<char*>(scratch(ctx, partial_bytes + table_bytes));
  if (!base) return set_error(ctx, QCFG_ENOMEM, "sweep scratch (%zu bytes)", partial_bytes + table_bytes);
  char* tab = base + partial_bytes;
  // the tables only depend on the tensor list: a repeated sweep of the same tensors (same scratch
  // buffer) finds them on the device already
  if (!sweep_tables_cached(ctx, base, st, host, table_bytes, nullptr, 0)) {
    const cudaError_t e = cudaMemcpyAsync(tab, host, table_bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "sweep table upload");
  }
  return run_plan(ctx, P, reinterpret_cast<const SweepSeg*>(tab), reinterpret_cast<const SweepBlock*>(tab + seg_bytes),
                  reinterpret_cast<const TensorSlots*>(tab + seg_bytes + blk_bytes), reinterpret_cast<double*>(base), w, rows,
                  cols, n_tensors, granularity == QCFG_PER_TENSOR, b_lo, b_hi, sse, absmax, st);
}


// ------------------------------------------------------------------ sweep without allocation
//
// Same sweep, for callers that must not allocate device memory at call time: the segment
// partials and the tables live in a fixed device array that is part of the loaded library image
// (about 0.6 MiB on every GPU that loads the library, until the process exits).

constexpr int kStaticMaxTensors = 1024;
constexpr int kStaticMaxBlocks = 4096;                                  // 9 variants x 3 blocks x up to 151 SMs
constexpr int kStaticMaxSegs = kStaticMaxBlocks + kStaticMaxTensors;
constexpr int64_t kStaticMaxElems = (int64_t)1 << 35;                   // elements per call

struct StaticSweepScratch {
  double partial[kStaticMaxSegs * 8];
  SweepSeg segs[kStaticMaxSegs];
  SweepBlock blocks[kStaticMaxBlocks];
  TensorSlots slots[kStaticMaxTensors];
};

static __device__ __align__(256) unsigned char g_static_sweep_scratch[sizeof(StaticSweepScratch)];

// Device address of the array above, per device ordinal.  In host code the array's name is only a
// handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress, asked
// once per device while that device is current.
constexpr int kMaxDevices = 64;
static void* g_static_sweep_addr[kMaxDevices] = {nullptr};

int launch_sweep_static(Ctx* ctx, const float* const* w, const int64_t* rows, const int64_t* cols,
                        int32_t n_tensors, int granularity, int b_lo, int b_hi, double* sse, float* absmax,
                        cudaStream_t st) {
  if (n_tensors == 0) return QCFG_OK;
  if (n_tensors > kStaticMaxTensors)
    return set_error(ctx, QCFG_ENOMEM, "static sweep: %d tensors exceed the fixed scratch (at most %d per call)",
                     n_tensors, kStaticMaxTensors);
  int64_t total = 0;
  for (int t = 0; t < n_tensors; ++t) {
    if (rows[t] > kStaticMaxElems || (cols[t] > 0 && rows[t] > kStaticMaxElems / cols[t])) total = kStaticMaxElems + 1;
    else total += rows[t] * cols[t];
    if (total > kStaticMaxElems)
      return set_error(ctx, QCFG_ENOMEM, "static sweep: more than 2^35 elements in one call; split the tensors over several calls");
  }
  if (kClasses * sm_count(ctx) * kBlocksPerSM > kStaticMaxBlocks)
    return set_error(ctx, QCFG_ENOMEM, "static sweep: the device has more SMs than the fixed tables are sized for");

  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return check_cuda(ctx, e, "static sweep: cudaGetDevice");
  if (dev != device_of(ctx) || dev < 0 || dev >= kMaxDevices)
    return set_error(ctx, QCFG_ESTATE, "static sweep: the context's device (%d) must be the current device (%d)",
                     device_of(ctx), dev);
  if (!g_static_sweep_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_sweep_scratch);
    if (e != cudaSuccess || !p) return check_cuda(ctx, e == cudaSuccess ? cudaErrorInvalidSymbol : e, "static sweep: cudaGetSymbolAddress");
    g_static_sweep_addr[dev] = p;
  }
  StaticSweepScratch* S = static_cast<StaticSweepScratch*>(g_static_sweep_addr[dev]);

  // the plan is written into a host buffer the context owns (no large arrays on the caller's stack)
  const size_t seg_bytes = sizeof(S->segs), blk_bytes = sizeof(S->blocks), slot_bytes = sizeof(S->slots);
  char* host = static_cast<char*>(host_scratch(ctx, seg_bytes + blk_bytes + slot_bytes));
  if (!host) return set_error(ctx, QCFG_ENOMEM, "static sweep: host tables");
  PlanTables T{reinterpret_cast<SweepSeg*>(host), kStaticMaxSegs, reinterpret_cast<SweepBlock*>(host + seg_bytes), kStaticMaxBlocks,
               reinterpret_cast<TensorSlots*>(host + seg_bytes + blk_bytes), kStaticMaxTensors};
  Plan P;
  if (!plan_sweep(w, rows, cols, n_tensors, sm_count(ctx), T, &P))
    return set_error(ctx, QCFG_ENOMEM, "static sweep: the plan does not fit the fixed tables");

  // Every segment overwrites all 8 values of its own slot and the finalize kernel reads only the
  // slots of this call, so nothing left in the array by an earlier call needs clearing.  The copies
  // come from pageable host memory, so they have left the host buffer when the calls return.
  e = cudaMemcpyAsync(S->segs, T.segs, (size_t)P.n_segs * sizeof(SweepSeg), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(S->blocks, T.blocks, (size_t)P.n_blocks * sizeof(SweepBlock), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(S->slots, T.slots, (size_t)n_tensors * sizeof(TensorSlots), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return check_cuda(ctx, e, "static sweep: table upload");
  return run_plan(ctx, P, S->segs, S->blocks, S->slots, S->partial, w, rows, cols, n_tensors,
                  granularity == QCFG_PER_TENSOR, b_lo, b_hi, sse, absmax, st);
}

}  // namespace qcfg
