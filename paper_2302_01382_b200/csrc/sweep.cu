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
// Sums are fp32 within one row per thread, fp64 across rows, and reduced in a fixed order
// (block partials in scratch memory, then one finalize block per tensor): deterministic.
#include <vector>

#include "common.cuh"

namespace qcfg {

namespace {

constexpr int kThreads = 256;
constexpr int kNB = 7;                       // bit widths 2..8
constexpr float kMagic = 12582912.0f;        // 1.5 * 2^23
constexpr int kRing = 3;                     // shared-memory row stages per thread
constexpr int kItemFloatsMin = 8 * 1024;     // elements per work item (one block): bounds
constexpr int kItemFloatsMax = 256 * 1024;

// Work-item size for a call: about eight items per SM (two resident blocks, four rounds), so
// that a block's start-up cost is amortised and the last round stays short.
inline int64_t item_floats_for(const int64_t* rows, const int64_t* cols, int32_t n_tensors, int sms) {
  int64_t total = 0;
  for (int t = 0; t < n_tensors; ++t) total += rows[t] * cols[t];
  int64_t f = total / ((int64_t)sms * 8);
  if (f < kItemFloatsMin) f = kItemFloatsMin;
  if (f > kItemFloatsMax) f = kItemFloatsMax;
  return f;
}

struct SweepDesc {
  const float* w;
  int64_t rows;
  int32_t cols;
  int32_t item0;          // first work item (block) of this tensor within the launch
  int32_t rows_per_item;
  int32_t tensor;         // index into the caller's tensor list
  int32_t team_log2;      // team size = 32 << team_log2
  int32_t pad;
};

// The descriptor whose item range holds `item`: every thread tests a few descriptors (one
// round of loads instead of a dependent chain), the winner publishes its index.
__device__ __forceinline__ SweepDesc find_desc(const SweepDesc* __restrict__ d, int n, int item) {
  __shared__ int s_idx;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int lo = d[i].item0;
    const int hi = (i + 1 < n) ? d[i + 1].item0 : 0x7fffffff;
    if (lo <= item && item < hi) s_idx = i;       // exactly one i qualifies (item0 strictly increases)
  }
  __syncthreads();
  return d[s_idx];
}

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

// Writes the block's 7 sums and its maximum to partial[item*8 .. item*8+7].
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
}

// Two elements per instruction: the four operations of one (element, b) evaluation as packed
// fp32 arithmetic (sm_100 fma.rn.f32x2 / add.rn.f32x2), which halves the issue slots they need.
__device__ __forceinline__ void err8(float2 x, float2 s, float2 inv, float2& acc) {
  const float2 magic = make_float2(kMagic, kMagic), nmagic = make_float2(-kMagic, -kMagic);
  float2 u = __ffma2_rn(x, inv, magic);
  float2 r = __fadd2_rn(u, nmagic);
  float2 e = __ffma2_rn(make_float2(-s.x, -s.y), r, x);
  acc = __ffma2_rn(e, e, acc);
}

// Rows of up to 32*V*team float4; cols % 4 == 0 and 16-byte aligned rows.  All 7 bit widths are
// always evaluated (a narrower request only selects columns in the finalize kernel).
template <int V>
__global__ void __launch_bounds__(kThreads, 3)
sweep_rows_kernel(const SweepDesc* __restrict__ descs, int n_desc, int per_tensor,
                  const float* __restrict__ tensor_absmax, int jlo, int jhi,
                  double* __restrict__ partial) {
  const SweepDesc d = find_desc(descs, n_desc, blockIdx.x);
  const int T = 32 << d.team_log2;
  const int nteams = kThreads / T;
  const int team = threadIdx.x / T;
  const int tl = threadIdx.x % T;
  const int lane = threadIdx.x & 31;
  const int c4 = d.cols >> 2;
  const int64_t row0 = (int64_t)(blockIdx.x - d.item0) * d.rows_per_item;
  int64_t row1 = row0 + d.rows_per_item;
  if (row1 > d.rows) row1 = d.rows;
  const int n_iter = (int)((row1 - row0 + nteams - 1) / nteams);
  const float A_tensor = per_tensor ? tensor_absmax[d.tensor] : 0.0f;

  __shared__ float smax2[2][kThreads / 32];
  int row_parity = 0;

  double dacc[kNB];
#pragma unroll
  for (int j = 0; j < kNB; ++j) dacc[j] = 0.0;
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
      if (lane == 0) slot[threadIdx.x >> 5] = m;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(T) : "memory");
      const int w0 = team * (T >> 5);
      m = slot[w0];
      for (int w = 1; w < (T >> 5); ++w) m = fmaxf(m, slot[w0 + w]);
      row_parity ^= 1;
    }
    amax_blk = fmaxf(amax_blk, m);
    if (per_tensor) m = A_tensor;

    float s_l, inv_l;
    scales_for_lane(m, lane, s_l, inv_l);
    float2 s[kNB], inv[kNB], facc[kNB];
#pragma unroll
    for (int j = 0; j < kNB; ++j) {
      const float sj = __shfl_sync(0xffffffffu, s_l, j), ij = __shfl_sync(0xffffffffu, inv_l, j);
      s[j] = make_float2(sj, sj);
      inv[j] = make_float2(ij, ij);
      facc[j] = make_float2(0.0f, 0.0f);
    }
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const float2 lo = make_float2(cur[v].x, cur[v].y), hi = make_float2(cur[v].z, cur[v].w);
#pragma unroll
      for (int j = 0; j < kNB; ++j) {
        err8(lo, s[j], inv[j], facc[j]);
        err8(hi, s[j], inv[j], facc[j]);
      }
    }
#pragma unroll
    for (int j = 0; j < kNB; ++j) dacc[j] += (double)(facc[j].x + facc[j].y);
  };

  // Rows stream through a three-stage ring in shared memory filled by cp.async, two rows ahead
  // of the one being processed: enough loads in flight to cover HBM latency without holding
  // future rows in registers.  Every thread copies and reads back only its own 16-byte slots, so
  // no barrier is needed between the copy and the read.
  extern __shared__ float4 ring[];                       // [kRing][V][kThreads]
  auto issue_row = [&](int stage, int64_t row) {
    const float4* p = reinterpret_cast<const float4*>(d.w + row * (int64_t)d.cols);
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const int c = tl + v * T;
      float4* dst = &ring[(stage * V + v) * kThreads + threadIdx.x];
      if (row < row1 && c < c4) {
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(p + c) : "memory");
      } else {
        *dst = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  issue_row(0, row0 + team);
  issue_row(1, row0 + (int64_t)nteams + team);
  int stage = 0;
  for (int it = 0; it < n_iter; ++it) {
    int nxt = stage + 2; if (nxt >= kRing) nxt -= kRing;
    issue_row(nxt, row0 + (int64_t)(it + 2) * nteams + team);      // zeros past the end
    asm volatile("cp.async.wait_group 2;" ::: "memory");            // the row of this iteration has landed
    float4 cur[V];
#pragma unroll
    for (int v = 0; v < V; ++v) cur[v] = ring[(stage * V + v) * kThreads + threadIdx.x];
    process_row(cur);
    if (++stage == kRing) stage = 0;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  block_reduce_store(dacc, amax_blk, partial + (int64_t)blockIdx.x * 8);
}

// Any shape or alignment: the whole block works on one row at a time and reads it twice
// (the second read hits L1/L2).
__global__ void __launch_bounds__(kThreads)
sweep_generic_kernel(const SweepDesc* __restrict__ descs, int n_desc, int per_tensor,
                     const float* __restrict__ tensor_absmax, int jlo, int jhi,
                     double* __restrict__ partial) {
  const SweepDesc d = find_desc(descs, n_desc, blockIdx.x);
  const int lane = threadIdx.x & 31;
  const int64_t row0 = (int64_t)(blockIdx.x - d.item0) * d.rows_per_item;
  int64_t row1 = row0 + d.rows_per_item;
  if (row1 > d.rows) row1 = d.rows;
  const float A_tensor = per_tensor ? tensor_absmax[d.tensor] : 0.0f;
  __shared__ float smax[kThreads / 32];
  double dacc[kNB];
#pragma unroll
  for (int j = 0; j < kNB; ++j) dacc[j] = 0.0;
  float amax_blk = 0.0f;
  for (int64_t row = row0; row < row1; ++row) {
    const float* p = d.w + row * (int64_t)d.cols;
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
    for (int c = threadIdx.x; c < d.cols; c += kThreads) {
      float x = __ldg(p + c);
#pragma unroll
      for (int j = 0; j < kNB; ++j)
        if (j >= jlo && j <= jhi) err4(x, s[j], inv[j], facc[j]);
    }
#pragma unroll
    for (int j = 0; j < kNB; ++j) dacc[j] += (double)facc[j];
  }
  block_reduce_store(dacc, amax_blk, partial + (int64_t)blockIdx.x * 8);
}

struct TensorItems { int32_t item0, item1; };

// One block per tensor: 32 groups of 8 threads stride over the tensor's block partials (thread j
// of a group owns column j: 7 sums and the maximum), then thread j < 8 combines the 32 group
// results in a fixed order.
__global__ void __launch_bounds__(256)
sweep_finalize_kernel(const double* __restrict__ partial, const TensorItems* __restrict__ ti, int jlo, int nb,
                      double* __restrict__ sse, float* __restrict__ absmax, int write_absmax) {
  __shared__ double sm[32][8];
  const int t = blockIdx.x;
  const int j = threadIdx.x & 7, g = threadIdx.x >> 3;
  const TensorItems r = ti[t];
  double v = 0.0;
  for (int i = r.item0 + g; i < r.item1; i += 32) {
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

template <int V>
void launch_rows(const SweepDesc* d, int n, int items, int per_tensor, const float* amax, int jlo, int jhi,
                 double* partial, cudaStream_t st) {
  constexpr size_t smem = (size_t)kRing * V * kThreads * sizeof(float4);
  sweep_rows_kernel<V><<<items, kThreads, smem, st>>>(d, n, per_tensor, amax, jlo, jhi, partial);
}

template <int V>
cudaError_t set_rows_smem() {
  return cudaFuncSetAttribute(sweep_rows_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)((size_t)kRing * V * kThreads * sizeof(float4)));
}

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
  const int nb = b_hi - b_lo + 1;
  const int per_tensor = granularity == QCFG_PER_TENSOR;
  if (n_tensors == 0) return QCFG_OK;

  const int64_t item_floats = item_floats_for(rows, cols, n_tensors, sm_count(ctx));
  // Group tensors by kernel variant: class 0 = generic, class V (1..8) = register-resident rows.
  std::vector<SweepDesc> groups[9];
  std::vector<TensorItems> titems(n_tensors);
  for (int t = 0; t < n_tensors; ++t) {
    SweepDesc d{};
    d.w = w[t]; d.rows = rows[t]; d.cols = (int32_t)cols[t]; d.tensor = t;
    int cls = 0;
    const bool vec = ((uintptr_t)w[t] % 16 == 0) && (cols[t] % 4 == 0) && cols[t] <= 8192 && cols[t] > 0;
    if (vec) {
      int64_t c4 = cols[t] / 4;
      int tl = 0;
      while (tl < 3 && c4 > (int64_t)(32 << tl) * 8) ++tl;
      d.team_log2 = tl;
      cls = (int)((c4 + (32 << tl) - 1) / (32 << tl));     // float4 per thread, 1..8
    }
    int64_t rpi = cols[t] > 0 ? item_floats / cols[t] : 1;
    if (cls > 0) {
      int nteams = kThreads / (32 << d.team_log2);
      rpi = (rpi / nteams) * nteams;
      if (rpi < nteams) rpi = nteams;
    }
    if (rpi < 1) rpi = 1;
    d.rows_per_item = (int32_t)rpi;
    groups[cls].push_back(d);
  }
  // Assign work items: global numbering over all groups so every block owns one partial slot.
  int total_items = 0;
  int group_item0[9], group_items[9];
  for (int c = 0; c < 9; ++c) {
    group_item0[c] = total_items;
    int local = 0;
    for (auto& d : groups[c]) {
      int n = (int)((d.rows + d.rows_per_item - 1) / d.rows_per_item);
      d.item0 = local;
      titems[d.tensor].item0 = total_items + local;
      titems[d.tensor].item1 = total_items + local + n;
      local += n;
    }
    group_items[c] = local;
    total_items += local;
  }

  // Scratch layout: partials | descriptors (all groups) | tensor item ranges.
  const size_t partial_bytes = (size_t)(total_items > 0 ? total_items : 1) * 8 * sizeof(double);
  const size_t desc_bytes = (size_t)n_tensors * sizeof(SweepDesc);
  const size_t ti_bytes = (size_t)n_tensors * sizeof(TensorItems);
  char* base = static_cast<char*>(scratch(ctx, partial_bytes + desc_bytes + ti_bytes));
  if (!base) return set_error(ctx, QCFG_ENOMEM, "sweep scratch (%zu bytes)", partial_bytes + desc_bytes + ti_bytes);
  double* partial = reinterpret_cast<double*>(base);
  SweepDesc* ddev = reinterpret_cast<SweepDesc*>(base + partial_bytes);
  TensorItems* tidev = reinterpret_cast<TensorItems*>(base + partial_bytes + desc_bytes);

  std::vector<SweepDesc> flat;
  int group_desc0[9];
  for (int c = 0; c < 9; ++c) {
    group_desc0[c] = (int)flat.size();
    flat.insert(flat.end(), groups[c].begin(), groups[c].end());
  }
  // the tables only depend on the tensor list: a repeated sweep of the same tensors (same scratch
  // buffer) finds them on the device already
  cudaError_t e = cudaSuccess;
  if (!sweep_tables_cached(ctx, base, st, flat.data(), desc_bytes, titems.data(), ti_bytes)) {
    e = cudaMemcpyAsync(ddev, flat.data(), desc_bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(tidev, titems.data(), ti_bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "sweep descriptor upload");
  }

  if (per_tensor) {
    for (int t = 0; t < n_tensors; ++t) {
      int rc = launch_absmax(ctx, w[t], rows[t], cols[t], cols[t], QCFG_PER_TENSOR, absmax + t, st);
      if (rc != QCFG_OK) return rc;
    }
  }
  const int jlo = b_lo - 2, jhi = b_hi - 2;
  for (int c = 0; c < 9; ++c) {
    if (group_items[c] == 0) continue;
    const SweepDesc* d = ddev + group_desc0[c];
    const int n = (int)groups[c].size();
    double* part = partial + (int64_t)group_item0[c] * 8;
    prof_begin(ctx, 2, st);
    switch (c) {
      case 0: sweep_generic_kernel<<<group_items[c], kThreads, 0, st>>>(d, n, per_tensor, absmax, jlo, jhi, part); break;
      case 1: launch_rows<1>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 2: launch_rows<2>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 3: launch_rows<3>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 4: launch_rows<4>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 5: launch_rows<5>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 6: launch_rows<6>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 7: launch_rows<7>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      default: launch_rows<8>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
    }
    prof_end(ctx, 2, 0.0, st);
    count_launch(ctx);
    e = cudaGetLastError();
    if (e != cudaSuccess) return check_cuda(ctx, e, "sweep launch");
  }
  sweep_finalize_kernel<<<n_tensors, 256, 0, st>>>(partial, tidev, jlo, nb, sse, absmax, per_tensor ? 0 : 1);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "sweep finalize launch");
}


// ------------------------------------------------------------------ sweep without allocation
//
// Same sweep, for callers that must not allocate device memory at call time: the block
// partials and the descriptor tables live in a fixed device array that is part of the loaded
// library image (about 1.05 MiB on every GPU that loads the library, until the process exits).

constexpr int kStaticMaxItems = 16384;     // work items (blocks) per call
constexpr int kStaticMaxTensors = 1024;

struct StaticSweepScratch {
  double partial[kStaticMaxItems * 8];
  SweepDesc descs[kStaticMaxTensors];
  TensorItems items[kStaticMaxTensors];
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
  const int nb = b_hi - b_lo + 1;
  const int per_tensor = granularity == QCFG_PER_TENSOR;
  if (n_tensors == 0) return QCFG_OK;
  if (n_tensors > kStaticMaxTensors)
    return set_error(ctx, QCFG_ENOMEM, "static sweep: %d tensors exceed the fixed scratch (at most %d per call)",
                     n_tensors, kStaticMaxTensors);

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

  const int64_t item_floats = item_floats_for(rows, cols, n_tensors, sm_count(ctx));
  // Plan on the stack: descriptor and kernel class per tensor, then descriptors ordered by class.
  SweepDesc plan[kStaticMaxTensors];
  unsigned char cls_of[kStaticMaxTensors];
  int class_count[9] = {0};
  for (int t = 0; t < n_tensors; ++t) {
    SweepDesc d{};
    d.w = w[t]; d.rows = rows[t]; d.cols = (int32_t)cols[t]; d.tensor = t;
    int cls = 0;
    const bool vec = ((uintptr_t)w[t] % 16 == 0) && (cols[t] % 4 == 0) && cols[t] <= 8192 && cols[t] > 0;
    if (vec) {
      int64_t c4 = cols[t] / 4;
      int tl = 0;
      while (tl < 3 && c4 > (int64_t)(32 << tl) * 8) ++tl;
      d.team_log2 = tl;
      cls = (int)((c4 + (32 << tl) - 1) / (32 << tl));
    }
    int64_t rpi = cols[t] > 0 ? item_floats / cols[t] : 1;
    if (cls > 0) {
      int nteams = kThreads / (32 << d.team_log2);
      rpi = (rpi / nteams) * nteams;
      if (rpi < nteams) rpi = nteams;
    }
    if (rpi < 1) rpi = 1;
    d.rows_per_item = (int32_t)rpi;
    plan[t] = d;
    cls_of[t] = (unsigned char)cls;
    class_count[cls]++;
  }
  int group_desc0[9], fill[9];
  for (int c = 0, acc = 0; c < 9; ++c) { group_desc0[c] = acc; fill[c] = acc; acc += class_count[c]; }
  SweepDesc flat[kStaticMaxTensors];
  for (int t = 0; t < n_tensors; ++t) flat[fill[cls_of[t]]++] = plan[t];

  TensorItems titems[kStaticMaxTensors];
  int group_item0[9], group_items[9];
  int64_t total_items = 0;
  for (int c = 0; c < 9; ++c) {
    group_item0[c] = (int)total_items;
    int64_t local = 0;
    for (int i = 0; i < class_count[c]; ++i) {
      SweepDesc& d = flat[group_desc0[c] + i];
      int64_t n = (d.rows + d.rows_per_item - 1) / d.rows_per_item;
      if (total_items + local + n > kStaticMaxItems)
        return set_error(ctx, QCFG_ENOMEM,
                         "static sweep: the tensors need more than %d work items (of about %lld elements each); "
                         "split the call or use qcfg_quant_error_sweep", kStaticMaxItems, (long long)item_floats);
      d.item0 = (int32_t)local;
      titems[d.tensor].item0 = (int32_t)(total_items + local);
      titems[d.tensor].item1 = (int32_t)(total_items + local + n);
      local += n;
    }
    group_items[c] = (int)local;
    total_items += local;
  }

  // Every block overwrites all 8 slots of its own partial entry and the finalize kernel reads only
  // the entries of this call, so nothing left in the array by an earlier call needs clearing.
  e = cudaMemcpyAsync(S->descs, flat, (size_t)n_tensors * sizeof(SweepDesc), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(S->items, titems, (size_t)n_tensors * sizeof(TensorItems), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return check_cuda(ctx, e, "static sweep: descriptor upload");

  if (per_tensor) {
    for (int t = 0; t < n_tensors; ++t) {
      int rc = launch_absmax(ctx, w[t], rows[t], cols[t], cols[t], QCFG_PER_TENSOR, absmax + t, st);
      if (rc != QCFG_OK) return rc;
    }
  }
  const int jlo = b_lo - 2, jhi = b_hi - 2;
  for (int c = 0; c < 9; ++c) {
    if (group_items[c] == 0) continue;
    const SweepDesc* d = S->descs + group_desc0[c];
    const int n = class_count[c];
    double* part = S->partial + (int64_t)group_item0[c] * 8;
    prof_begin(ctx, 2, st);
    switch (c) {
      case 0: sweep_generic_kernel<<<group_items[c], kThreads, 0, st>>>(d, n, per_tensor, absmax, jlo, jhi, part); break;
      case 1: launch_rows<1>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 2: launch_rows<2>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 3: launch_rows<3>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 4: launch_rows<4>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 5: launch_rows<5>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 6: launch_rows<6>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      case 7: launch_rows<7>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
      default: launch_rows<8>(d, n, group_items[c], per_tensor, absmax, jlo, jhi, part, st); break;
    }
    prof_end(ctx, 2, 0.0, st);
    count_launch(ctx);
    e = cudaGetLastError();
    if (e != cudaSuccess) return check_cuda(ctx, e, "static sweep launch");
  }
  sweep_finalize_kernel<<<n_tensors, 256, 0, st>>>(S->partial, S->items, jlo, nb, sse, absmax, per_tensor ? 0 : 1);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "static sweep finalize launch");
}

}  // namespace qcfg
