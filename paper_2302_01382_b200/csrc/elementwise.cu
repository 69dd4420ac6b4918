// HBM-bound elementwise steps: max calibration (absmax), scales, b-bit quantize.
// Section 3.1 of the paper (max calibration) and Eq. 1 (the quantizer).
#include "common.cuh"

namespace qcfg {

// ------------------------------------------------------------------------------- absmax

__device__ __forceinline__ unsigned max4(float4 v) {
  unsigned a = abs_bits(v.x), b = abs_bits(v.y), c = abs_bits(v.z), d = abs_bits(v.w);
  a = a > b ? a : b;
  c = c > d ? c : d;
  return a > c ? a : c;
}

// Per-tensor: grid-stride over a dense or strided [rows x cols] matrix; the result is an
// integer max over |x| bit patterns, so it is exact and independent of the order.
__global__ void __launch_bounds__(256) absmax_tensor_kernel(const float* __restrict__ x, int64_t rows,
                                                            int64_t cols, int64_t ld, int vec,
                                                            unsigned* __restrict__ out) {
  unsigned m = 0;
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t nth = (int64_t)gridDim.x * blockDim.x;
  if (vec) {
    const int64_t c4 = cols >> 2;
    const int64_t total = rows * c4;
    if (ld == cols) {
      const float4* p = reinterpret_cast<const float4*>(x);
      for (int64_t i = tid; i < total; i += nth) {
        unsigned a = max4(__ldg(p + i));
        m = m > a ? m : a;
      }
    } else {
      for (int64_t i = tid; i < total; i += nth) {
        int64_t r = i / c4, c = i - r * c4;
        unsigned a = max4(__ldg(reinterpret_cast<const float4*>(x + r * ld) + c));
        m = m > a ? m : a;
      }
    }
  } else {
    const int64_t total = rows * cols;
    for (int64_t i = tid; i < total; i += nth) {
      int64_t r = i / cols, c = i - r * cols;
      unsigned a = abs_bits(__ldg(x + r * ld + c));
      m = m > a ? m : a;
    }
  }
  m = warp_max_u(m);
  __shared__ unsigned sm[8];
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < (blockDim.x >> 5) ? sm[threadIdx.x] : 0u;
    m = warp_max_u(m);
    if (threadIdx.x == 0 && m) atomicMax(out, m);
  }
}

// Per-row: one warp per row.
__global__ void __launch_bounds__(256) absmax_rows_kernel(const float* __restrict__ x, int64_t rows,
                                                          int64_t cols, int64_t ld, int vec,
                                                          float* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float* p = x + row * ld;
  unsigned m = 0;
  if (vec) {
    const float4* p4 = reinterpret_cast<const float4*>(p);
    for (int64_t i = lane; i < (cols >> 2); i += 32) {
      unsigned a = max4(__ldg(p4 + i));
      m = m > a ? m : a;
    }
  } else {
    for (int64_t i = lane; i < cols; i += 32) {
      unsigned a = abs_bits(__ldg(p + i));
      m = m > a ? m : a;
    }
  }
  m = warp_max_u(m);
  if (lane == 0) out[row] = __uint_as_float(m);
}

static inline bool vec4_ok(const void* p, int64_t cols, int64_t ld) {
  return ((uintptr_t)p % 16 == 0) && (cols % 4 == 0) && (ld % 4 == 0);
}

int launch_absmax(Ctx* ctx, const float* x, int64_t rows, int64_t cols, int64_t ld, int granularity,
                  float* absmax, cudaStream_t st) {
  const int vec = vec4_ok(x, cols, ld) ? 1 : 0;
  if (granularity == QCFG_PER_TENSOR) {
    cudaError_t e = cudaMemsetAsync(absmax, 0, sizeof(float), st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "memset absmax");
    if (rows * cols == 0) return QCFG_OK;
    int64_t work = vec ? rows * cols / 4 : rows * cols;
    int64_t blocks = (work + 256 * 4 - 1) / (256 * 4);
    int64_t cap = (int64_t)sm_count(ctx) * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    prof_begin(ctx, 2, st);
    absmax_tensor_kernel<<<(unsigned)blocks, 256, 0, st>>>(x, rows, cols, ld, vec,
                                                            reinterpret_cast<unsigned*>(absmax));
    prof_end(ctx, 2, 0.0, st);
  } else {
    if (rows == 0) return QCFG_OK;
    int64_t blocks = (rows + 7) / 8;
    prof_begin(ctx, 2, st);
    absmax_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(x, rows, cols, ld, vec, absmax);
    prof_end(ctx, 2, 0.0, st);
  }
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "absmax launch");
}

// ------------------------------------------------------------------------------- scales

__global__ void scales_kernel(const float* __restrict__ absmax, int64_t n, float qmax,
                              float* __restrict__ scale, float* __restrict__ inv_scale) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float A = absmax[i];
  float s = 1.0f, inv = 1.0f;
  if (A != 0.0f) {
    s = __fdiv_rn(A, qmax);
    inv = __fdiv_rn(qmax, A);
  }
  if (scale) scale[i] = s;
  if (inv_scale) inv_scale[i] = inv;
}

int launch_scales(Ctx* ctx, const float* absmax, int64_t n, int bits, float* scale, float* inv_scale,
                  cudaStream_t st) {
  if (n == 0) return QCFG_OK;
  prof_begin(ctx, 2, st);
  scales_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(absmax, n, qmax_of(bits), scale, inv_scale);
  prof_end(ctx, 2, 0.0, st);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "scales launch");
}

// ------------------------------------------------------------------------------- quantize

// Code of Eq. 1 for one value: clamp before rounding (the bounds are integers and rounding
// is monotone, so this equals rounding first), then round half to even.
__device__ __forceinline__ int quant_code(float x, float inv_scale, float qmax) {
  float t = __fmul_rn(x, inv_scale);
  t = fminf(fmaxf(t, -qmax), qmax);
  return __float2int_rn(t);
}

// Each thread produces 8 consecutive output elements of one row.  With `amax` set the launch also
// folds max |x| of everything it read into *amax (bit patterns, so exact in any order): calibration
// reads each activation tensor once for both its range and its 16-bit operand.
template <bool BF16>
__global__ void __launch_bounds__(256) quantize_kernel(const float* __restrict__ x, int64_t rows, int64_t cols,
                                                       int64_t ld, const float* __restrict__ inv_scale_ptr,
                                                       float inv_scale_val, int per_row, float qmax,
                                                       void* __restrict__ q, int64_t ldq, int vec,
                                                       unsigned* __restrict__ amax) {
  const int64_t gpr = ldq >> 3;  // groups of 8 per output row
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  unsigned m = 0;
  if (idx < rows * gpr) {
    const int64_t row = idx / gpr;
    const int64_t c0 = (idx - row * gpr) << 3;
    float v[8];
    const float* p = x + row * ld + c0;
    if (vec && c0 + 8 <= cols) {
      float4 a = __ldg(reinterpret_cast<const float4*>(p));
      float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = (c0 + j < cols) ? __ldg(p + j) : 0.0f;
    }
    if (BF16) {
      if (amax) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          unsigned a = abs_bits(v[j]);
          m = m > a ? m : a;
        }
      }
      uint32_t o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
        o[j] = *reinterpret_cast<uint32_t*>(&h);
      }
      *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(q) + row * ldq + c0) =
          make_uint4(o[0], o[1], o[2], o[3]);
    } else {
      float inv = inv_scale_ptr ? (per_row ? __ldg(inv_scale_ptr + row) : __ldg(inv_scale_ptr)) : inv_scale_val;
      uint32_t lo = 0, hi = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        lo |= (uint32_t)(quant_code(v[j], inv, qmax) & 0xff) << (8 * j);
        hi |= (uint32_t)(quant_code(v[j + 4], inv, qmax) & 0xff) << (8 * j);
      }
      *reinterpret_cast<uint2*>(reinterpret_cast<int8_t*>(q) + row * ldq + c0) = make_uint2(lo, hi);
    }
  }
  if (BF16 && amax) {       // uniform over the block: no thread has left
    m = warp_max_u(m);
    __shared__ unsigned sm[8];
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
      m = threadIdx.x < 8 ? sm[threadIdx.x] : 0u;
      m = warp_max_u(m);
      if (threadIdx.x == 0 && m) atomicMax(amax, m);
    }
  }
}

int launch_quantize(Ctx* ctx, const float* x, int64_t rows, int64_t cols, int64_t ld,
                    const float* inv_scale_ptr, float inv_scale_val, int granularity, int bits, void* q,
                    int64_t ldq, cudaStream_t st, float* absmax) {
  if (absmax) {
    if (bits != 16) return set_error(ctx, QCFG_EINVAL, "quantize: the fused range is computed with 16-bit operands only");
    cudaError_t e = cudaMemsetAsync(absmax, 0, sizeof(float), st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "memset absmax");
  }
  if (rows == 0 || ldq == 0) return QCFG_OK;
  // vector loads need every row start and every group start 16-byte aligned
  const int vec = ((uintptr_t)x % 16 == 0 && ld % 4 == 0) ? 1 : 0;
  const int64_t total = rows * (ldq >> 3);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (bits == 16) {
    prof_begin(ctx, 2, st);
    quantize_kernel<true><<<blocks, 256, 0, st>>>(x, rows, cols, ld, nullptr, 1.0f, 0, 0.0f, q, ldq, vec,
                                                  reinterpret_cast<unsigned*>(absmax));
    prof_end(ctx, 2, 0.0, st);
  } else {
    prof_begin(ctx, 2, st);
    quantize_kernel<false><<<blocks, 256, 0, st>>>(x, rows, cols, ld, inv_scale_ptr, inv_scale_val,
                                                   granularity == QCFG_PER_ROW, qmax_of(bits), q, ldq, vec, nullptr);
    prof_end(ctx, 2, 0.0, st);
  }
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "quantize launch");
}


// ------------------------------------------------------------------------------- noise injection (Eqs. 3-5)

// bf16 operand of a weight tensor with Gaussian noise added: w + (lambda * max|w|) * nu, nu being
// the caller's standard-normal draws; one fp32 multiply for the deviation, one for the scaled
// draw, one add (no FMA), then round-to-nearest-even to bf16.  Columns cols..ldq-1 are zero.
__global__ void __launch_bounds__(256) perturb_bf16_kernel(const float* __restrict__ w, const float* __restrict__ nu,
                                                           const float* __restrict__ amax, float lambda, int64_t rows,
                                                           int64_t cols, __nv_bfloat16* __restrict__ q, int64_t ldq) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * ldq) return;
  const int64_t r = idx / ldq, c = idx - r * ldq;
  float v = 0.0f;
  if (c < cols) {
    const float sigma = __fmul_rn(lambda, __ldg(amax));
    v = __fadd_rn(__ldg(w + r * cols + c), __fmul_rn(sigma, __ldg(nu + r * cols + c)));
  }
  q[idx] = __float2bfloat16_rn(v);
}

int launch_perturb_bf16(Ctx* ctx, const float* w, const float* nu, const float* amax_dev, float lambda, int64_t rows,
                        int64_t cols, void* q, int64_t ldq, cudaStream_t st) {
  const int64_t total = rows * ldq;
  if (total == 0) return QCFG_OK;
  prof_begin(ctx, 2, st);
  perturb_bf16_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w, nu, amax_dev, lambda, rows, cols,
                                                                      reinterpret_cast<__nv_bfloat16*>(q), ldq);
  prof_end(ctx, 2, 0.0, st);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "perturb launch");
}

// ------------------------------------------------------------------------------- output fidelity

// Per-block partial sums of (y - ref)^2 and ref^2 in fp64 (fixed grid, fixed order: deterministic).
__global__ void __launch_bounds__(256) sqdiff_kernel(const float* __restrict__ y, const float* __restrict__ ref,
                                                     int64_t n, double* __restrict__ partial) {
  double d2 = 0.0, r2 = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const double r = (double)__ldg(ref + i), d = (double)__ldg(y + i) - r;
    d2 += d * d;
    r2 += r * r;
  }
  d2 = warp_sum(d2);
  r2 = warp_sum(r2);
  __shared__ double sm[8][2];
  if ((threadIdx.x & 31) == 0) { sm[threadIdx.x >> 5][0] = d2; sm[threadIdx.x >> 5][1] = r2; }
  __syncthreads();
  if (threadIdx.x < 2) {
    double v = 0.0;
    for (int w = 0; w < 8; ++w) v += sm[w][threadIdx.x];
    partial[2 * blockIdx.x + threadIdx.x] = v;
  }
}

int launch_sqdiff(Ctx* ctx, const float* y, const float* ref, int64_t n, double* partial, int blocks, cudaStream_t st) {
  prof_begin(ctx, 2, st);
  sqdiff_kernel<<<blocks, 256, 0, st>>>(y, ref, n, partial);
  prof_end(ctx, 2, 0.0, st);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "fidelity launch");
}

}  // namespace qcfg
