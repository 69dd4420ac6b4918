// Glue for the convolutional layer table: pooling in fp32 and the quantize step of a
// convolution's GEMM operand (patch gather in (kh, kw, cin) order fused with Eq. 1's code
// computation, or with the bf16 rounding of 16-bit layers).  All HBM-bound.
#include "common.cuh"

namespace qcfg {

// ------------------------------------------------------------------------------- max-pool 3x3 / 2, pad 1

__global__ void __launch_bounds__(256) maxpool3s2_kernel(const float* __restrict__ src, int64_t B, int H, int W, int C,
                                                         int OH, int OW, float* __restrict__ dst, int vec) {
  const int cg = vec ? (C >> 2) : C;
  const int64_t total = B * OH * OW * cg;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = (int)(idx % cg);
  int64_t t = idx / cg;
  const int ow = (int)(t % OW); t /= OW;
  const int oh = (int)(t % OH);
  const int64_t b = t / OH;
  const float ninf = __int_as_float(0xff800000);
  float4 m = make_float4(ninf, ninf, ninf, ninf);
#pragma unroll
  for (int dy = 0; dy < 3; ++dy) {
    const int ih = 2 * oh - 1 + dy;
    if (ih < 0 || ih >= H) continue;
#pragma unroll
    for (int dx = 0; dx < 3; ++dx) {
      const int iw = 2 * ow - 1 + dx;
      if (iw < 0 || iw >= W) continue;
      const float* p = src + ((b * H + ih) * W + iw) * (int64_t)C;
      if (vec) {
        float4 v = __ldg(reinterpret_cast<const float4*>(p) + c);
        m.x = fmaxf(m.x, v.x); m.y = fmaxf(m.y, v.y); m.z = fmaxf(m.z, v.z); m.w = fmaxf(m.w, v.w);
      } else {
        m.x = fmaxf(m.x, __ldg(p + c));
      }
    }
  }
  float* q = dst + ((b * OH + oh) * OW + ow) * (int64_t)C;
  if (vec) reinterpret_cast<float4*>(q)[c] = m; else q[c] = m.x;
}

int launch_maxpool3s2(Ctx* ctx, const float* src, int64_t B, int H, int W, int C, float* dst, cudaStream_t st) {
  const int OH = (H + 2 - 3) / 2 + 1, OW = (W + 2 - 3) / 2 + 1;
  const int vec = (C % 4 == 0 && (uintptr_t)src % 16 == 0 && (uintptr_t)dst % 16 == 0) ? 1 : 0;
  const int64_t total = B * OH * OW * (vec ? C / 4 : C);
  if (total == 0) return QCFG_OK;
  prof_begin(ctx, 2, st);
  maxpool3s2_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(src, B, H, W, C, OH, OW, dst, vec);
  prof_end(ctx, 2, 0.0, st);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "maxpool launch");
}

// ------------------------------------------------------------------------------- global average pool

// One thread per (image, channel): fp64 sum over the H*W positions, divided once.
__global__ void __launch_bounds__(256) avgpool_kernel(const float* __restrict__ src, int64_t B, int HW, int C,
                                                      float* __restrict__ dst) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= B * C) return;
  const int c = (int)(idx % C);
  const int64_t b = idx / C;
  const float* p = src + b * HW * (int64_t)C + c;
  double s = 0.0;
  for (int i = 0; i < HW; ++i) s += (double)__ldg(p + (int64_t)i * C);
  dst[idx] = (float)(s / (double)HW);
}

int launch_avgpool(Ctx* ctx, const float* src, int64_t B, int HW, int C, float* dst, cudaStream_t st) {
  if (B * C == 0) return QCFG_OK;
  prof_begin(ctx, 2, st);
  avgpool_kernel<<<(unsigned)((B * C + 255) / 256), 256, 0, st>>>(src, B, HW, C, dst);
  prof_end(ctx, 2, 0.0, st);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "avgpool launch");
}

// ------------------------------------------------------------------------------- im2col + quantize

struct ConvGeom {
  int H, W, C, kh, kw, stride, pad, OH, OW, K;
};

__device__ __forceinline__ int conv_code(float x, float inv_scale, float qmax) {
  float t = __fmul_rn(x, inv_scale);
  t = fminf(fmaxf(t, -qmax), qmax);
  return __float2int_rn(t);
}

// Each thread produces 8 consecutive elements of one row of the [B*OH*OW x ldq] operand.
template <bool BF16>
__global__ void __launch_bounds__(256) im2col_quantize_kernel(const float* __restrict__ src, int64_t rows, ConvGeom g,
                                                              float inv_scale, float qmax, void* __restrict__ q,
                                                              int64_t ldq, int vec) {
  const int64_t gpr = ldq >> 3;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * gpr) return;
  const int64_t row = idx / gpr;
  const int k0 = (int)((idx - row * gpr) << 3);
  const int ow = (int)(row % g.OW);
  const int64_t t = row / g.OW;
  const int oh = (int)(t % g.OH);
  const int64_t b = t / g.OH;
  float v[8];
  if (vec && k0 + 8 <= g.K) {      // C % 8 == 0: the 8 elements are 8 channels of one tap
    const int tap = k0 / g.C, c = k0 - tap * g.C;
    const int dy = tap / g.kw, dx = tap - dy * g.kw;
    const int ih = oh * g.stride - g.pad + dy, iw = ow * g.stride - g.pad + dx;
    if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) {
      const float4* p = reinterpret_cast<const float4*>(src + ((b * g.H + ih) * g.W + iw) * (int64_t)g.C + c);
      float4 a = __ldg(p), bb = __ldg(p + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = bb.x; v[5] = bb.y; v[6] = bb.z; v[7] = bb.w;
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = 0.0f;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int k = k0 + j;
      float x = 0.0f;
      if (k < g.K) {
        const int tap = k / g.C, c = k - tap * g.C;
        const int dy = tap / g.kw, dx = tap - dy * g.kw;
        const int ih = oh * g.stride - g.pad + dy, iw = ow * g.stride - g.pad + dx;
        if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) x = __ldg(src + ((b * g.H + ih) * g.W + iw) * (int64_t)g.C + c);
      }
      v[j] = x;
    }
  }
  if (BF16) {
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
      o[j] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(q) + row * ldq + k0) = make_uint4(o[0], o[1], o[2], o[3]);
  } else {
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      lo |= (uint32_t)(conv_code(v[j], inv_scale, qmax) & 0xff) << (8 * j);
      hi |= (uint32_t)(conv_code(v[j + 4], inv_scale, qmax) & 0xff) << (8 * j);
    }
    *reinterpret_cast<uint2*>(reinterpret_cast<int8_t*>(q) + row * ldq + k0) = make_uint2(lo, hi);
  }
}

int launch_im2col_quantize(Ctx* ctx, const float* src, int64_t B, int H, int W, int C, int kh, int kw, int stride,
                           int pad, float inv_scale, int bits, void* q, int64_t ldq, cudaStream_t st) {
  ConvGeom g;
  g.H = H; g.W = W; g.C = C; g.kh = kh; g.kw = kw; g.stride = stride; g.pad = pad;
  g.OH = (H + 2 * pad - kh) / stride + 1;
  g.OW = (W + 2 * pad - kw) / stride + 1;
  g.K = kh * kw * C;
  const int64_t rows = B * g.OH * g.OW;
  if (rows == 0) return QCFG_OK;
  const int vec = (C % 8 == 0 && (uintptr_t)src % 16 == 0) ? 1 : 0;
  const int64_t total = rows * (ldq >> 3);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  prof_begin(ctx, 2, st);
  if (bits == 16) im2col_quantize_kernel<true><<<blocks, 256, 0, st>>>(src, rows, g, 1.0f, 0.0f, q, ldq, vec);
  else im2col_quantize_kernel<false><<<blocks, 256, 0, st>>>(src, rows, g, inv_scale, qmax_of(bits), q, ldq, vec);
  prof_end(ctx, 2, 0.0, st);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "im2col launch");
}

}  // namespace qcfg
