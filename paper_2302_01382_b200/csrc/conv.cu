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
  int c, ow, oh;
  int64_t b;
  if (total <= 0x7fffffff) {            // 32-bit index arithmetic (64-bit divisions cost an order of magnitude more)
    const unsigned i = (unsigned)idx, t1 = i / (unsigned)cg, t2 = t1 / (unsigned)OW;
    c = (int)(i - t1 * cg); ow = (int)(t1 - t2 * OW);
    const unsigned t3 = t2 / (unsigned)OH;
    oh = (int)(t2 - t3 * OH); b = t3;
  } else {
    c = (int)(idx % cg);
    int64_t t = idx / cg;
    ow = (int)(t % OW); t /= OW;
    oh = (int)(t % OH);
    b = t / OH;
  }
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
  int kwC, WC;                 // elements of one kernel row (kw * C) and of one image row (W * C)
  uint32_t dm, ds1, ds2;       // division by kwC as multiply-high and shifts
};

// floor(n / d) for any 32-bit n with the constants of fastdiv_init(d)
__device__ __forceinline__ uint32_t fastdiv(uint32_t n, uint32_t m, uint32_t s1, uint32_t s2) {
  const uint32_t t = __umulhi(m, n);
  return (t + ((n - t) >> s1)) >> s2;
}
static void fastdiv_init(uint32_t d, uint32_t* m, uint32_t* s1, uint32_t* s2) {
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;                                  // ceil(log2 d)
  *m = (uint32_t)((((1ull << l) - d) << 32) / d + 1);
  *s1 = l < 1 ? l : 1;
  *s2 = l > 0 ? l - 1 : 0;
}

// int8 code of Eq. 1 in the low byte of the returned word: one multiply, the clamp to +-qmax as
// min(|t|, qmax) with t's sign, and a round-half-even by adding 1.5 * 2^23 (the low mantissa byte is
// then the two's-complement code) -- all on the fp32 pipe, no float-to-int conversion.
__device__ __forceinline__ uint32_t conv_code(float x, float inv_scale, float qmax) {
  const float t = __fmul_rn(x, inv_scale);
  float c;
  asm("min.xorsign.abs.f32 %0, %1, %2;" : "=f"(c) : "f"(t), "f"(qmax));
  return __float_as_uint(__fadd_rn(c, 12582912.0f));
}
__device__ __forceinline__ uint32_t conv_pack4(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

// Operand row (b, oh, ow) holds the patch in (kh, kw, cin) order.  For a fixed kernel row dy the kw * C
// values are contiguous in the NHWC source, so element k = dy * kwC + r comes from offset
// (ow * stride - pad) * C + r of image row ih = oh * stride - pad + dy, if that offset lies inside the
// row: one division per group instead of one per index level.  blockIdx.x = b * OH + oh,
// blockIdx.y and threadIdx.y give ow, threadIdx.x strides over groups of 8 consecutive k.
template <bool BF16>
__global__ void __launch_bounds__(256) im2col_quantize_kernel(const float* __restrict__ src, ConvGeom g, float inv_scale,
                                                              float qmax, void* __restrict__ q, int64_t ldq, int vec) {
  const int boh = blockIdx.x;
  const int b = boh / g.OH, oh = boh - b * g.OH;
  const int ow = blockIdx.y * blockDim.y + threadIdx.y;
  if (ow >= g.OW) return;
  const int64_t row = (int64_t)boh * g.OW + ow;
  const int off0 = (ow * g.stride - g.pad) * g.C;
  const int ih0 = oh * g.stride - g.pad;
  const float* img = src + (int64_t)b * g.H * g.WC;
  const int gpr = (int)(ldq >> 3);
  for (int kg = threadIdx.x; kg < gpr; kg += blockDim.x) {
    const int k0 = kg << 3;
    float v[8];
    if (vec) {                       // C % 8 == 0: the 8 elements share dy, dx and validity
      bool ok = k0 < g.K;
      const int dy = (int)fastdiv((uint32_t)k0, g.dm, g.ds1, g.ds2);
      const int off = off0 + (k0 - dy * g.kwC), ih = ih0 + dy;
      ok = ok && ih >= 0 && ih < g.H && off >= 0 && off < g.WC;
      if (ok) {
        const float4* p = reinterpret_cast<const float4*>(img + (int64_t)ih * g.WC + off);
        const float4 a = __ldg(p), c = __ldg(p + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = 0.0f;
      }
    } else if (g.kwC >= 8) {         // one division per group: the 8 elements lie in at most two kernel rows
      int dy = (int)fastdiv((uint32_t)k0, g.dm, g.ds1, g.ds2);
      int r = k0 - dy * g.kwC;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (r >= g.kwC) { r -= g.kwC; ++dy; }
        const int off = off0 + r, ih = ih0 + dy;
        float x = 0.0f;
        if (k0 + j < g.K && ih >= 0 && ih < g.H && off >= 0 && off < g.WC) x = __ldg(img + (int64_t)ih * g.WC + off);
        v[j] = x;
        ++r;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int k = k0 + j;
        const int dy = (int)fastdiv((uint32_t)k, g.dm, g.ds1, g.ds2);
        const int off = off0 + (k - dy * g.kwC), ih = ih0 + dy;
        float x = 0.0f;
        if (k < g.K && ih >= 0 && ih < g.H && off >= 0 && off < g.WC) x = __ldg(img + (int64_t)ih * g.WC + off);
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
      const uint32_t lo = conv_pack4(conv_code(v[0], inv_scale, qmax), conv_code(v[1], inv_scale, qmax),
                                     conv_code(v[2], inv_scale, qmax), conv_code(v[3], inv_scale, qmax));
      const uint32_t hi = conv_pack4(conv_code(v[4], inv_scale, qmax), conv_code(v[5], inv_scale, qmax),
                                     conv_code(v[6], inv_scale, qmax), conv_code(v[7], inv_scale, qmax));
      *reinterpret_cast<uint2*>(reinterpret_cast<int8_t*>(q) + row * ldq + k0) = make_uint2(lo, hi);
    }
  }
}


// Inputs with few channels (the 3-channel stem): one block per output row (b, oh).  The kh input
// rows the row's patches draw from are staged in shared memory with coalesced loads, zero-padded on
// both sides (and zero where they fall outside the image), so building the patches needs no bounds
// checks and no divisions: a table gives every k its offset (dy * row length + position in the
// kernel row).  Consecutive threads write consecutive 8-element groups of an output row.
template <bool BF16>
__global__ void __launch_bounds__(256) im2col_rows_kernel(const float* __restrict__ src, ConvGeom g, float inv_scale, float qmax,
                                                          void* __restrict__ q, int64_t ldq) {
  extern __shared__ float srows[];                 // [kh][rowlen] then int koff[ldq]
  const int rowlen = (g.W + 2 * g.pad) * g.C;
  int* koff = reinterpret_cast<int*>(srows + g.kh * rowlen);
  const int boh = blockIdx.x;
  const int b = boh / g.OH, oh = boh - b * g.OH;
  const float* img = src + (int64_t)b * g.H * g.WC;
  for (int i = threadIdx.x; i < g.kh * rowlen; i += blockDim.x) {
    const int dy = i / rowlen, p = i - dy * rowlen - g.pad * g.C;
    const int ih = oh * g.stride - g.pad + dy;
    srows[i] = (ih >= 0 && ih < g.H && p >= 0 && p < g.WC) ? __ldg(img + (int64_t)ih * g.WC + p) : 0.0f;
  }
  for (int k = threadIdx.x; k < (int)ldq; k += blockDim.x) {
    const int dy = k / g.kwC;
    koff[k] = k < g.K ? dy * rowlen + (k - dy * g.kwC) : -1;
  }
  __syncthreads();
  const int gpr = (int)(ldq >> 3);
  for (int it = threadIdx.x; it < g.OW * gpr; it += blockDim.x) {
    const int ow = it / gpr, k0 = (it - ow * gpr) << 3;
    const int base = ow * g.stride * g.C;
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int o = koff[k0 + j];
      v[j] = o >= 0 ? srows[o + base] : 0.0f;
    }
    const int64_t row = (int64_t)boh * g.OW + ow;
    if (BF16) {
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
        w[j] = *reinterpret_cast<uint32_t*>(&h);
      }
      *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(q) + row * ldq + k0) = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
      const uint32_t lo = conv_pack4(conv_code(v[0], inv_scale, qmax), conv_code(v[1], inv_scale, qmax),
                                     conv_code(v[2], inv_scale, qmax), conv_code(v[3], inv_scale, qmax));
      const uint32_t hi = conv_pack4(conv_code(v[4], inv_scale, qmax), conv_code(v[5], inv_scale, qmax),
                                     conv_code(v[6], inv_scale, qmax), conv_code(v[7], inv_scale, qmax));
      *reinterpret_cast<uint2*>(reinterpret_cast<int8_t*>(q) + row * ldq + k0) = make_uint2(lo, hi);
    }
  }
}

int launch_im2col_quantize(Ctx* ctx, const float* src, int64_t B, int H, int W, int C, int kh, int kw, int stride,
                           int pad, float inv_scale, int bits, void* q, int64_t ldq, cudaStream_t st) {
  ConvGeom g;
  g.H = H; g.W = W; g.C = C; g.kh = kh; g.kw = kw; g.stride = stride; g.pad = pad;
  g.OH = (H + 2 * pad - kh) / stride + 1;
  g.OW = (W + 2 * pad - kw) / stride + 1;
  g.K = kh * kw * C;
  g.kwC = kw * C; g.WC = W * C;
  fastdiv_init((uint32_t)g.kwC, &g.dm, &g.ds1, &g.ds2);
  const int64_t rows = B * g.OH * g.OW;
  if (rows == 0) return QCFG_OK;
  if (B * g.OH > 0x7fffffff || (int64_t)W * C > 0x7fffffff) return set_error(ctx, QCFG_ESHAPE, "im2col: image too large");
  const int vec = (C % 8 == 0 && (uintptr_t)src % 16 == 0) ? 1 : 0;
  const size_t rows_smem = ((size_t)kh * (W + 2 * pad) * C + (size_t)ldq) * 4;
  if (!vec && rows_smem <= 48 * 1024) {          // few channels: the row-staged kernel
    prof_begin(ctx, 2, st);
    if (bits == 16) im2col_rows_kernel<true><<<(unsigned)(B * g.OH), 256, rows_smem, st>>>(src, g, 1.0f, 0.0f, q, ldq);
    else im2col_rows_kernel<false><<<(unsigned)(B * g.OH), 256, rows_smem, st>>>(src, g, inv_scale, qmax_of(bits), q, ldq);
    prof_end(ctx, 2, 0.0, st);
    count_launch(ctx);
    return check_cuda(ctx, cudaGetLastError(), "im2col launch");
  }
  const int gpr = (int)(ldq >> 3);
  const int bx = gpr >= 24 ? 32 : (gpr >= 12 ? 16 : 8);
  const int by = 256 / bx;
  const dim3 block((unsigned)bx, (unsigned)by);
  const dim3 grid((unsigned)(B * g.OH), (unsigned)((g.OW + by - 1) / by));
  if (grid.y > 65535) return set_error(ctx, QCFG_ESHAPE, "im2col: output row too wide");
  prof_begin(ctx, 2, st);
  if (bits == 16) im2col_quantize_kernel<true><<<grid, block, 0, st>>>(src, g, 1.0f, 0.0f, q, ldq, vec);
  else im2col_quantize_kernel<false><<<grid, block, 0, st>>>(src, g, inv_scale, qmax_of(bits), q, ldq, vec);
  prof_end(ctx, 2, 0.0, st);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "im2col launch");
}


// Patches of an int8 NHWC code tensor (parity taps of convolutions whose GEMM gathers its operand
// itself): one thread per 16 codes of an output row.
__global__ void __launch_bounds__(256) im2col_codes_kernel(const int8_t* __restrict__ src, int64_t rows, int H, int W, int C, int kh,
                                                           int kw, int stride, int pad, int OH, int OW, int8_t* __restrict__ dst,
                                                           int64_t ldd) {
  const int cpr = kh * kw * C / 16;                 // 16-code chunks per output row
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * cpr) return;
  const int64_t row = idx / cpr;
  const int k0 = (int)(idx - row * cpr) * 16;
  const int tap = k0 / C, c = k0 - tap * C, dy = tap / kw, dx = tap - dy * kw;
  const int64_t b = row / ((int64_t)OH * OW);
  const int pix = (int)(row - b * OH * OW), oh = pix / OW, ow = pix - oh * OW;
  const int ih = oh * stride - pad + dy, iw = ow * stride - pad + dx;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (ih >= 0 && ih < H && iw >= 0 && iw < W)
    v = *reinterpret_cast<const uint4*>(src + ((b * H + ih) * W + iw) * C + c);
  int8_t* o = dst + row * ldd + k0;
  if ((reinterpret_cast<uintptr_t>(o) & 15) == 0) *reinterpret_cast<uint4*>(o) = v;
  else {
    const int8_t* pv = reinterpret_cast<const int8_t*>(&v);
    for (int j = 0; j < 16; ++j) o[j] = pv[j];
  }
}

int launch_im2col_codes(Ctx* ctx, const int8_t* src, int64_t B, int H, int W, int C, int kh, int kw, int stride, int pad,
                        int8_t* dst, int64_t ldd, cudaStream_t st) {
  const int OH = (H + 2 * pad - kh) / stride + 1, OW = (W + 2 * pad - kw) / stride + 1;
  const int64_t rows = B * OH * OW, total = rows * (kh * kw * C / 16);
  if (total == 0) return QCFG_OK;
  im2col_codes_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(src, rows, H, W, C, kh, kw, stride, pad, OH, OW, dst, ldd);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "code patch launch");
}

}  // namespace qcfg
