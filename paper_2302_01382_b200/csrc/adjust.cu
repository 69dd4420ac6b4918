// Kernels of the scale-adjustment step (Section 3.1, second step of the scale estimation: the
// quantization scales are adapted by backpropagation while the model's parameters stay fixed).
// The two backward GEMMs of a layer run on the tensor-core kernel of gemm.cu with bf16 operands;
// what is here is the element-wise and reduction work around them: activation forward and
// derivative, the loss gradient, the straight-through derivative of the quantizer (1 inside the
// clip range, 0 outside), the reductions that give the gradient of each scale, and the update.
#include "common.cuh"

namespace qcfg {

namespace {

__device__ __forceinline__ float act_forward(float y, int act) {
  if (act == QCFG_ACT_RELU) return fmaxf(y, 0.0f);
  if (act == QCFG_ACT_GELU_TANH) return gelu_tanh(y);
  return y;
}
// derivative of the activation at y
__device__ __forceinline__ float act_derivative(float y, int act) {
  if (act == QCFG_ACT_RELU) return y > 0.0f ? 1.0f : 0.0f;
  if (act == QCFG_ACT_GELU_TANH) {
    const float c = 0.7978845608028654f, a = 0.044715f;
    const float u = c * (y + a * y * y * y);
    const float sig = 1.0f / (1.0f + __expf(-2.0f * u));
    return sig + y * sig * (1.0f - sig) * 2.0f * c * (1.0f + 3.0f * a * y * y);
  }
  return 1.0f;
}

__global__ void __launch_bounds__(256) act_apply_kernel(const float* __restrict__ ylin, const float* __restrict__ res,
                                                        int64_t ldr, int act, float* __restrict__ y, int64_t rows, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * n) return;
  float v = ylin[i];
  if (res) { const int64_t r = i / n; v = __fadd_rn(v, res[r * ldr + (i - r * n)]); }
  y[i] = act_forward(v, act);
}

__global__ void __launch_bounds__(256) loss_grad_kernel(const float* __restrict__ y, const float* __restrict__ yref, float coef,
                                                        float* __restrict__ g, int64_t count) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) g[i] = coef * (y[i] - yref[i]);
}

__global__ void __launch_bounds__(256) act_backward_kernel(float* __restrict__ g, const float* __restrict__ ylin,
                                                           const float* __restrict__ res, int64_t ldr, int act, int64_t rows, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * n) return;
  float v = ylin[i];
  if (res) { const int64_t r = i / n; v = __fadd_rn(v, res[r * ldr + (i - r * n)]); }
  g[i] *= act_derivative(v, act);
}

// blockDim (32, 8): 32 columns per block, rows strided over threadIdx.y and blockIdx.y
__global__ void __launch_bounds__(256) col_dot_kernel(const float* __restrict__ a, const float* __restrict__ b, int64_t rows,
                                                      int64_t n, double* __restrict__ out) {
  __shared__ double sm[8][32];
  const int64_t c = (int64_t)blockIdx.x * 32 + threadIdx.x;
  double v = 0.0;
  if (c < n)
    for (int64_t r = (int64_t)blockIdx.y * 8 + threadIdx.y; r < rows; r += (int64_t)gridDim.y * 8)
      v += (double)a[r * n + c] * (double)b[r * n + c];
  sm[threadIdx.y][threadIdx.x] = v;
  __syncthreads();
  if (threadIdx.y == 0 && c < n) {
    for (int j = 1; j < 8; ++j) v += sm[j][threadIdx.x];
    atomicAdd(out + c, v);
  }
}

__global__ void __launch_bounds__(256) gamma_finish_kernel(const double* __restrict__ colsum, const float* __restrict__ s_w,
                                                           float s_x, int64_t n, double* __restrict__ d_sw, double* __restrict__ d_sx) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  double v = 0.0;
  if (i < n) {
    d_sw[i] = colsum[i] / (double)s_w[i];
    v = colsum[i] / (double)s_x;
  }
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0 && v != 0.0) atomicAdd(d_sx, v);
}

__global__ void __launch_bounds__(256) scale_cols_bf16_kernel(const float* __restrict__ g, const float* __restrict__ col_scale,
                                                              int64_t rows, int64_t n, __nv_bfloat16* __restrict__ out, int64_t ld) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * ld) return;
  const int64_t r = i / ld, c = i - r * ld;
  float v = 0.0f;
  if (c < n) { v = g[r * n + c]; if (col_scale) v *= col_scale[c]; }
  out[i] = __float2bfloat16_rn(v);
}

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<int8_t>(int8_t v) { return (float)v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// 32 x 32 tiles through shared memory; grid (ceil(ld_dst/32), ceil(cols/32)); dst columns beyond `rows` get zero
template <typename T>
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const T* __restrict__ src, int64_t rows, int64_t cols, int64_t ld_src,
                                                             __nv_bfloat16* __restrict__ dst, int64_t ld_dst) {
  __shared__ float tile[32][33];
  const int64_t r0 = (int64_t)blockIdx.x * 32, c0 = (int64_t)blockIdx.y * 32;
  for (int j = threadIdx.y; j < 32; j += 8) {
    const int64_t r = r0 + j, c = c0 + threadIdx.x;
    tile[j][threadIdx.x] = (r < rows && c < cols) ? to_float<T>(src[r * ld_src + c]) : 0.0f;
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += 8) {
    const int64_t c = c0 + j, r = r0 + threadIdx.x;      // dst[c][r]
    if (c < cols && r < ld_dst) dst[c * ld_dst + r] = __float2bfloat16_rn(tile[threadIdx.x][j]);
  }
}

__global__ void __launch_bounds__(256) input_backward_kernel(const float* __restrict__ dxq, const float* __restrict__ x, int64_t ldx,
                                                             float s_x, float inv_x, float qmax, int64_t rows, int64_t k,
                                                             float* __restrict__ gprod, int64_t ldg, double* __restrict__ d_ix) {
  double part = 0.0;
  const float pass = __fmul_rn(s_x, inv_x);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < rows * k; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / k, c = i - r * k;
    const float d = dxq[i];
    if (qmax == 0.0f) {                         // 16-bit layer: rounding passed through
      if (gprod) gprod[r * ldg + c] += d;
      continue;
    }
    const float xv = x[r * ldx + c];
    const bool inside = fabsf(__fmul_rn(xv, inv_x)) <= qmax;     // derivative of the clip
    if (inside) {
      part += (double)d * (double)xv;
      if (gprod) gprod[r * ldg + c] += d * pass;
    }
  }
  part = warp_sum(part);
  __shared__ double sm[8];
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = part;
  __syncthreads();
  if (threadIdx.x == 0 && d_ix) {
    double v = 0.0;
    for (int w = 0; w < 8; ++w) v += sm[w];
    if (v != 0.0) atomicAdd(d_ix, v * (double)s_x);
  }
}

// one warp per weight row
__global__ void __launch_bounds__(256) weight_alpha_kernel(const float* __restrict__ dwq, const float* __restrict__ w,
                                                           const float* __restrict__ s_w, const float* __restrict__ inv_w, float s_x,
                                                           float qmax, int64_t n, int64_t k, double* __restrict__ d_iw) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n) return;
  const float iw = inv_w[row];
  double v = 0.0;
  for (int64_t c = lane; c < k; c += 32) {
    const float wv = w[row * k + c];
    if (fabsf(__fmul_rn(wv, iw)) <= qmax) v += (double)dwq[row * k + c] * (double)wv;
  }
  v = warp_sum(v);
  if (lane == 0) d_iw[row] = v * (double)s_x * (double)s_w[row];
}

__global__ void __launch_bounds__(256) sgd_kernel(float* __restrict__ s, const double* __restrict__ g, double lr, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) s[i] = (float)__dsub_rn((double)s[i], __dmul_rn(lr, g[i]));     // two roundings, as written
}

inline unsigned blocks_for(int64_t count) { return (unsigned)((count + 255) / 256); }

}  // namespace

int launch_act_apply(Ctx* ctx, const float* ylin, const float* res, int64_t ldr, int act, float* y, int64_t rows, int64_t n, cudaStream_t st) {
  if (rows * n == 0) return QCFG_OK;
  act_apply_kernel<<<blocks_for(rows * n), 256, 0, st>>>(ylin, res, ldr, act, y, rows, n);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "activation launch");
}
int launch_loss_grad(Ctx* ctx, const float* y, const float* yref, float coef, float* g, int64_t count, cudaStream_t st) {
  if (count == 0) return QCFG_OK;
  loss_grad_kernel<<<blocks_for(count), 256, 0, st>>>(y, yref, coef, g, count);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "loss gradient launch");
}
int launch_act_backward(Ctx* ctx, float* g, const float* ylin, const float* res, int64_t ldr, int act, int64_t rows, int64_t n, cudaStream_t st) {
  if (rows * n == 0) return QCFG_OK;
  act_backward_kernel<<<blocks_for(rows * n), 256, 0, st>>>(g, ylin, res, ldr, act, rows, n);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "activation backward launch");
}
int launch_col_dot(Ctx* ctx, const float* a, const float* b, int64_t rows, int64_t n, double* out, cudaStream_t st) {
  if (rows * n == 0) return QCFG_OK;
  int64_t gy = (rows + 63) / 64;
  if (gy > 64) gy = 64;
  col_dot_kernel<<<dim3((unsigned)((n + 31) / 32), (unsigned)gy), dim3(32, 8), 0, st>>>(a, b, rows, n, out);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "column reduction launch");
}
int launch_gamma_finish(Ctx* ctx, const double* colsum, const float* s_w, float s_x, int64_t n, double* d_sw, double* d_sx, cudaStream_t st) {
  if (n == 0) return QCFG_OK;
  gamma_finish_kernel<<<blocks_for(n), 256, 0, st>>>(colsum, s_w, s_x, n, d_sw, d_sx);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "scale gradient launch");
}
int launch_scale_cols_bf16(Ctx* ctx, const float* g, const float* col_scale, int64_t rows, int64_t n, void* out, int64_t ld, cudaStream_t st) {
  if (rows * ld == 0) return QCFG_OK;
  scale_cols_bf16_kernel<<<blocks_for(rows * ld), 256, 0, st>>>(g, col_scale, rows, n, reinterpret_cast<__nv_bfloat16*>(out), ld);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "gradient operand launch");
}
int launch_transpose_bf16(Ctx* ctx, const void* src, int kind, int64_t rows, int64_t cols, int64_t ld_src, void* dst, int64_t ld_dst, cudaStream_t st) {
  if (cols == 0 || ld_dst == 0) return QCFG_OK;
  const dim3 grid((unsigned)((ld_dst + 31) / 32), (unsigned)((cols + 31) / 32)), block(32, 8);
  __nv_bfloat16* d = reinterpret_cast<__nv_bfloat16*>(dst);
  if (kind == 0) transpose_bf16_kernel<float><<<grid, block, 0, st>>>(reinterpret_cast<const float*>(src), rows, cols, ld_src, d, ld_dst);
  else if (kind == 1) transpose_bf16_kernel<int8_t><<<grid, block, 0, st>>>(reinterpret_cast<const int8_t*>(src), rows, cols, ld_src, d, ld_dst);
  else transpose_bf16_kernel<__nv_bfloat16><<<grid, block, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(src), rows, cols, ld_src, d, ld_dst);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "transpose launch");
}
int launch_input_backward(Ctx* ctx, const float* dxq, const float* x, int64_t ldx, float s_x, float inv_x, float qmax,
                          int64_t rows, int64_t k, float* gprod, int64_t ldg, double* d_ix, cudaStream_t st) {
  if (rows * k == 0) return QCFG_OK;
  int64_t blocks = (rows * k + 1023) / 1024;
  if (blocks > (int64_t)sm_count(ctx) * 8) blocks = (int64_t)sm_count(ctx) * 8;
  input_backward_kernel<<<(unsigned)blocks, 256, 0, st>>>(dxq, x, ldx, s_x, inv_x, qmax, rows, k, gprod, ldg, d_ix);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "input backward launch");
}
int launch_weight_alpha(Ctx* ctx, const float* dwq, const float* w, const float* s_w, const float* inv_w, float s_x, float qmax,
                        int64_t n, int64_t k, double* d_iw, cudaStream_t st) {
  if (n == 0) return QCFG_OK;
  weight_alpha_kernel<<<(unsigned)((n + 7) / 8), 256, 0, st>>>(dwq, w, s_w, inv_w, s_x, qmax, n, k, d_iw);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "weight scale gradient launch");
}
int launch_sgd(Ctx* ctx, float* s, const double* g, double lr, int64_t n, cudaStream_t st) {
  if (n == 0) return QCFG_OK;
  sgd_kernel<<<blocks_for(n), 256, 0, st>>>(s, g, lr, n);
  count_launch(ctx);
  return check_cuda(ctx, cudaGetLastError(), "scale update launch");
}

}  // namespace qcfg
