// Shared host/device helpers for the qcfg kernels (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/qcfg.h"

namespace qcfg {

// Device error word bits (ORed into the context's error word by kernels).
enum : unsigned { ERR_TIMEOUT = 1u, ERR_NONFINITE = 2u };

struct Ctx;  // defined in api.cu

// ----- context services (api.cu) ------------------------------------------------------
void count_launch(Ctx* ctx, int n = 1);
int set_error(Ctx* ctx, int code, const char* fmt, ...);
int check_cuda(Ctx* ctx, cudaError_t e, const char* what);
unsigned* err_word(Ctx* ctx);
int sm_count(Ctx* ctx);
bool ctx_pair_enabled(Ctx* ctx);
int* pair_cluster_cache(Ctx* ctx);   // [2]: resident CTA pairs of the int8 / bf16 pair kernels, 0 = not yet queried
int device_of(Ctx* ctx);
void*& chain_slot(Ctx* ctx);         // gemm.cu's per-context state
bool ctx_chain_enabled(Ctx* ctx);
void ctx_disable_chains(Ctx* ctx);
int prof_mode(Ctx* ctx);
// grows (never shrinks) the context's scratch buffer; returns nullptr on failure
void* scratch(Ctx* ctx, size_t bytes);
// grows (never shrinks) a host buffer owned by the context; returns nullptr on failure
void* host_scratch(Ctx* ctx, size_t bytes);
// true when the same two host tables were the last ones uploaded to this scratch address on
// this context in this stream (the caller may then skip the upload); records them otherwise
bool sweep_tables_cached(Ctx* ctx, const void* dev_base, cudaStream_t st, const void* a, size_t na, const void* b, size_t nb);
// optional per-launch timing of one kernel class (0 = int8 GEMM, 1 = bf16 GEMM) with CUDA events
void prof_begin(Ctx* ctx, int cls, cudaStream_t st);
void prof_end(Ctx* ctx, int cls, double ops, cudaStream_t st);
// in-kernel time stamps (profile mode 2): a device slot of two 64-bit words the launch's CTAs
// fold their start and end times into, or nullptr when the mode is off or the ring is full
unsigned long long* prof_stamp(Ctx* ctx, int cls, double ops);

// ----- elementwise.cu -----------------------------------------------------------------
int launch_absmax(Ctx* ctx, const float* x, int64_t rows, int64_t cols, int64_t ld,
                  int granularity, float* absmax, cudaStream_t st);
int launch_scales(Ctx* ctx, const float* absmax, int64_t n, int bits, float* scale,
                  float* inv_scale, cudaStream_t st);
// inv_scale_ptr (device) or, when null, inv_scale_val for the whole tensor; with `absmax` set
// (16-bit only) the same launch also leaves max |x| of the tensor there
int launch_quantize(Ctx* ctx, const float* x, int64_t rows, int64_t cols, int64_t ld,
                    const float* inv_scale_ptr, float inv_scale_val, int granularity, int bits,
                    void* q, int64_t ldq, cudaStream_t st, float* absmax = nullptr);

int launch_perturb_bf16(Ctx* ctx, const float* w, const float* nu, const float* amax_dev, float lambda, int64_t rows,
                        int64_t cols, void* q, int64_t ldq, cudaStream_t st);
int launch_sqdiff(Ctx* ctx, const float* y, const float* ref, int64_t n, double* partial, int blocks, cudaStream_t st);

// ----- conv.cu ------------------------------------------------------------------------
int launch_maxpool3s2(Ctx* ctx, const float* src, int64_t B, int H, int W, int C, float* dst, cudaStream_t st);
int launch_avgpool(Ctx* ctx, const float* src, int64_t B, int HW, int C, float* dst, cudaStream_t st);
int launch_im2col_quantize(Ctx* ctx, const float* src, int64_t B, int H, int W, int C, int kh, int kw, int stride,
                           int pad, float inv_scale, int bits, void* q, int64_t ldq, cudaStream_t st);

// patches of int8 codes in (kh, kw, cin) order: dst [B*OH*OW x ldd] from NHWC codes [B*H*W x C] (C % 16 == 0)
int launch_im2col_codes(Ctx* ctx, const int8_t* src, int64_t B, int H, int W, int C, int kh, int kw, int stride, int pad,
                        int8_t* dst, int64_t ldd, cudaStream_t st);

// ----- sweep.cu -----------------------------------------------------------------------
int sweep_init(Ctx* ctx);   // per-device kernel attributes
int launch_sweep(Ctx* ctx, const float* const* w, const int64_t* rows, const int64_t* cols,
                 int32_t n_tensors, int granularity, int b_lo, int b_hi, double* sse,
                 float* absmax, cudaStream_t st);

int launch_sweep_static(Ctx* ctx, const float* const* w, const int64_t* rows, const int64_t* cols,
                        int32_t n_tensors, int granularity, int b_lo, int b_hi, double* sse,
                        float* absmax, cudaStream_t st);

// ----- adjust.cu (scale adjustment, Section 3.1 second step) --------------------------
// y = act(ylin + res) elementwise over [rows x n] (res may be null; ldr its row pitch)
int launch_act_apply(Ctx* ctx, const float* ylin, const float* res, int64_t ldr, int act, float* y, int64_t rows, int64_t n, cudaStream_t st);
// g = coef * (y - yref)
int launch_loss_grad(Ctx* ctx, const float* y, const float* yref, float coef, float* g, int64_t count, cudaStream_t st);
// g *= act'(ylin + res) in place
int launch_act_backward(Ctx* ctx, float* g, const float* ylin, const float* res, int64_t ldr, int act, int64_t rows, int64_t n, cudaStream_t st);
// out[c] += sum_r a[r][c] * b[r][c]   (out must be zeroed by the caller)
int launch_col_dot(Ctx* ctx, const float* a, const float* b, int64_t rows, int64_t n, double* out, cudaStream_t st);
// d_sw[c] = colsum[c] / s_w[c];  *d_sx += sum_c colsum[c] / s_x
int launch_gamma_finish(Ctx* ctx, const double* colsum, const float* s_w, float s_x, int64_t n, double* d_sw, double* d_sx, cudaStream_t st);
// out[r][c] = bf16(g[r][c] * (col_scale ? col_scale[c] : 1)), columns n..ld-1 zero
int launch_scale_cols_bf16(Ctx* ctx, const float* g, const float* col_scale, int64_t rows, int64_t n, void* out, int64_t ld, cudaStream_t st);
// dst[c][r] = bf16(src[r][c]); kind 0 fp32, 1 int8, 2 bf16 source; dst row pitch ld_dst (columns rows..ld_dst-1 zero)
int launch_transpose_bf16(Ctx* ctx, const void* src, int kind, int64_t rows, int64_t cols, int64_t ld_src, void* dst, int64_t ld_dst, cudaStream_t st);
// integer layer: mask = |x*inv_x| <= qmax;  *d_ix += s_x * sum dxq*mask*x;  gprod[r][c] += dxq*(s_x*inv_x)*mask
// 16-bit layer (qmax == 0): gprod += dxq.  gprod may be null (external input).
int launch_input_backward(Ctx* ctx, const float* dxq, const float* x, int64_t ldx, float s_x, float inv_x, float qmax,
                          int64_t rows, int64_t k, float* gprod, int64_t ldg, double* d_ix, cudaStream_t st);
// d_iw[r] = s_x * s_w[r] * sum_c dwq[r][c] * w[r][c] * (|w[r][c]*inv_w[r]| <= qmax)
int launch_weight_alpha(Ctx* ctx, const float* dwq, const float* w, const float* s_w, const float* inv_w, float s_x, float qmax,
                        int64_t n, int64_t k, double* d_iw, cudaStream_t st);
// s[i] = float(double(s[i]) - lr * g[i])
int launch_sgd(Ctx* ctx, float* s, const double* g, double lr, int64_t n, cudaStream_t st);

// ----- gemm.cu ------------------------------------------------------------------------
constexpr int kMaxSlots = 3;
struct CodeSlot {          // one fused re-quantize output of a GEMM epilogue
  void* ptr;               // int8 (kind 1) or bf16 (kind 2) [m x ld]
  int64_t ld;
  float inv_scale;         // consumer's calibrated pre-rounding scale
  float qmax;              // consumer's grid limit
  int kind;                // 0 = unused
};
struct GemmArgs {
  const void* a; int64_t lda;   // [m x lda] int8 or bf16, K-major
  const void* b; int64_t ldb;   // [n x ldb]
  int64_t m, n, k;
  int is_bf16;
  float scale_x;                // int8 only
  const float* scale_w;         // int8 only, [n]
  int act;
  float* y; int64_t ldy;        // optional fp32 output
  const float* residual; int64_t ldr;  // optional fp32 addend (before act)
  int32_t* acc;                 // optional raw accumulators (int8 only) [m x n]
  CodeSlot slots[kMaxSlots];
  float* amax = nullptr;        // optional: max |output| (after shortcut and activation) is folded into *amax, which
                                // the caller has set to zero (calibration: the range of the consumers' input)
  // implicit-GEMM convolution (conv_kh > 0): `a` is the NHWC code tensor [batch*H*W x C] of the layer's
  // input (lda = C), m = batch*OH*OW, k = kh*kw*C; the kernel gathers the patches itself
  int conv_kh = 0, conv_kw = 0, conv_stride = 0, conv_pad = 0, conv_h = 0, conv_w = 0, conv_c = 0;
};
int launch_gemm(Ctx* ctx, const GemmArgs& g, cudaStream_t st);
// up to three GEMMs of equal m, k, operand type and tile width in one launch
bool gemm_groupable(const GemmArgs& a, const GemmArgs& b);
int launch_gemm_group(Ctx* ctx, const GemmArgs* gs, int count, cudaStream_t st);
int gemm_init(Ctx* ctx);   // resolves the tensor-map encoder, sets smem attributes
void gemm_destroy(Ctx* ctx);
// Chains: while one is open, GEMM launches that qualify (pair flavour, 256-column tiles, no
// gather) are collected and go to the device as one launch at the next flush; anything else that
// is put on the stream in between must flush first.
void gemm_chain_open(Ctx* ctx);
int gemm_chain_flush(Ctx* ctx);
int gemm_chain_close(Ctx* ctx);
int gemm_chain_reset(Ctx* ctx);
int launch_wait_timeout(Ctx* ctx, uint64_t limit_ns, cudaStream_t st);

// ----- small device helpers -----------------------------------------------------------
__device__ __forceinline__ unsigned warp_max_u(unsigned v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned t = __shfl_xor_sync(0xffffffffu, v, o);
    v = t > v ? t : v;
  }
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// |x| as an unsigned integer: orders like the float for finite values, and NaN/Inf
// compare above every finite value, so a max over these bits propagates them.
__device__ __forceinline__ unsigned abs_bits(float x) { return __float_as_uint(x) & 0x7fffffffu; }

// tanh-GELU as y / (1 + exp(-2u)), u = sqrt(2/pi) (y + 0.044715 y^3), which equals
// 0.5 y (1 + tanh u).  exp(-2u) = 2^(y (c1 + c3 y^2)) with the constants folded; one ex2 and
// one reciprocal on the special-function unit, five FMA-pipe operations.
__device__ __forceinline__ float gelu_tanh(float y) {
  const float c1 = -2.302208198f;            // -2 sqrt(2/pi) log2(e)
  const float c3 = -0.1029432396f;           // c1 * 0.044715
  float y2 = y * y;
  float t = y * fmaf(c3, y2, c1);
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(t));
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return y * r;
}
__host__ __device__ __forceinline__ float qmax_of(int bits) { return (float)((1 << (bits - 1)) - 1); }

}  // namespace qcfg
