// C-ABI of the library: context, model (layer table, weight-code cache, calibration tables)
// and the host planner that turns one bit configuration into a sequence of kernel launches.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

namespace qcfg {

struct Ctx {
  int device = 0;
  int sms = 0;
  unsigned* err_dev = nullptr;
  void* scratch_buf = nullptr;
  size_t scratch_bytes = 0;
  int64_t launches = 0;
  int fuse = 1;
  int pair = 1;                     // two-CTA GEMM tiles where they apply
  int group = 1;                    // independent GEMMs of equal shape share a launch
  int implicit = 1;                 // convolutions gather their patches inside the GEMM (no im2col matrix)
  int chain = 1;                    // consecutive GEMMs of a forward pass share one cooperative launch
  void* chain_state = nullptr;      // owned by gemm.cu
  int reuse = 0;                    // evaluations restart at the first layer whose bit width changed
  int64_t epoch = 0;                // bumped by every switch that changes which buffers hold what
  int pair_clusters[2] = {0, 0};
  char msg[512] = {0};
  // last sweep tables uploaded to the scratch buffer
  const void* sweep_base = nullptr;
  cudaStream_t sweep_stream = nullptr;
  std::vector<char> sweep_tables;
  std::vector<char> host_buf;       // host-side planning tables
  // per-launch event timing (off by default)
  int prof = 0;
  std::vector<cudaEvent_t> ev;      // pairs: ev[2i] before, ev[2i+1] after
  std::vector<int> ev_cls;
  size_t ev_used = 0;               // pairs in flight
  double prof_ms[3] = {0, 0, 0}, prof_ops[3] = {0, 0, 0};
  int64_t prof_n[3] = {0, 0, 0};
  // in-kernel time stamps (profile mode 2): ring of {earliest start, latest end} pairs
  unsigned long long* stamp_dev = nullptr;
  std::vector<unsigned long long> stamp_host;   // the ring's initial pattern, then its read-back
  std::vector<int> stamp_cls;
  std::vector<double> stamp_ops;
  size_t stamp_used = 0;
  int64_t stamp_dropped = 0;
};

constexpr size_t kProfPairs = 8192;
constexpr size_t kStampSlots = 65536;

static int stamp_reset(Ctx* ctx) {
  for (size_t i = 0; i < kStampSlots; ++i) { ctx->stamp_host[2 * i] = ~0ull; ctx->stamp_host[2 * i + 1] = 0ull; }
  ctx->stamp_used = 0;
  return check_cuda(ctx, cudaMemcpy(ctx->stamp_dev, ctx->stamp_host.data(), kStampSlots * 16, cudaMemcpyHostToDevice), "stamp ring reset");
}
// Waits for the device, folds the stamped launches into the per-class sums and clears the ring.
static int stamp_drain(Ctx* ctx) {
  if (!ctx->stamp_dev || ctx->stamp_used == 0) return QCFG_OK;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(ctx->stamp_host.data(), ctx->stamp_dev, ctx->stamp_used * 16, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return check_cuda(ctx, e, "stamp ring read");
  for (size_t i = 0; i < ctx->stamp_used; ++i) {
    const unsigned long long t0 = ctx->stamp_host[2 * i], t1 = ctx->stamp_host[2 * i + 1];
    if (t1 <= t0) continue;                       // the launch did not run
    const int c = ctx->stamp_cls[i];
    ctx->prof_ms[c] += (double)(t1 - t0) * 1e-6;
    ctx->prof_ops[c] += ctx->stamp_ops[i];
    ctx->prof_n[c] += 1;
  }
  return stamp_reset(ctx);
}
unsigned long long* prof_stamp(Ctx* ctx, int cls, double ops) {
  if (ctx->prof != 2) return nullptr;
  if (ctx->stamp_used == kStampSlots) { ctx->stamp_dropped++; return nullptr; }
  ctx->stamp_cls[ctx->stamp_used] = cls;
  ctx->stamp_ops[ctx->stamp_used] = ops;
  return ctx->stamp_dev + 2 * ctx->stamp_used++;
}

static void prof_drain(Ctx* ctx) {
  if (ctx->ev_used == 0) return;
  cudaEventSynchronize(ctx->ev[2 * ctx->ev_used - 1]);
  for (size_t i = 0; i < ctx->ev_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->ev[2 * i], ctx->ev[2 * i + 1]) == cudaSuccess) {
      ctx->prof_ms[ctx->ev_cls[i]] += ms;
      ctx->prof_n[ctx->ev_cls[i]] += 1;
    }
  }
  ctx->ev_used = 0;
}
void prof_begin(Ctx* ctx, int cls, cudaStream_t st) {
  if (ctx->prof != 1) return;
  if (ctx->ev_used == kProfPairs) prof_drain(ctx);
  ctx->ev_cls[ctx->ev_used] = cls;
  cudaEventRecord(ctx->ev[2 * ctx->ev_used], st);
}
void prof_end(Ctx* ctx, int cls, double ops, cudaStream_t st) {
  if (ctx->prof != 1) return;
  cudaEventRecord(ctx->ev[2 * ctx->ev_used + 1], st);
  ctx->prof_ops[cls] += ops;
  ctx->ev_used += 1;
}

void count_launch(Ctx* ctx, int n) { ctx->launches += n; }
unsigned* err_word(Ctx* ctx) { return ctx->err_dev; }
int sm_count(Ctx* ctx) { return ctx->sms; }
bool ctx_pair_enabled(Ctx* ctx) { return ctx->pair != 0; }
int* pair_cluster_cache(Ctx* ctx) { return ctx->pair_clusters; }
int device_of(Ctx* ctx) { return ctx->device; }
void*& chain_slot(Ctx* ctx) { return ctx->chain_state; }
bool ctx_chain_enabled(Ctx* ctx) { return ctx->chain != 0; }
void ctx_disable_chains(Ctx* ctx) { ctx->chain = 0; }
int prof_mode(Ctx* ctx) { return ctx->prof; }

int set_error(Ctx* ctx, int code, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->msg, sizeof(ctx->msg), fmt, ap);
    va_end(ap);
  }
  return code;
}
int check_cuda(Ctx* ctx, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return QCFG_OK;
  return set_error(ctx, e == cudaErrorMemoryAllocation ? QCFG_ENOMEM : QCFG_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}
bool sweep_tables_cached(Ctx* ctx, const void* dev_base, cudaStream_t st, const void* a, size_t na, const void* b, size_t nb) {
  if (ctx->sweep_base == dev_base && ctx->sweep_stream == st && ctx->sweep_tables.size() == na + nb &&
      memcmp(ctx->sweep_tables.data(), a, na) == 0 && (nb == 0 || memcmp(ctx->sweep_tables.data() + na, b, nb) == 0))
    return true;
  ctx->sweep_tables.resize(na + nb);
  memcpy(ctx->sweep_tables.data(), a, na);
  if (nb) memcpy(ctx->sweep_tables.data() + na, b, nb);
  ctx->sweep_base = dev_base;
  ctx->sweep_stream = st;
  return false;
}
void* host_scratch(Ctx* ctx, size_t bytes) {
  try {
    if (ctx->host_buf.size() < bytes) ctx->host_buf.resize(bytes);
  } catch (...) {
    return nullptr;
  }
  return ctx->host_buf.data();
}
void* scratch(Ctx* ctx, size_t bytes) {
  if (bytes <= ctx->scratch_bytes) return ctx->scratch_buf;
  // the old buffer may still be in use by queued work on some stream
  if (ctx->scratch_buf) { cudaDeviceSynchronize(); cudaFree(ctx->scratch_buf); ctx->scratch_buf = nullptr; ctx->scratch_bytes = 0; }
  size_t want = bytes + bytes / 4 + 4096;
  void* p = nullptr;
  if (cudaMalloc(&p, want) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  ctx->scratch_buf = p;
  ctx->scratch_bytes = want;
  ctx->sweep_base = nullptr;
  return p;
}

namespace {

inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }
inline bool bits_int(int b) { return b >= 2 && b <= 8; }
inline bool bits_ok(int b) { return bits_int(b) || b == 16; }

struct DevBuf {
  void* p = nullptr;
  size_t bytes = 0;
  int ensure(Ctx* ctx, size_t want) {
    if (want <= bytes) return QCFG_OK;
    if (p) { gemm_chain_flush(ctx); cudaDeviceSynchronize(); cudaFree(p); p = nullptr; bytes = 0; }   // nothing deferred may still name p
    cudaError_t e = cudaMalloc(&p, want);
    if (e != cudaSuccess) { cudaGetLastError(); p = nullptr; return set_error(ctx, QCFG_ENOMEM, "cudaMalloc of %zu bytes failed", want); }
    bytes = want;
    return QCFG_OK;
  }
  void release() { if (p) cudaFree(p); p = nullptr; bytes = 0; }
};

struct WeightCodes {
  DevBuf codes;           // int8 or bf16 [n_out x ldk]
  DevBuf scale;           // fp32 [n_out] post-rounding scales (int only)
  DevBuf inv;             // fp32 [n_out] pre-rounding scales (int only)
  bool ready = false;     // codes match the scales
  bool adjusted = false;  // the scales no longer come from the calibrated maxima (scale adjustment)
};

struct LayerState {
  qcfg_layer d;
  int64_t ldk = 0;                 // padded k_in of the code matrices
  DevBuf w_absmax;                 // fp32 [n_out]
  WeightCodes wc[17];              // by bit width
  float act_absmax = 0.0f;         // calibrated max|input|
  // activation scales after scale adjustment, by bit width (otherwise derived from act_absmax)
  bool adj_act[17] = {false};
  float adj_sx[17] = {0}, adj_ix[17] = {0};
  DevBuf ylin, yact, gout, dsw, diw;   // scale adjustment: rescaled accumulators, activated output, dL/d(output), weight scale gradients
  std::vector<int> consumers;      // layers reading this layer's output as GEMM input
  bool feeds_residual = false;
  // per-evaluation state
  int64_t rows = 0;
  DevBuf ybuf;                     // internal fp32 output [rows x n_out]
  DevBuf abuf;                     // GEMM input codes [rows x ldk] (sized for bf16)
  DevBuf prebuf;                   // pooled fp32 input (convolution table only)
  const float* pre_ptr = nullptr;  // pooled input actually used (may alias another layer's prebuf)
  const void* a_ptr = nullptr;     // codes actually used (may alias another layer's abuf)
  const float* y_ptr = nullptr;    // where this layer's fp32 output went (nullptr: not materialised)
  bool a_ready = false;
  bool y_internal = false;         // y_ptr is this layer's own buffer (not the caller's)
  bool implicit = false;           // a_ptr holds the NHWC codes of the input, the GEMM gathers the patches
  int bits = 0;
};

}  // namespace

struct Model {
  Ctx* ctx = nullptr;
  std::vector<LayerState> L;
  bool calibrated = false;
  bool evaluated = false;
  DevBuf act_absmax_dev;           // fp32 [n_layers], filled by calibration
  std::vector<int> calib_same_as;  // layer whose calibrated maximum layer l shares (same input tensor), or -1
  DevBuf search_ref, search_out, search_partial;   // buffers of the search drivers
  DevBuf noise_codes, noise_amax;                  // perturbed bf16 weights of one layer and its max|w|
  DevBuf adj_gs, adj_gt, adj_qxt, adj_qwt, adj_dx, adj_dw, adj_colsum, adj_dscal;   // scale adjustment temporaries
  int64_t last_m = 0;
  // what the layers' buffers hold after the last evaluation (for prefix reuse)
  bool reuse_valid = false;
  const float* reuse_x = nullptr;
  int64_t reuse_m = 0, reuse_epoch = -1;
};

namespace {

int64_t layer_rows(const Model* M, int l, int64_t m_ext) {
  const qcfg_layer& d = M->L[l].d;
  if (d.kh > 0) {
    int64_t oh = (d.in_h + 2 * d.pad - d.kh) / d.stride + 1;
    int64_t ow = (d.in_w + 2 * d.pad - d.kw) / d.stride + 1;
    return m_ext * oh * ow;
  }
  if (d.pool_before == QCFG_POOL_GLOBAL_AVG) return m_ext;
  return d.src < 0 ? m_ext : layer_rows(M, d.src, m_ext);
}

// The layer's GEMM operand is its source's rows as they are (a linear layer, or a 1x1
// convolution with stride 1 and no padding), with no pooling in between.
bool reads_rows_directly(const qcfg_layer& d) {
  return d.pool_before == QCFG_POOL_NONE && (d.kh == 0 || (d.kh == 1 && d.kw == 1 && d.stride == 1 && d.pad == 0));
}
// A convolution whose operand the GEMM can gather from the NHWC codes of its input: not a plain
// row read, and channels in whole 16-byte chunks at either operand width.
bool implicit_capable(const qcfg_layer& d) { return d.kh > 0 && !reads_rows_directly(d) && d.in_c % 16 == 0 && !(d.kh == 1 && d.kw == 1 && d.stride == 1 && d.pad == 0); }
bool same_input(const qcfg_layer& a, const qcfg_layer& b) {
  return a.src == b.src && a.src_col0 == b.src_col0 && a.k_in == b.k_in && a.kh == b.kh && a.kw == b.kw &&
         a.stride == b.stride && a.pad == b.pad && a.pool_before == b.pool_before && a.in_h == b.in_h &&
         a.in_w == b.in_w && a.in_c == b.in_c;
}

// Weight codes and per-row scales for (layer, bits); computed once and kept.
int ensure_weight_codes(Ctx* ctx, LayerState& S, int bits, cudaStream_t st) {
  WeightCodes& W = S.wc[bits];
  if (W.ready) return QCFG_OK;
  const int64_t n = S.d.n_out, k = S.d.k_in;
  int rc = gemm_chain_flush(ctx);      // other kernels follow on the stream
  if (!rc) rc = W.codes.ensure(ctx, (size_t)(n * S.ldk) * (bits == 16 ? 2 : 1));
  if (rc) return rc;
  if (bits == 16) {
    rc = launch_quantize(ctx, S.d.w_dev, n, k, k, nullptr, 1.0f, QCFG_PER_ROW, 16, W.codes.p, S.ldk, st);
  } else {
    rc = W.scale.ensure(ctx, (size_t)n * 4);
    if (!rc) rc = W.inv.ensure(ctx, (size_t)n * 4);
    if (!rc && !W.adjusted) rc = launch_scales(ctx, (const float*)S.w_absmax.p, n, bits, (float*)W.scale.p, (float*)W.inv.p, st);
    if (!rc) rc = launch_quantize(ctx, S.d.w_dev, n, k, k, (const float*)W.inv.p, 1.0f, QCFG_PER_ROW, bits, W.codes.p, S.ldk, st);
  }
  if (rc) return rc;
  W.ready = true;
  return QCFG_OK;
}

// Host copy of the scale rule (one IEEE fp32 division each; the device kernels use __fdiv_rn).
inline void host_scales(float A, int bits, float* scale, float* inv) {
  const float qm = qmax_of(bits);
  if (A == 0.0f) { *scale = 1.0f; *inv = 1.0f; return; }
  volatile float s = A / qm, i = qm / A;
  *scale = s; *inv = i;
}

// The activation scales layer S uses at `bits`: adjusted ones if the adjustment step set them,
// else the max-calibrated ones.
inline void act_scales(const LayerState& S, int bits, float* scale, float* inv) {
  if (S.adj_act[bits]) { *scale = S.adj_sx[bits]; *inv = S.adj_ix[bits]; return; }
  host_scales(S.act_absmax, bits, scale, inv);
}
inline float act_inv(const LayerState& S, int bits) { float s, i; act_scales(S, bits, &s, &i); return i; }

// Row length of the external input: widest slice any layer reads from it (channels for images).
int64_t ext_ld_of(const Model* M) {
  int64_t ld = 0;
  for (auto& S : M->L) {
    if (S.d.src >= 0) continue;
    int64_t w = S.d.kh > 0 ? S.d.in_c : S.d.src_col0 + S.d.k_in;
    if (w > ld) ld = w;
  }
  return ld;
}

// Back to the max-calibrated scales everywhere (after a scale adjustment).
void reset_adjusted_scales(Model* M) {
  for (auto& S : M->L) {
    for (int b = 0; b < 17; ++b) {
      S.adj_act[b] = false;
      if (S.wc[b].adjusted) { S.wc[b].adjusted = false; S.wc[b].ready = false; }
    }
  }
  M->reuse_valid = false;
}

// One forward pass.  calibrate = true: every layer at 16 bit, record max|input| per layer.
int forward(Ctx* ctx, Model* M, const uint8_t* bits, const float* x_dev, int64_t x_ld, int64_t m,
            float* const* y_dev, bool calibrate, cudaStream_t st, cudaEvent_t* layer_ev = nullptr) {
  const int n = (int)M->L.size();
  // GEMM launches of this pass may be collected into chains; every way out closes the chain
  struct ChainScope {
    Ctx* c; bool armed;
    ~ChainScope() { if (armed) gemm_chain_close(c); }
  } scope{ctx, true};
  gemm_chain_open(ctx);
  // Prefix reuse: the layers' buffers still hold the previous evaluation (same input, same rows).
  // A layer is recomputed ("dirty") when its bit width changed, when the caller wants its output,
  // or when a layer it reads was recomputed; everything else keeps its buffers and launches
  // nothing.  A dirty layer that needs new input codes takes them from its producer's fp32
  // output if that was materialised, otherwise the producer is recomputed as well (its epilogue
  // then writes the codes).  The arithmetic of every recomputed layer is the ordinary one, on
  // inputs that are bit-identical to what a full evaluation would produce.
  std::vector<char> dirty((size_t)n, 1);
  const bool reuse = ctx->reuse && !calibrate && !layer_ev && M->reuse_valid && M->reuse_x == x_dev &&
                     M->reuse_m == m && M->reuse_epoch == ctx->epoch;
  if (reuse) {
    std::vector<char> changed((size_t)n, 0);
    for (int l = 0; l < n; ++l) {
      const qcfg_layer& d = M->L[l].d;
      changed[l] = M->L[l].bits != bits[l];
      dirty[l] = changed[l] || (y_dev && y_dev[l]) || (d.src >= 0 && dirty[d.src]) ||
                 (d.residual_from >= 0 && dirty[d.residual_from]);
    }
    for (int l = n - 1; l >= 0; --l) {
      if (!dirty[l]) continue;
      LayerState& S = M->L[l];
      const qcfg_layer& d = S.d;
      if (d.residual_from >= 0 && !dirty[d.residual_from]) {
        LayerState& R = M->L[d.residual_from];
        if (!(R.y_ptr && R.y_internal)) dirty[d.residual_from] = 1;
      }
      if (d.src < 0 || dirty[d.src]) continue;
      LayerState& P = M->L[d.src];
      const bool codes_kept = !changed[l] && S.a_ready && S.a_ptr && S.a_ptr == S.abuf.p;
      if (!codes_kept && !(P.y_ptr && P.y_internal)) dirty[d.src] = 1;
    }
  }
  for (int l = 0; l < n; ++l) {
    LayerState& S = M->L[l];
    S.rows = layer_rows(M, l, m);
    if (!dirty[l]) continue;                         // buffers and pointers stay as they are
    S.implicit = ctx->implicit && !calibrate && implicit_capable(S.d);
    const bool codes_kept = reuse && S.bits == bits[l] && S.a_ready && S.a_ptr && S.a_ptr == S.abuf.p &&
                            (S.d.src < 0 || !dirty[S.d.src]);
    if (!codes_kept) { S.a_ready = false; S.a_ptr = nullptr; }
    S.y_ptr = nullptr; S.pre_ptr = nullptr; S.y_internal = false;
    S.bits = calibrate ? 16 : bits[l];
  }
  M->reuse_valid = false;                            // until this evaluation has been enqueued completely
  if (calibrate) {
    // maxima are folded into the table by atomic max, from epilogues as well: start from zero
    const int zrc = check_cuda(ctx, cudaMemsetAsync(M->act_absmax_dev.p, 0, (size_t)n * 4, st), "calibration table clear");
    if (zrc) return zrc;
    std::fill(M->calib_same_as.begin(), M->calib_same_as.end(), -1);
  }
  // GEMMs that are ready together and have the same m, k, operand type and tile width (the three
  // projections of an attention block) are collected and launched as one grouped kernel.
  std::vector<GemmArgs> pending;
  std::vector<int> pending_layers;
  auto flush = [&]() -> int {
    if (pending.empty()) return QCFG_OK;
    const int frc = launch_gemm_group(ctx, pending.data(), (int)pending.size(), st);
    pending.clear();
    pending_layers.clear();
    return frc;
  };
  const bool grouping = ctx->group && !layer_ev;
  for (int l = 0; l < n; ++l) {
    LayerState& S = M->L[l];
    const qcfg_layer& d = S.d;
    const int b = S.bits;
    if (!dirty[l]) continue;
    for (int pl : pending_layers)
      if (d.src == pl || d.residual_from == pl) {
        // With chained launches the order of independent GEMMs is a free choice, and the best
        // one keeps a GEMM away from the one it reads: only the layers this one reads go out
        // now, with half of the others behind them as a buffer; the rest wait and are launched
        // behind this layer (q, k, v, o: [v, q] now, then [o, k]).
        if (ctx->chain && pending.size() > 1) {
          std::vector<GemmArgs> now, later;
          std::vector<int> now_l, later_l;
          for (size_t i = 0; i < pending.size(); ++i)
            if (d.src == pending_layers[i] || d.residual_from == pending_layers[i]) { now.push_back(pending[i]); now_l.push_back(pending_layers[i]); }
          size_t others = pending.size() - now.size(), taken = 0;
          for (size_t i = 0; i < pending.size(); ++i) {
            if (d.src == pending_layers[i] || d.residual_from == pending_layers[i]) continue;
            if (taken < (others + 1) / 2) { now.push_back(pending[i]); now_l.push_back(pending_layers[i]); ++taken; }
            else { later.push_back(pending[i]); later_l.push_back(pending_layers[i]); }
          }
          const int frc = launch_gemm_group(ctx, now.data(), (int)now.size(), st);
          if (frc) return frc;
          pending.swap(later);
          pending_layers.swap(later_l);
        } else {
          const int frc = flush();
          if (frc) return frc;
        }
        break;
      }
    int rc = ensure_weight_codes(ctx, S, b, st);
    if (rc) return rc;
    // optional per-layer timing: everything this layer launches (operand preparation and GEMM)
    if (layer_ev) {
      rc = gemm_chain_flush(ctx);
      if (rc) return rc;
      if (cudaEventRecord(layer_ev[2 * l], st) != cudaSuccess) return check_cuda(ctx, cudaGetLastError(), "event record");
    }

    // ---- GEMM input codes
    if (!S.a_ready) {
      rc = gemm_chain_flush(ctx);      // the kernels below follow the deferred GEMMs on the stream
      if (rc) return rc;
      // the fp32 tensor this layer reads: [srows x sld], NHWC for the convolutional table
      const float* sp; int64_t sld, srows;
      if (d.src < 0) {
        sp = x_dev; sld = x_ld;
        srows = d.kh > 0 || d.pool_before != QCFG_POOL_NONE ? m * (int64_t)d.src_h * d.src_w : m;
      } else {
        LayerState& P = M->L[d.src];
        if (!P.y_ptr) return set_error(ctx, QCFG_ESTATE, "layer %d: producer %d output not materialised", l, d.src);
        sp = P.y_ptr; sld = P.d.n_out; srows = P.rows;
      }
      if (d.pool_before != QCFG_POOL_NONE) {
        if (m * (int64_t)d.src_h * d.src_w != srows)
          return set_error(ctx, QCFG_ESHAPE, "layer %d: source has %lld rows, src_h*src_w*m = %lld", l, (long long)srows,
                           (long long)(m * (int64_t)d.src_h * d.src_w));
        const int64_t prows = d.pool_before == QCFG_POOL_MAX3S2
                                  ? m * (int64_t)((d.src_h - 1) / 2 + 1) * ((d.src_w - 1) / 2 + 1) : m;
        for (int j = 0; j < l && !S.pre_ptr; ++j) {
          LayerState& T = M->L[j];
          if (T.pre_ptr && T.d.src == d.src && T.d.pool_before == d.pool_before && T.d.src_h == d.src_h && T.d.src_w == d.src_w)
            S.pre_ptr = T.pre_ptr;
        }
        if (!S.pre_ptr) {
          rc = S.prebuf.ensure(ctx, (size_t)(prows * sld) * 4);
          if (rc) return rc;
          if (d.pool_before == QCFG_POOL_MAX3S2)
            rc = launch_maxpool3s2(ctx, sp, m, d.src_h, d.src_w, (int)sld, (float*)S.prebuf.p, st);
          else
            rc = launch_avgpool(ctx, sp, m, d.src_h * d.src_w, (int)sld, (float*)S.prebuf.p, st);
          if (rc) return rc;
          S.pre_ptr = (const float*)S.prebuf.p;
        }
        sp = S.pre_ptr; srows = prows;
      }
      const bool direct = d.kh == 0 || (d.kh == 1 && d.kw == 1 && d.stride == 1 && d.pad == 0);
      if (d.kh > 0) {
        if (sld != d.in_c || srows != m * (int64_t)d.in_h * d.in_w)
          return set_error(ctx, QCFG_ESHAPE, "layer %d: convolution input is [%lld x %lld], expected [%lld x %d]", l,
                           (long long)srows, (long long)sld, (long long)(m * (int64_t)d.in_h * d.in_w), d.in_c);
      } else if (srows != S.rows) {
        return set_error(ctx, QCFG_ESHAPE, "layer %d: source rows %lld differ from layer rows %lld", l, (long long)srows, (long long)S.rows);
      }
      const int64_t width = d.kh > 0 ? d.in_c : d.k_in;       // columns of the tensor that is calibrated
      const float* tp = sp + (d.kh > 0 ? 0 : d.src_col0);
      // calibration: a tensor that is also turned into a 16-bit row operand below gets its range
      // from that same launch; one that an earlier layer already read takes that layer's value
      bool range_pending = calibrate;
      if (calibrate) M->calib_same_as[l] = -1;
      if (calibrate && !(direct && !S.implicit)) {
        rc = launch_absmax(ctx, tp, srows, width, sld, QCFG_PER_TENSOR, (float*)M->act_absmax_dev.p + l, st);
        if (rc) return rc;
        range_pending = false;
      }
      // reuse the codes of an earlier layer that reads the same input with the same grid
      int share = -1;
      for (int j = 0; j < l && share < 0; ++j) {
        LayerState& T = M->L[j];
        if (same_input(T.d, d) && T.bits == b && T.a_ptr && (b == 16 || act_inv(T, b) == act_inv(S, b)) &&
            (dirty[j] || T.a_ptr == T.abuf.p))       // a skipped layer's codes are trusted only in its own buffer
          share = j;
      }
      if (share >= 0) {
        S.a_ptr = M->L[share].a_ptr;
        if (range_pending) {
          // same tensor, same maximum; a chain of sharers ends at the layer that measured it
          if (M->calib_same_as[share] >= 0 || (reads_rows_directly(M->L[share].d) && !M->L[share].implicit)) {
            M->calib_same_as[l] = M->calib_same_as[share] >= 0 ? M->calib_same_as[share] : share;
          } else {
            rc = launch_absmax(ctx, tp, srows, width, sld, QCFG_PER_TENSOR, (float*)M->act_absmax_dev.p + l, st);
            if (rc) return rc;
          }
        }
      } else {
        rc = S.abuf.ensure(ctx, (size_t)(S.implicit ? srows * d.in_c : S.rows * S.ldk) * 2);
        if (rc) return rc;
        float sc = 1.0f, inv = 1.0f;
        if (b != 16) act_scales(S, b, &sc, &inv);
        if (S.implicit)      // the input tensor's own codes, NHWC; the GEMM gathers the patches
          rc = launch_quantize(ctx, sp, srows, d.in_c, sld, nullptr, inv, QCFG_PER_TENSOR, b, S.abuf.p, d.in_c, st);
        else if (direct)
          rc = launch_quantize(ctx, tp, S.rows, d.k_in, sld, nullptr, inv, QCFG_PER_TENSOR, b, S.abuf.p, S.ldk, st,
                               range_pending ? (float*)M->act_absmax_dev.p + l : nullptr);
        else
          rc = launch_im2col_quantize(ctx, sp, m, d.in_h, d.in_w, d.in_c, d.kh, d.kw, d.stride, d.pad, inv, b, S.abuf.p, S.ldk, st);
        if (rc) return rc;
        S.a_ptr = S.abuf.p;
      }
      S.a_ready = true;
    }

    // ---- GEMM + epilogue
    GemmArgs g{};
    g.a = S.a_ptr; g.lda = S.ldk;
    g.b = S.wc[b].codes.p; g.ldb = S.ldk;
    g.m = S.rows; g.n = S.d.n_out; g.k = S.d.k_in;
    g.is_bf16 = b == 16;
    g.act = S.d.act;
    if (S.implicit) {
      g.lda = d.in_c;
      g.conv_kh = d.kh; g.conv_kw = d.kw; g.conv_stride = d.stride; g.conv_pad = d.pad;
      g.conv_h = d.in_h; g.conv_w = d.in_w; g.conv_c = d.in_c;
    }
    if (b != 16) {
      float sx, ix;
      act_scales(S, b, &sx, &ix);
      g.scale_x = sx;
      g.scale_w = (const float*)S.wc[b].scale.p;
    }
    // fused re-quantize outputs for consumers whose input is this whole output
    bool all_fused = !S.consumers.empty();
    int nslots = 0, first_ranged = -1;
    for (int c : S.consumers) {
      LayerState& C = M->L[c];
      const int cb = calibrate ? 16 : bits[c];
      // a consumer whose operand is this whole output: a plain row read, or a convolution the GEMM gathers for
      const bool c_implicit = ctx->implicit && !calibrate && implicit_capable(C.d) && C.d.pool_before == QCFG_POOL_NONE;
      // (in the calibration forward the epilogue also takes the range of what the consumer reads)
      const bool fusable = ctx->fuse && C.d.src_col0 == 0 &&
                           ((reads_rows_directly(C.d) && C.d.k_in == S.d.n_out) || (!calibrate && c_implicit && C.d.in_c == S.d.n_out));
      if (!fusable) { all_fused = false; continue; }
      const int64_t c_ld = c_implicit ? C.d.in_c : C.ldk;
      float csc = 1.0f, cinv = 1.0f;
      if (cb != 16) act_scales(C, cb, &csc, &cinv);
      // an existing slot with the same grid serves this consumer too
      int found = -1;
      for (int s = 0; s < nslots; ++s)
        if (g.slots[s].ld == c_ld &&
            ((cb == 16 && g.slots[s].kind == 2) || (cb != 16 && g.slots[s].kind == 1 && g.slots[s].inv_scale == cinv && g.slots[s].qmax == qmax_of(cb))))
          found = s;
      if (found < 0) {
        if (nslots == kMaxSlots) { all_fused = false; continue; }
        rc = C.abuf.ensure(ctx, (size_t)(S.rows * c_ld) * 2);
        if (rc) return rc;
        g.slots[nslots].ptr = C.abuf.p;
        g.slots[nslots].ld = c_ld;
        g.slots[nslots].inv_scale = cinv;
        g.slots[nslots].qmax = cb == 16 ? 0.0f : qmax_of(cb);
        g.slots[nslots].kind = cb == 16 ? 2 : 1;
        found = nslots++;
      }
      C.a_ptr = g.slots[found].ptr;
      C.a_ready = true;
      C.bits = cb;
      C.implicit = c_implicit;
      if (calibrate) {      // one maximum per output tensor; further readers of it take the first one's
        if (!g.amax) { g.amax = (float*)M->act_absmax_dev.p + c; first_ranged = c; M->calib_same_as[c] = -1; }
        else M->calib_same_as[c] = first_ranged;
      }
    }
    float* y_out = (y_dev && y_dev[l]) ? y_dev[l] : nullptr;
    const bool need_y = y_out || !all_fused || S.feeds_residual;
    if (need_y && !y_out) {
      rc = S.ybuf.ensure(ctx, (size_t)(S.rows * S.d.n_out) * 4);
      if (rc) return rc;
      y_out = (float*)S.ybuf.p;
    }
    g.y = y_out; g.ldy = S.d.n_out;
    S.y_ptr = y_out;
    S.y_internal = y_out && y_out == (float*)S.ybuf.p;
    if (d.residual_from >= 0) {
      LayerState& R = M->L[d.residual_from];
      if (!R.y_ptr || R.rows != S.rows) return set_error(ctx, QCFG_ESHAPE, "layer %d: shortcut from layer %d is unavailable or has other rows", l, d.residual_from);
      g.residual = R.y_ptr; g.ldr = R.d.n_out;
    }
    if (grouping) {
      if (!pending.empty() && (pending.size() == 3 || !gemm_groupable(pending[0], g))) { rc = flush(); if (rc) return rc; }
      pending.push_back(g);
      pending_layers.push_back(l);
    } else {
      rc = launch_gemm(ctx, g, st);
      if (rc) return rc;
    }
    if (layer_ev) {
      rc = gemm_chain_flush(ctx);
      if (rc) return rc;
      if (cudaEventRecord(layer_ev[2 * l + 1], st) != cudaSuccess) return check_cuda(ctx, cudaGetLastError(), "event record");
    }
  }
  int frc = flush();
  const int crc = gemm_chain_close(ctx);
  scope.armed = false;
  if (frc == QCFG_OK) frc = crc;
  if (frc == QCFG_OK && !calibrate && !layer_ev) {
    M->reuse_valid = true; M->reuse_x = x_dev; M->reuse_m = m; M->reuse_epoch = ctx->epoch;
  }
  return frc;
}

}  // namespace
}  // namespace qcfg

using namespace qcfg;

struct qcfg_ctx { Ctx c; };
struct qcfg_model { Model m; };

extern "C" {

int qcfg_create(qcfg_ctx** out, int device) {
  if (!out) return QCFG_EINVAL;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) { cudaGetLastError(); return QCFG_ECUDA; }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return QCFG_ECUDA;
  if (prop.major != 10) return QCFG_EARCH;
  if (cudaSetDevice(device) != cudaSuccess) return QCFG_ECUDA;
  qcfg_ctx* h = new (std::nothrow) qcfg_ctx();
  if (!h) return QCFG_ENOMEM;
  h->c.device = device;
  h->c.sms = prop.multiProcessorCount;
  if (cudaMalloc(&h->c.err_dev, sizeof(unsigned)) != cudaSuccess || cudaMemset(h->c.err_dev, 0, sizeof(unsigned)) != cudaSuccess) {
    delete h;
    return QCFG_ENOMEM;
  }
  int rc = gemm_init(&h->c);
  if (!rc) rc = sweep_init(&h->c);
  if (rc) { gemm_destroy(&h->c); cudaFree(h->c.err_dev); delete h; return rc; }
  *out = h;
  return QCFG_OK;
}

int qcfg_destroy(qcfg_ctx* ctx) {
  if (!ctx) return QCFG_EINVAL;
  cudaDeviceSynchronize();
  for (auto& e : ctx->c.ev) cudaEventDestroy(e);
  if (ctx->c.scratch_buf) cudaFree(ctx->c.scratch_buf);
  if (ctx->c.stamp_dev) cudaFree(ctx->c.stamp_dev);
  if (ctx->c.err_dev) cudaFree(ctx->c.err_dev);
  gemm_destroy(&ctx->c);
  delete ctx;
  return QCFG_OK;
}

int qcfg_sync_status(qcfg_ctx* ctx, void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return check_cuda(c, e, "stream synchronize");
  unsigned w = 0;
  e = cudaMemcpy(&w, c->err_dev, sizeof(w), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return check_cuda(c, e, "error word read");
  if (w) {
    cudaMemset(c->err_dev, 0, sizeof(w));
    gemm_chain_reset(c);
    if (w & ERR_TIMEOUT) return set_error(c, QCFG_ETIMEOUT, "a bounded device-side wait gave up");
    if (w & ERR_NONFINITE) return set_error(c, QCFG_ENONFINITE, "non-finite value found on the device");
  }
  return QCFG_OK;
}

int qcfg_selftest_wait_timeout(qcfg_ctx* ctx, uint64_t limit_ns, void* stream) {
  if (!ctx) return QCFG_EINVAL;
  if (limit_ns == 0 || limit_ns > 100000000ull) return set_error(&ctx->c, QCFG_EINVAL, "selftest: limit must be 1 ns .. 100 ms");
  return launch_wait_timeout(&ctx->c, limit_ns, (cudaStream_t)stream);
}

const char* qcfg_last_error(qcfg_ctx* ctx) { return ctx ? ctx->c.msg : "null context"; }
int64_t qcfg_launch_count(qcfg_ctx* ctx) { return ctx ? ctx->c.launches : 0; }
int qcfg_profile_enable(qcfg_ctx* ctx, int enabled) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (enabled < 0 || enabled > 2) return set_error(c, QCFG_EINVAL, "profile: mode must be 0, 1 or 2");
  if (enabled == 1 && c->ev.empty()) {
    c->ev.resize(2 * kProfPairs);
    c->ev_cls.resize(kProfPairs);
    for (auto& e : c->ev)
      if (cudaEventCreate(&e) != cudaSuccess) return set_error(c, QCFG_ECUDA, "profile: event creation failed");
  }
  if (enabled == 2 && !c->stamp_dev) {
    if (cudaMalloc(&c->stamp_dev, kStampSlots * 16) != cudaSuccess) { cudaGetLastError(); return set_error(c, QCFG_ENOMEM, "profile: stamp ring"); }
    c->stamp_host.resize(2 * kStampSlots);
    c->stamp_cls.resize(kStampSlots);
    c->stamp_ops.resize(kStampSlots);
    const int rc = stamp_reset(c);
    if (rc) return rc;
  }
  if (c->prof == 1 && enabled != 1) prof_drain(c);
  if (c->prof == 2 && enabled != 2) { const int rc = stamp_drain(c); if (rc) return rc; }
  c->prof = enabled;
  return QCFG_OK;
}
int qcfg_profile_read(qcfg_ctx* ctx, int kernel_class, double* ms, int64_t* launches, double* ops, int reset) {
  if (!ctx || kernel_class < 0 || kernel_class > 2) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  prof_drain(c);
  { const int rc = stamp_drain(c); if (rc) return rc; }
  if (ms) *ms = c->prof_ms[kernel_class];
  if (launches) *launches = c->prof_n[kernel_class];
  if (ops) *ops = c->prof_ops[kernel_class];
  if (reset) { c->prof_ms[kernel_class] = 0; c->prof_n[kernel_class] = 0; c->prof_ops[kernel_class] = 0; }
  return QCFG_OK;
}
int qcfg_set_pair_tiles(qcfg_ctx* ctx, int enabled) {
  if (!ctx) return QCFG_EINVAL;
  ctx->c.pair = enabled ? 1 : 0;
  ctx->c.epoch++;
  return QCFG_OK;
}
int qcfg_set_grouping(qcfg_ctx* ctx, int enabled) {
  if (!ctx) return QCFG_EINVAL;
  ctx->c.group = enabled ? 1 : 0;
  ctx->c.epoch++;
  return QCFG_OK;
}
int qcfg_set_fusion(qcfg_ctx* ctx, int enabled) {
  if (!ctx) return QCFG_EINVAL;
  ctx->c.fuse = enabled ? 1 : 0;
  ctx->c.epoch++;
  return QCFG_OK;
}
int qcfg_set_implicit_conv(qcfg_ctx* ctx, int enabled) {
  if (!ctx) return QCFG_EINVAL;
  ctx->c.implicit = enabled ? 1 : 0;
  ctx->c.epoch++;
  return QCFG_OK;
}
int qcfg_set_gemm_chains(qcfg_ctx* ctx, int enabled) {
  if (!ctx) return QCFG_EINVAL;
  ctx->c.chain = enabled ? 1 : 0;
  return QCFG_OK;
}
int qcfg_set_prefix_reuse(qcfg_ctx* ctx, int enabled) {
  if (!ctx) return QCFG_EINVAL;
  ctx->c.reuse = enabled ? 1 : 0;
  ctx->c.epoch++;
  return QCFG_OK;
}

int qcfg_calibrate(qcfg_ctx* ctx, const float* x_dev, int64_t rows, int64_t cols, int64_t ld, int granularity,
                   float* absmax_dev, void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (!absmax_dev || rows < 0 || cols < 0 || (rows * cols > 0 && !x_dev)) return set_error(c, QCFG_EINVAL, "calibrate: null pointer or negative size");
  if (granularity != QCFG_PER_TENSOR && granularity != QCFG_PER_ROW) return set_error(c, QCFG_EINVAL, "calibrate: bad granularity");
  if (ld < cols) return set_error(c, QCFG_ESHAPE, "calibrate: ld < cols");
  if ((uintptr_t)x_dev % 4 || (uintptr_t)absmax_dev % 4) return set_error(c, QCFG_EALIGN, "calibrate: pointers must be 4-byte aligned");
  return launch_absmax(c, x_dev, rows, cols, ld, granularity, absmax_dev, (cudaStream_t)stream);
}

int qcfg_scales_from_absmax(qcfg_ctx* ctx, const float* absmax_dev, int64_t n, int bits, float* scale_dev,
                            float* inv_scale_dev, void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (!absmax_dev || n < 0) return set_error(c, QCFG_EINVAL, "scales: null pointer or negative size");
  if (!bits_int(bits)) return set_error(c, QCFG_EBITS, "scales: bits must be 2..8, got %d", bits);
  return launch_scales(c, absmax_dev, n, bits, scale_dev, inv_scale_dev, (cudaStream_t)stream);
}

int qcfg_quantize(qcfg_ctx* ctx, const float* x_dev, int64_t rows, int64_t cols, int64_t ld, const float* inv_scale_dev,
                  int granularity, int bits, void* q_dev, int64_t ldq, void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (!x_dev || !q_dev || rows < 0 || cols < 0) return set_error(c, QCFG_EINVAL, "quantize: null pointer or negative size");
  if (!bits_ok(bits)) return set_error(c, QCFG_EBITS, "quantize: bits must be 2..8 or 16, got %d", bits);
  if (bits != 16 && !inv_scale_dev) return set_error(c, QCFG_EINVAL, "quantize: inv_scale_dev is null");
  if (granularity != QCFG_PER_TENSOR && granularity != QCFG_PER_ROW) return set_error(c, QCFG_EINVAL, "quantize: bad granularity");
  if (ld < cols || ldq < cols) return set_error(c, QCFG_ESHAPE, "quantize: leading dimension below cols");
  if (ldq % 16 || (uintptr_t)q_dev % 16 || (uintptr_t)x_dev % 4) return set_error(c, QCFG_EALIGN, "quantize: q_dev must be 16-byte aligned with ldq a multiple of 16");
  return launch_quantize(c, x_dev, rows, cols, ld, inv_scale_dev, 1.0f, granularity, bits, q_dev, ldq, (cudaStream_t)stream);
}

int qcfg_quant_error_sweep(qcfg_ctx* ctx, const float* const* w_dev, const int64_t* rows, const int64_t* cols,
                           int32_t n_tensors, int granularity, int b_lo, int b_hi, double* sse_dev, float* absmax_dev,
                           void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (n_tensors < 0 || !sse_dev || !absmax_dev || (n_tensors > 0 && (!w_dev || !rows || !cols)))
    return set_error(c, QCFG_EINVAL, "sweep: null pointer or negative count");
  if (!bits_int(b_lo) || !bits_int(b_hi) || b_lo > b_hi) return set_error(c, QCFG_EBITS, "sweep: bit range must lie in 2..8");
  if (granularity != QCFG_PER_TENSOR && granularity != QCFG_PER_ROW) return set_error(c, QCFG_EINVAL, "sweep: bad granularity");
  for (int t = 0; t < n_tensors; ++t) {
    if (rows[t] < 0 || cols[t] < 0 || cols[t] > 0x7fffffff) return set_error(c, QCFG_ESHAPE, "sweep: tensor %d has a bad shape", t);
    if (rows[t] * cols[t] > 0 && !w_dev[t]) return set_error(c, QCFG_EINVAL, "sweep: tensor %d is null", t);
    if ((uintptr_t)w_dev[t] % 4) return set_error(c, QCFG_EALIGN, "sweep: tensor %d is not 4-byte aligned", t);
  }
  return launch_sweep(c, w_dev, rows, cols, n_tensors, granularity, b_lo, b_hi, sse_dev, absmax_dev, (cudaStream_t)stream);
}

int qcfg_quant_error_sweep_static(qcfg_ctx* ctx, const float* const* w_dev, const int64_t* rows, const int64_t* cols,
                                  int32_t n_tensors, int granularity, int b_lo, int b_hi, double* sse_dev,
                                  float* absmax_dev, void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (n_tensors < 0 || !sse_dev || !absmax_dev || (n_tensors > 0 && (!w_dev || !rows || !cols)))
    return set_error(c, QCFG_EINVAL, "static sweep: null pointer or negative count");
  if (!bits_int(b_lo) || !bits_int(b_hi) || b_lo > b_hi) return set_error(c, QCFG_EBITS, "static sweep: bit range must lie in 2..8");
  if (granularity != QCFG_PER_TENSOR && granularity != QCFG_PER_ROW) return set_error(c, QCFG_EINVAL, "static sweep: bad granularity");
  for (int t = 0; t < n_tensors; ++t) {
    if (rows[t] < 0 || cols[t] < 0 || cols[t] > 0x7fffffff) return set_error(c, QCFG_ESHAPE, "static sweep: tensor %d has a bad shape", t);
    if (rows[t] * cols[t] > 0 && !w_dev[t]) return set_error(c, QCFG_EINVAL, "static sweep: tensor %d is null", t);
    if ((uintptr_t)w_dev[t] % 4) return set_error(c, QCFG_EALIGN, "static sweep: tensor %d is not 4-byte aligned", t);
  }
  return launch_sweep_static(c, w_dev, rows, cols, n_tensors, granularity, b_lo, b_hi, sse_dev, absmax_dev, (cudaStream_t)stream);
}

int qcfg_gemm_i8(qcfg_ctx* ctx, const int8_t* qx_dev, int64_t ldx, const int8_t* qw_dev, int64_t ldw, int64_t m,
                 int64_t n, int64_t k, float scale_x, const float* scale_w_dev, int act, float* y_dev, int32_t* acc_dev,
                 void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (!qx_dev || !qw_dev || (!y_dev && !acc_dev) || (y_dev && !scale_w_dev)) return set_error(c, QCFG_EINVAL, "gemm_i8: null pointer");
  if (act < QCFG_ACT_NONE || act > QCFG_ACT_GELU_TANH) return set_error(c, QCFG_EINVAL, "gemm_i8: bad activation");
  if ((uintptr_t)y_dev % 4 || (uintptr_t)acc_dev % 4 || (uintptr_t)scale_w_dev % 4) return set_error(c, QCFG_EALIGN, "gemm_i8: outputs must be 4-byte aligned");
  GemmArgs g{};
  g.a = qx_dev; g.lda = ldx; g.b = qw_dev; g.ldb = ldw; g.m = m; g.n = n; g.k = k;
  g.is_bf16 = 0; g.scale_x = scale_x; g.scale_w = scale_w_dev; g.act = act;
  g.y = y_dev; g.ldy = n; g.acc = acc_dev;
  if (!scale_w_dev) {   // accumulators only: the rescale is skipped by giving it nothing to write
    g.y = nullptr;
  }
  return launch_gemm(c, g, (cudaStream_t)stream);
}

int qcfg_gemm_i8_requant(qcfg_ctx* ctx, const int8_t* qx_dev, int64_t ldx, const int8_t* qw_dev, int64_t ldw, int64_t m,
                         int64_t n, int64_t k, float scale_x, const float* scale_w_dev, int act, float next_inv_scale,
                         int next_bits, void* q_out_dev, int64_t ldq, void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (!qx_dev || !qw_dev || !scale_w_dev || !q_out_dev) return set_error(c, QCFG_EINVAL, "gemm_i8_requant: null pointer");
  if (act < QCFG_ACT_NONE || act > QCFG_ACT_GELU_TANH) return set_error(c, QCFG_EINVAL, "gemm_i8_requant: bad activation");
  if (!bits_ok(next_bits)) return set_error(c, QCFG_EBITS, "gemm_i8_requant: next_bits must be 2..8 or 16, got %d", next_bits);
  if (ldq < n) return set_error(c, QCFG_ESHAPE, "gemm_i8_requant: ldq < n");
  if (ldq % 16 || (uintptr_t)q_out_dev % 16 || (uintptr_t)scale_w_dev % 4) return set_error(c, QCFG_EALIGN, "gemm_i8_requant: q_out_dev must be 16-byte aligned with ldq a multiple of 16");
  GemmArgs g{};
  g.a = qx_dev; g.lda = ldx; g.b = qw_dev; g.ldb = ldw; g.m = m; g.n = n; g.k = k;
  g.is_bf16 = 0; g.scale_x = scale_x; g.scale_w = scale_w_dev; g.act = act;
  g.slots[0].ptr = q_out_dev; g.slots[0].ld = ldq; g.slots[0].inv_scale = next_inv_scale;
  g.slots[0].qmax = next_bits == 16 ? 0.0f : qmax_of(next_bits);
  g.slots[0].kind = next_bits == 16 ? 2 : 1;
  return launch_gemm(c, g, (cudaStream_t)stream);
}

int qcfg_gemm_bf16(qcfg_ctx* ctx, const void* x_bf16_dev, int64_t ldx, const void* w_bf16_dev, int64_t ldw, int64_t m,
                   int64_t n, int64_t k, int act, float* y_dev, void* stream) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (!x_bf16_dev || !w_bf16_dev || !y_dev) return set_error(c, QCFG_EINVAL, "gemm_bf16: null pointer");
  if (act < QCFG_ACT_NONE || act > QCFG_ACT_GELU_TANH) return set_error(c, QCFG_EINVAL, "gemm_bf16: bad activation");
  if ((uintptr_t)y_dev % 4) return set_error(c, QCFG_EALIGN, "gemm_bf16: y_dev must be 4-byte aligned");
  GemmArgs g{};
  g.a = x_bf16_dev; g.lda = ldx; g.b = w_bf16_dev; g.ldb = ldw; g.m = m; g.n = n; g.k = k;
  g.is_bf16 = 1; g.act = act; g.y = y_dev; g.ldy = n;
  return launch_gemm(c, g, (cudaStream_t)stream);
}

int qcfg_model_create(qcfg_ctx* ctx, const qcfg_layer* layers, int32_t n_layers, qcfg_model** out) {
  if (!ctx) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  if (!out) return set_error(c, QCFG_EINVAL, "model_create: out is null");
  *out = nullptr;
  if (!layers || n_layers <= 0) return set_error(c, QCFG_EINVAL, "model_create: no layers");
  for (int l = 0; l < n_layers; ++l) {
    const qcfg_layer& d = layers[l];
    if (!d.w_dev || d.n_out <= 0 || d.k_in <= 0) return set_error(c, QCFG_EINVAL, "layer %d: null weight or empty shape", l);
    if ((uintptr_t)d.w_dev % 4) return set_error(c, QCFG_EALIGN, "layer %d: weight pointer not 4-byte aligned", l);
    if (d.src >= l || d.src < -1 || d.residual_from >= l || d.residual_from < -1) return set_error(c, QCFG_ESHAPE, "layer %d: src / residual_from must be earlier layers", l);
    if (d.act < QCFG_ACT_NONE || d.act > QCFG_ACT_GELU_TANH) return set_error(c, QCFG_EINVAL, "layer %d: bad activation", l);
    if (d.src_col0 < 0) return set_error(c, QCFG_ESHAPE, "layer %d: negative src_col0", l);
    if (d.kh == 0 && d.src >= 0 && d.src_col0 + d.k_in > layers[d.src].n_out)
      return set_error(c, QCFG_ESHAPE, "layer %d: reads columns beyond its producer's output", l);
    if (d.kh > 0 && (d.kw <= 0 || d.stride <= 0 || d.pad < 0 || d.in_h <= 0 || d.in_w <= 0 || d.in_c <= 0 ||
                     (int64_t)d.kh * d.kw * d.in_c != d.k_in))
      return set_error(c, QCFG_ESHAPE, "layer %d: inconsistent convolution geometry", l);
    if (d.pool_before != QCFG_POOL_NONE && (d.pool_before < 0 || d.pool_before > QCFG_POOL_GLOBAL_AVG || d.src_h <= 0 || d.src_w <= 0))
      return set_error(c, QCFG_ESHAPE, "layer %d: pooling needs src_h and src_w", l);
    if (d.kh > 0 && d.src >= 0 && layers[d.src].n_out != d.in_c) return set_error(c, QCFG_ESHAPE, "layer %d: in_c differs from its producer's width", l);
    if (d.residual_from >= 0 && layers[d.residual_from].n_out != d.n_out) return set_error(c, QCFG_ESHAPE, "layer %d: shortcut width differs", l);
  }
  qcfg_model* h = new (std::nothrow) qcfg_model();
  if (!h) return set_error(c, QCFG_ENOMEM, "model_create: host allocation failed");
  Model* M = &h->m;
  M->ctx = c;
  M->L.resize(n_layers);
  M->calib_same_as.assign(n_layers, -1);
  int rc = M->act_absmax_dev.ensure(c, (size_t)n_layers * 4);
  for (int l = 0; l < n_layers && !rc; ++l) {
    LayerState& S = M->L[l];
    S.d = layers[l];
    S.ldk = round_up(S.d.k_in, 16);
    if (S.d.src >= 0) M->L[S.d.src].consumers.push_back(l);
    if (S.d.residual_from >= 0) M->L[S.d.residual_from].feeds_residual = true;
    rc = S.w_absmax.ensure(c, (size_t)S.d.n_out * 4);
    if (!rc) rc = launch_absmax(c, S.d.w_dev, S.d.n_out, S.d.k_in, S.d.k_in, QCFG_PER_ROW, (float*)S.w_absmax.p, 0);
  }
  if (!rc) rc = check_cuda(c, cudaStreamSynchronize(0), "model_create sync");
  if (rc) { qcfg_model_destroy(h); return rc; }
  *out = h;
  return QCFG_OK;
}

int qcfg_model_destroy(qcfg_model* model) {
  if (!model) return QCFG_EINVAL;
  cudaDeviceSynchronize();
  Model* M = &model->m;
  for (auto& S : M->L) {
    S.w_absmax.release(); S.ybuf.release(); S.abuf.release(); S.prebuf.release();
    S.ylin.release(); S.yact.release(); S.gout.release(); S.dsw.release(); S.diw.release();
    for (auto& W : S.wc) { W.codes.release(); W.scale.release(); W.inv.release(); }
  }
  M->act_absmax_dev.release();
  M->search_ref.release(); M->search_out.release(); M->search_partial.release();
  M->noise_codes.release(); M->noise_amax.release();
  M->adj_gs.release(); M->adj_gt.release(); M->adj_qxt.release(); M->adj_qwt.release();
  M->adj_dx.release(); M->adj_dw.release(); M->adj_colsum.release(); M->adj_dscal.release();
  delete model;
  return QCFG_OK;
}

int qcfg_calibrate_model(qcfg_ctx* ctx, qcfg_model* model, const float* x_dev, int64_t m, void* stream) {
  if (!ctx || !model) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  Model* M = &model->m;
  if (!x_dev || m <= 0) return set_error(c, QCFG_EINVAL, "calibrate_model: null input or m <= 0");
  if ((uintptr_t)x_dev % 4) return set_error(c, QCFG_EALIGN, "calibrate_model: x_dev not 4-byte aligned");
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t ext_ld = ext_ld_of(M);
  int rc = forward(c, M, nullptr, x_dev, ext_ld, m, nullptr, true, st);
  if (rc) return rc;
  std::vector<float> host(M->L.size());
  rc = check_cuda(c, cudaMemcpyAsync(host.data(), M->act_absmax_dev.p, host.size() * 4, cudaMemcpyDeviceToHost, st), "calibration table copy");
  if (!rc) rc = qcfg_sync_status(ctx, stream);
  if (rc) return rc;
  for (size_t l = 0; l < host.size(); ++l)
    if (M->calib_same_as[l] >= 0) host[l] = host[(size_t)M->calib_same_as[l]];
  for (size_t l = 0; l < host.size(); ++l)
    if (!std::isfinite(host[l])) return set_error(c, QCFG_ENONFINITE, "layer %zu: calibrated input maximum is not finite", l);
  for (size_t l = 0; l < host.size(); ++l) M->L[l].act_absmax = host[l];
  reset_adjusted_scales(M);
  M->calibrated = true;
  M->evaluated = false;
  return QCFG_OK;
}

int qcfg_model_act_absmax(qcfg_model* model, float* absmax_host) {
  if (!model || !absmax_host) return QCFG_EINVAL;
  if (!model->m.calibrated) return QCFG_ESTATE;
  for (size_t l = 0; l < model->m.L.size(); ++l) absmax_host[l] = model->m.L[l].act_absmax;
  return QCFG_OK;
}

int qcfg_model_weight_absmax(qcfg_model* model, int32_t layer, float* absmax_host) {
  if (!model || !absmax_host) return QCFG_EINVAL;
  Model* M = &model->m;
  if (layer < 0 || layer >= (int)M->L.size()) return set_error(M->ctx, QCFG_EINVAL, "weight_absmax: bad layer index");
  LayerState& S = M->L[layer];
  return check_cuda(M->ctx, cudaMemcpy(absmax_host, S.w_absmax.p, (size_t)S.d.n_out * 4, cudaMemcpyDeviceToHost), "weight maxima copy");
}

int qcfg_eval_config(qcfg_ctx* ctx, qcfg_model* model, const uint8_t* bits, const float* x_dev, int64_t m,
                     float* const* y_dev, void* stream) {
  if (!ctx || !model) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  Model* M = &model->m;
  if (!bits || !x_dev || m <= 0) return set_error(c, QCFG_EINVAL, "eval_config: null pointer or m <= 0");
  if (!M->calibrated) return set_error(c, QCFG_ESTATE, "eval_config: model is not calibrated");
  if ((uintptr_t)x_dev % 4) return set_error(c, QCFG_EALIGN, "eval_config: x_dev not 4-byte aligned");
  for (size_t l = 0; l < M->L.size(); ++l) {
    if (!bits_ok(bits[l])) return set_error(c, QCFG_EBITS, "eval_config: layer %zu has bit width %d", l, (int)bits[l]);
    if (y_dev && y_dev[l] && (uintptr_t)y_dev[l] % 4) return set_error(c, QCFG_EALIGN, "eval_config: y_dev[%zu] not 4-byte aligned", l);
  }
  const int64_t ext_ld = ext_ld_of(M);
  int rc = forward(c, M, bits, x_dev, ext_ld, m, y_dev, false, (cudaStream_t)stream);
  if (rc) return rc;
  M->evaluated = true;
  M->last_m = m;
  return QCFG_OK;
}

// ---- latency table and configuration cost (Section 4, "Compute Latency Estimates"; Table 1) ----

int qcfg_latency_table(qcfg_ctx* ctx, qcfg_model* model, const float* x_dev, int64_t m, const uint8_t* bs, int32_t n_bs,
                       int32_t reps, float* ms_host, void* stream) {
  if (!ctx || !model) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  Model* M = &model->m;
  if (!x_dev || !bs || !ms_host || m <= 0 || n_bs <= 0 || reps <= 0) return set_error(c, QCFG_EINVAL, "latency_table: null pointer or non-positive count");
  if (!M->calibrated) return set_error(c, QCFG_ESTATE, "latency_table: model is not calibrated");
  if ((uintptr_t)x_dev % 4) return set_error(c, QCFG_EALIGN, "latency_table: x_dev not 4-byte aligned");
  for (int i = 0; i < n_bs; ++i)
    if (!bits_ok(bs[i])) return set_error(c, QCFG_EBITS, "latency_table: bs[%d] = %d", i, (int)bs[i]);
  const int n = (int)M->L.size();
  cudaStream_t st = (cudaStream_t)stream;
  std::vector<cudaEvent_t> ev((size_t)2 * n, nullptr);
  int rc = QCFG_OK;
  for (auto& e : ev)
    if (rc == QCFG_OK && cudaEventCreate(&e) != cudaSuccess) rc = set_error(c, QCFG_ECUDA, "latency_table: cudaEventCreate failed");
  std::vector<uint8_t> bits((size_t)n);
  std::vector<double> sum((size_t)n);
  const int64_t ext_ld = ext_ld_of(M);
  for (int i = 0; i < n_bs && rc == QCFG_OK; ++i) {
    std::fill(bits.begin(), bits.end(), bs[i]);
    std::fill(sum.begin(), sum.end(), 0.0);
    rc = forward(c, M, bits.data(), x_dev, ext_ld, m, nullptr, false, st);        // fills the weight-code cache
    for (int r = 0; r < reps && rc == QCFG_OK; ++r) {
      rc = forward(c, M, bits.data(), x_dev, ext_ld, m, nullptr, false, st, ev.data());
      if (rc == QCFG_OK) rc = check_cuda(c, cudaEventSynchronize(ev[(size_t)2 * n - 1]), "latency_table: event synchronize");
      for (int l = 0; l < n && rc == QCFG_OK; ++l) {
        float ms = 0.f;
        rc = check_cuda(c, cudaEventElapsedTime(&ms, ev[2 * l], ev[2 * l + 1]), "latency_table: elapsed time");
        sum[l] += ms;
      }
    }
    if (rc == QCFG_OK)
      for (int l = 0; l < n; ++l) ms_host[(size_t)l * n_bs + i] = (float)(sum[l] / reps);
  }
  for (auto& e : ev) if (e) cudaEventDestroy(e);
  if (rc == QCFG_OK) { M->evaluated = true; M->last_m = m; }
  return rc;
}

int qcfg_config_cost(qcfg_model* model, const uint8_t* bits, const uint8_t* bs, int32_t n_bs, const float* ms_host,
                     double* latency_ms, double* size_bytes) {
  if (!model || !bits) return QCFG_EINVAL;
  Model* M = &model->m;
  Ctx* c = M->ctx;
  if (latency_ms && (!bs || !ms_host || n_bs <= 0)) return set_error(c, QCFG_EINVAL, "config_cost: latency wanted without a table");
  const int n = (int)M->L.size();
  double lat = 0.0, size = 0.0;
  for (int l = 0; l < n; ++l) {
    if (!bits_ok(bits[l])) return set_error(c, QCFG_EBITS, "config_cost: layer %d has bit width %d", l, (int)bits[l]);
    size += (double)M->L[l].d.n_out * (double)M->L[l].d.k_in * (double)bits[l] / 8.0;
    if (latency_ms) {
      int col = -1;
      for (int i = 0; i < n_bs; ++i) if (bs[i] == bits[l]) col = i;
      if (col < 0) return set_error(c, QCFG_EBITS, "config_cost: layer %d uses %d bit, which the table does not cover", l, (int)bits[l]);
      lat += (double)ms_host[(size_t)l * n_bs + col];
    }
  }
  if (latency_ms) *latency_ms = lat;
  if (size_bytes) *size_bytes = size;
  return QCFG_OK;
}

// ---- search drivers (Algorithms 1 and 2 over qcfg_eval_config) ---------------------------------

namespace {

struct SearchState {
  qcfg_ctx* ctx; qcfg_model* model;
  const float* x; int64_t m; cudaStream_t st;
  int n; int64_t out_elems; int blocks;
  std::vector<float*> ys;
  std::vector<double> host_partial;
  uint8_t* visited; int32_t cap; double* acc_out; int32_t evals;
  int rc;
};

// accuracy proxy of one configuration: 1 - ||y - ref||_2 / ||ref||_2 on the last layer's output
double search_evaluate(SearchState& S, const std::vector<uint8_t>& cfg) {
  Model* M = &S.model->m;
  Ctx* c = &S.ctx->c;
  if (S.rc) return 0.0;
  S.rc = qcfg_eval_config(S.ctx, S.model, cfg.data(), S.x, S.m, S.ys.data(), S.st);
  if (!S.rc) S.rc = launch_sqdiff(c, (const float*)M->search_out.p, (const float*)M->search_ref.p, S.out_elems,
                                  (double*)M->search_partial.p, S.blocks, S.st);
  if (!S.rc) S.rc = check_cuda(c, cudaMemcpyAsync(S.host_partial.data(), M->search_partial.p, (size_t)S.blocks * 16,
                                                  cudaMemcpyDeviceToHost, S.st), "fidelity copy");
  if (!S.rc) S.rc = qcfg_sync_status(S.ctx, S.st);
  if (S.rc) return 0.0;
  double d2 = 0.0, r2 = 0.0;
  for (int b = 0; b < S.blocks; ++b) { d2 += S.host_partial[2 * b]; r2 += S.host_partial[2 * b + 1]; }
  const double a = r2 > 0.0 ? 1.0 - std::sqrt(d2 / r2) : (d2 == 0.0 ? 1.0 : 0.0);
  if (S.evals < S.cap) {
    if (S.visited) memcpy(S.visited + (size_t)S.evals * S.n, cfg.data(), S.n);
    if (S.acc_out) S.acc_out[S.evals] = a;
  }
  S.evals++;
  return a;
}

}  // namespace

int qcfg_search(qcfg_ctx* ctx, qcfg_model* model, int algorithm, const int32_t* order, const uint8_t* bs, int32_t n_bs,
                double target, const float* x_dev, int64_t m, uint8_t* bits_out, uint8_t* visited, double* accuracies,
                int32_t capacity, int32_t* n_evals, void* stream) {
  if (!ctx || !model) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  Model* M = &model->m;
  const int n = (int)M->L.size();
  if (!order || !bs || n_bs < 1 || !x_dev || m <= 0 || !bits_out || capacity < 0)
    return set_error(c, QCFG_EINVAL, "search: null pointer or bad size");
  if (algorithm != QCFG_SEARCH_BISECTION && algorithm != QCFG_SEARCH_GREEDY) return set_error(c, QCFG_EINVAL, "search: unknown algorithm");
  if (!M->calibrated) return set_error(c, QCFG_ESTATE, "search: model is not calibrated");
  std::vector<char> seen(n, 0);
  for (int i = 0; i < n; ++i) {
    if (order[i] < 0 || order[i] >= n || seen[order[i]]) return set_error(c, QCFG_EINVAL, "search: order is not a permutation of the layers");
    seen[order[i]] = 1;
  }
  int top = 0;
  for (int i = 0; i < n_bs; ++i) { if (!bits_ok(bs[i])) return set_error(c, QCFG_EBITS, "search: bit width %d", (int)bs[i]); if (bs[i] > top) top = bs[i]; }
  std::vector<int> lower;                       // the other bit widths, high to low
  for (int i = 0; i < n_bs; ++i) if (bs[i] != top) lower.push_back(bs[i]);
  std::sort(lower.begin(), lower.end(), [](int a, int b) { return a > b; });
  lower.erase(std::unique(lower.begin(), lower.end()), lower.end());

  SearchState S{};
  S.ctx = ctx; S.model = model; S.x = x_dev; S.m = m; S.st = (cudaStream_t)stream; S.n = n;
  S.visited = visited; S.cap = capacity; S.acc_out = accuracies; S.evals = 0; S.rc = 0;
  S.out_elems = layer_rows(M, n - 1, m) * M->L[n - 1].d.n_out;
  S.blocks = c->sms * 4;
  S.host_partial.resize((size_t)S.blocks * 2);
  int rc = M->search_ref.ensure(c, (size_t)S.out_elems * 4);
  if (!rc) rc = M->search_out.ensure(c, (size_t)S.out_elems * 4);
  if (!rc) rc = M->search_partial.ensure(c, (size_t)S.blocks * 16);
  if (rc) return rc;
  S.ys.assign(n, nullptr);

  // reference output: every layer at max(bs), the configuration both searches start from
  std::vector<uint8_t> w(n, (uint8_t)top);
  S.ys[n - 1] = (float*)M->search_ref.p;
  rc = qcfg_eval_config(ctx, model, w.data(), x_dev, m, S.ys.data(), stream);
  if (rc) return rc;
  S.ys[n - 1] = (float*)M->search_out.p;

  // `config` is the working configuration; `candidates` are the layers still eligible for a lower
  // width, least sensitive first.  Both searches lower widths one value of `lower` at a time.
  std::vector<uint8_t>& config = w;
  std::vector<int> candidates(order, order + n);
  // the working configuration with the first `count` candidates set to `width`
  auto with_prefix = [&](int count, int width) {
    std::vector<uint8_t> trial(config);
    for (int i = 0; i < count; ++i) trial[candidates[i]] = (uint8_t)width;
    return trial;
  };
  if (algorithm == QCFG_SEARCH_BISECTION) {
    // Algorithm 1: binary search for the longest prefix of the candidates that can take `width`.
    // `passing` is the longest prefix known to meet the target, `failing` the shortest known not
    // to (or one past the list); the probe moves halfway (floor) towards whichever bound is open
    // and the search ends when it stops moving.  The prefix written is `passing`.
    for (int width : lower) {
      const int count = (int)candidates.size();
      int passing = 0, failing = count, probe = count / 2;
      bool moved = true;
      while (moved) {
        const double fidelity = search_evaluate(S, with_prefix(probe, width));
        if (S.rc) return S.rc;
        int next;
        if (fidelity >= target) { passing = probe; next = probe + (failing - probe) / 2; }
        else { failing = probe; next = probe - (probe - passing) / 2; }
        moved = next != probe;
        probe = next;
      }
      config = with_prefix(passing, width);
      candidates.resize(passing);
    }
  } else {
    // Algorithm 2: try `width` on one candidate at a time, keeping each change that meets the
    // target; only the layers that took this width stay candidates for the next one.
    for (int width : lower) {
      std::vector<int> kept;
      for (int layer : candidates) {
        const uint8_t before = config[layer];
        config[layer] = (uint8_t)width;
        const double fidelity = search_evaluate(S, config);
        if (S.rc) return S.rc;
        if (fidelity >= target) kept.push_back(layer);
        else config[layer] = before;
      }
      candidates.swap(kept);
    }
  }
  memcpy(bits_out, w.data(), n);
  if (n_evals) *n_evals = S.evals;
  return QCFG_OK;
}

// ---- noise-injection sensitivity E_N (Section 3.1, Eqs. 3-5) ----------------------------------

int qcfg_noise_sensitivity(qcfg_ctx* ctx, qcfg_model* model, const float* x_dev, int64_t m, const float* const* noise_dev,
                           float lambda, double* e_n_host, void* stream) {
  if (!ctx || !model) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  Model* M = &model->m;
  const int n = (int)M->L.size();
  if (!x_dev || !noise_dev || !e_n_host || m <= 0) return set_error(c, QCFG_EINVAL, "noise_sensitivity: null pointer or m <= 0");
  if (!(lambda >= 0.0f) || !std::isfinite(lambda)) return set_error(c, QCFG_EINVAL, "noise_sensitivity: lambda must be finite and >= 0");
  if ((uintptr_t)x_dev % 4) return set_error(c, QCFG_EALIGN, "noise_sensitivity: x_dev not 4-byte aligned");
  for (int l = 0; l < n; ++l)
    if (noise_dev[l] && (uintptr_t)noise_dev[l] % 4) return set_error(c, QCFG_EALIGN, "noise_sensitivity: noise_dev[%d] not 4-byte aligned", l);
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t out_elems = layer_rows(M, n - 1, m) * M->L[n - 1].d.n_out;
  const int blocks = c->sms * 4;
  size_t code_bytes = 0;
  for (auto& S : M->L) code_bytes = std::max(code_bytes, (size_t)(S.d.n_out * S.ldk) * 2);
  int rc = M->search_ref.ensure(c, (size_t)out_elems * 4);
  if (!rc) rc = M->search_out.ensure(c, (size_t)out_elems * 4);
  if (!rc) rc = M->search_partial.ensure(c, (size_t)blocks * 16);
  if (!rc) rc = M->noise_codes.ensure(c, code_bytes);
  if (!rc) rc = M->noise_amax.ensure(c, 4);
  if (rc) return rc;
  std::vector<double> partial((size_t)blocks * 2);
  std::vector<uint8_t> bits((size_t)n, 16);
  std::vector<float*> ys((size_t)n, nullptr);
  const int64_t ext_ld = ext_ld_of(M);
  // the noise-free model: every layer at 16 bit
  ys[n - 1] = (float*)M->search_ref.p;
  rc = forward(c, M, bits.data(), x_dev, ext_ld, m, ys.data(), false, st);
  if (rc) return rc;
  ys[n - 1] = (float*)M->search_out.p;
  for (int i = 0; i < n; ++i) {
    e_n_host[i] = 0.0;
    if (!noise_dev[i]) continue;
    LayerState& S = M->L[i];
    rc = launch_absmax(c, S.d.w_dev, S.d.n_out, S.d.k_in, S.d.k_in, QCFG_PER_TENSOR, (float*)M->noise_amax.p, st);
    if (!rc) rc = launch_perturb_bf16(c, S.d.w_dev, noise_dev[i], (const float*)M->noise_amax.p, lambda, S.d.n_out, S.d.k_in,
                                      M->noise_codes.p, S.ldk, st);
    if (rc) return rc;
    void* clean = S.wc[16].codes.p;               // W* = W without w_i, plus w_i + nu
    S.wc[16].codes.p = M->noise_codes.p;
    M->reuse_valid = false;                       // the weights differ from the last forward's
    rc = forward(c, M, bits.data(), x_dev, ext_ld, m, ys.data(), false, st);
    M->reuse_valid = false;
    S.wc[16].codes.p = clean;
    if (!rc) rc = launch_sqdiff(c, (const float*)M->search_out.p, (const float*)M->search_ref.p, out_elems,
                                (double*)M->search_partial.p, blocks, st);
    if (!rc) rc = check_cuda(c, cudaMemcpyAsync(partial.data(), M->search_partial.p, (size_t)blocks * 16, cudaMemcpyDeviceToHost, st),
                             "noise_sensitivity: copy");
    if (!rc) rc = qcfg_sync_status(ctx, st);
    if (rc) return rc;
    double d2 = 0.0, r2 = 0.0;
    for (int b = 0; b < blocks; ++b) { d2 += partial[2 * b]; r2 += partial[2 * b + 1]; }
    e_n_host[i] = r2 > 0.0 ? std::sqrt(d2 / r2) : (d2 == 0.0 ? 0.0 : INFINITY);
  }
  M->evaluated = true;
  M->last_m = m;
  return QCFG_OK;
}


// ---- scale adjustment (Section 3.1, second step; learning rate of Section 4) -------------------

namespace {

// One pass of the adjustment: the forward of the model under `bits` with its current scales, layer
// by layer with the rescaled accumulators (ylin) and the activated outputs (yact) kept, the loss
// against yref, and (want_grads) the backward pass that leaves the gradients of the weight scales
// in every layer's dsw / diw and those of the activation scales in M->adj_dscal (two doubles per
// layer: d/d(scale), d/d(inv_scale)).  Linear layers only.  Synchronises the stream.
int adjust_pass(qcfg_ctx* h, Model* M, const uint8_t* bits, const float* x_dev, int64_t m, const float* yref, double* loss,
                bool want_grads, cudaStream_t st) {
  Ctx* c = &h->c;
  const int n = (int)M->L.size();
  const int64_t x_ld = ext_ld_of(M);
  M->reuse_valid = false;
  auto input_of = [&](int l, const float** p, int64_t* ld) {
    const qcfg_layer& d = M->L[l].d;
    if (d.src < 0) { *p = x_dev + d.src_col0; *ld = x_ld; }
    else { *p = (const float*)M->L[d.src].yact.p + d.src_col0; *ld = M->L[d.src].d.n_out; }
  };
  int rc = QCFG_OK;
  for (int l = 0; l < n && !rc; ++l) {
    LayerState& S = M->L[l];
    const qcfg_layer& d = S.d;
    if (d.kh > 0 || d.pool_before != QCFG_POOL_NONE)
      return set_error(c, QCFG_ESHAPE, "scale adjustment covers linear layers only (layer %d is a convolution or pooled)", l);
    const int b = bits[l];
    S.rows = m; S.bits = b;
    rc = ensure_weight_codes(c, S, b, st);
    if (!rc) rc = S.abuf.ensure(c, (size_t)(m * S.ldk) * 2);
    if (!rc) rc = S.ylin.ensure(c, (size_t)(m * d.n_out) * 4);
    if (!rc) rc = S.yact.ensure(c, (size_t)(m * d.n_out) * 4);
    if (rc) break;
    const float* xin; int64_t ldx;
    input_of(l, &xin, &ldx);
    float sx = 1.0f, ix = 1.0f;
    if (b != 16) act_scales(S, b, &sx, &ix);
    rc = launch_quantize(c, xin, m, d.k_in, ldx, nullptr, ix, QCFG_PER_TENSOR, b, S.abuf.p, S.ldk, st);
    if (rc) break;
    S.a_ptr = S.abuf.p; S.a_ready = true;
    GemmArgs g{};
    g.a = S.abuf.p; g.lda = S.ldk; g.b = S.wc[b].codes.p; g.ldb = S.ldk;
    g.m = m; g.n = d.n_out; g.k = d.k_in; g.is_bf16 = b == 16; g.act = QCFG_ACT_NONE;
    g.scale_x = sx; g.scale_w = b == 16 ? nullptr : (const float*)S.wc[b].scale.p;
    g.y = (float*)S.ylin.p; g.ldy = d.n_out;
    rc = launch_gemm(c, g, st);
    const float* res = d.residual_from >= 0 ? (const float*)M->L[d.residual_from].yact.p : nullptr;
    if (!rc) rc = launch_act_apply(c, (const float*)S.ylin.p, res, d.residual_from >= 0 ? M->L[d.residual_from].d.n_out : 0, d.act,
                                   (float*)S.yact.p, m, d.n_out, st);
    S.y_ptr = (const float*)S.yact.p; S.y_internal = false;
  }
  if (rc) return rc;
  LayerState& Z = M->L[n - 1];
  const int64_t out_elems = m * Z.d.n_out;
  const int blocks = c->sms * 4;
  rc = M->search_partial.ensure(c, (size_t)blocks * 16);
  std::vector<double> partial((size_t)blocks * 2);
  const float* ref = yref ? yref : (const float*)Z.yact.p;
  if (!rc) rc = launch_sqdiff(c, (const float*)Z.yact.p, ref, out_elems, (double*)M->search_partial.p, blocks, st);
  if (!rc) rc = check_cuda(c, cudaMemcpyAsync(partial.data(), M->search_partial.p, (size_t)blocks * 16, cudaMemcpyDeviceToHost, st), "adjust: loss copy");
  if (!rc) rc = qcfg_sync_status(h, st);
  if (rc) return rc;
  double d2 = 0.0, r2 = 0.0;
  for (int i = 0; i < blocks; ++i) { d2 += partial[2 * i]; r2 += partial[2 * i + 1]; }
  if (loss) *loss = r2 > 0.0 ? d2 / r2 : 0.0;
  if (!want_grads) return QCFG_OK;
  if (!(r2 > 0.0)) return set_error(c, QCFG_ESTATE, "scale adjustment: the reference output is all zero");

  // ---- backward
  int64_t max_n = 0, max_k = 0;
  for (auto& S : M->L) { max_n = std::max<int64_t>(max_n, S.d.n_out); max_k = std::max<int64_t>(max_k, S.d.k_in); }
  const int64_t ldm = round_up(m, 8);
  rc = M->adj_dscal.ensure(c, (size_t)n * 16);
  if (!rc) rc = M->adj_colsum.ensure(c, (size_t)max_n * 8);
  if (!rc) rc = M->adj_gs.ensure(c, (size_t)(m * round_up(max_n, 8)) * 2);
  if (!rc) rc = M->adj_gt.ensure(c, (size_t)(max_n * ldm) * 2);
  if (!rc) rc = M->adj_qxt.ensure(c, (size_t)(max_k * ldm) * 2);
  if (!rc) rc = M->adj_qwt.ensure(c, (size_t)(max_k * round_up(max_n, 8)) * 2);
  if (!rc) rc = M->adj_dx.ensure(c, (size_t)(m * max_k) * 4);
  if (!rc) rc = M->adj_dw.ensure(c, (size_t)(max_n * max_k) * 4);
  if (!rc) rc = check_cuda(c, cudaMemsetAsync(M->adj_dscal.p, 0, (size_t)n * 16, st), "adjust: memset");
  for (int l = 0; l < n && !rc; ++l) {
    LayerState& S = M->L[l];
    rc = S.gout.ensure(c, (size_t)(m * S.d.n_out) * 4);
    if (!rc) rc = S.dsw.ensure(c, (size_t)S.d.n_out * 8);
    if (!rc) rc = S.diw.ensure(c, (size_t)S.d.n_out * 8);
    if (!rc) rc = check_cuda(c, cudaMemsetAsync(S.gout.p, 0, (size_t)(m * S.d.n_out) * 4, st), "adjust: memset");
    if (!rc) rc = check_cuda(c, cudaMemsetAsync(S.dsw.p, 0, (size_t)S.d.n_out * 8, st), "adjust: memset");
    if (!rc) rc = check_cuda(c, cudaMemsetAsync(S.diw.p, 0, (size_t)S.d.n_out * 8, st), "adjust: memset");
  }
  if (!rc) rc = launch_loss_grad(c, (const float*)Z.yact.p, ref, (float)(2.0 / r2), (float*)Z.gout.p, out_elems, st);
  double* dscal = (double*)M->adj_dscal.p;
  for (int l = n - 1; l >= 0 && !rc; --l) {
    LayerState& S = M->L[l];
    const qcfg_layer& d = S.d;
    const int b = bits[l];
    const int64_t nn = d.n_out, kk = d.k_in, ldn = round_up(nn, 8);
    float* gpre = (float*)S.gout.p;
    const float* res = d.residual_from >= 0 ? (const float*)M->L[d.residual_from].yact.p : nullptr;
    const int64_t ldr = d.residual_from >= 0 ? M->L[d.residual_from].d.n_out : 0;
    rc = launch_act_backward(c, gpre, (const float*)S.ylin.p, res, ldr, d.act, m, nn, st);
    if (!rc && d.residual_from >= 0)          // the shortcut passes the gradient on unchanged
      rc = launch_input_backward(c, gpre, nullptr, 0, 1.0f, 1.0f, 0.0f, m, nn, (float*)M->L[d.residual_from].gout.p, ldr, nullptr, st);
    float sx = 1.0f, ix = 1.0f;
    if (b != 16) act_scales(S, b, &sx, &ix);
    const float qm = b == 16 ? 0.0f : qmax_of(b);
    if (!rc && b != 16) {       // post-rounding scales: d/ds_w[n] = sum_m g*ylin / s_w[n], d/ds_x = sum g*ylin / s_x
      rc = check_cuda(c, cudaMemsetAsync(M->adj_colsum.p, 0, (size_t)nn * 8, st), "adjust: memset");
      if (!rc) rc = launch_col_dot(c, gpre, (const float*)S.ylin.p, m, nn, (double*)M->adj_colsum.p, st);
      if (!rc) rc = launch_gamma_finish(c, (const double*)M->adj_colsum.p, (const float*)S.wc[b].scale.p, sx, nn, (double*)S.dsw.p, dscal + 2 * l, st);
    }
    // gradient of the input codes: dxq[m][k] = sum_n (g[m][n] s_w[n]) qw[n][k]   (bf16 tensor-core GEMM)
    if (!rc) rc = launch_scale_cols_bf16(c, gpre, b == 16 ? nullptr : (const float*)S.wc[b].scale.p, m, nn, M->adj_gs.p, ldn, st);
    if (!rc) rc = launch_transpose_bf16(c, S.wc[b].codes.p, b == 16 ? 2 : 1, nn, kk, S.ldk, M->adj_qwt.p, ldn, st);
    if (!rc) {
      GemmArgs g{};
      g.a = M->adj_gs.p; g.lda = ldn; g.b = M->adj_qwt.p; g.ldb = ldn;
      g.m = m; g.n = kk; g.k = nn; g.is_bf16 = 1; g.act = QCFG_ACT_NONE; g.y = (float*)M->adj_dx.p; g.ldy = kk;
      rc = launch_gemm(c, g, st);
    }
    const float* xin; int64_t ldx;
    input_of(l, &xin, &ldx);
    float* gprod = d.src >= 0 ? (float*)M->L[d.src].gout.p + d.src_col0 : nullptr;
    if (!rc) rc = launch_input_backward(c, (const float*)M->adj_dx.p, xin, ldx, sx, ix, qm, m, kk, gprod,
                                        d.src >= 0 ? M->L[d.src].d.n_out : 0, b == 16 ? nullptr : dscal + 2 * l + 1, st);
    if (!rc && b != 16) {       // gradient of the weight codes: dwq[n][k] = sum_m g[m][n] qx[m][k], then the pre-rounding scales
      rc = launch_transpose_bf16(c, gpre, 0, m, nn, nn, M->adj_gt.p, ldm, st);
      if (!rc) rc = launch_transpose_bf16(c, S.abuf.p, 1, m, kk, S.ldk, M->adj_qxt.p, ldm, st);
      if (!rc) {
        GemmArgs g{};
        g.a = M->adj_gt.p; g.lda = ldm; g.b = M->adj_qxt.p; g.ldb = ldm;
        g.m = nn; g.n = kk; g.k = m; g.is_bf16 = 1; g.act = QCFG_ACT_NONE; g.y = (float*)M->adj_dw.p; g.ldy = kk;
        rc = launch_gemm(c, g, st);
      }
      if (!rc) rc = launch_weight_alpha(c, (const float*)M->adj_dw.p, d.w_dev, (const float*)S.wc[b].scale.p, (const float*)S.wc[b].inv.p,
                                        sx, qm, nn, kk, (double*)S.diw.p, st);
    }
  }
  if (!rc) rc = qcfg_sync_status(h, st);
  return rc;
}

int adjust_check(Ctx* c, Model* M, const uint8_t* bits, const float* x_dev, int64_t m, const char* who) {
  if (!bits || !x_dev || m <= 0) return set_error(c, QCFG_EINVAL, "%s: null pointer or m <= 0", who);
  if (!M->calibrated) return set_error(c, QCFG_ESTATE, "%s: model is not calibrated", who);
  if ((uintptr_t)x_dev % 4) return set_error(c, QCFG_EALIGN, "%s: x_dev not 4-byte aligned", who);
  for (size_t l = 0; l < M->L.size(); ++l)
    if (!bits_ok(bits[l])) return set_error(c, QCFG_EBITS, "%s: layer %zu has bit width %d", who, l, (int)bits[l]);
  return QCFG_OK;
}

// reference output: the 16-bit model's last layer, kept in M->search_ref
int adjust_reference(qcfg_ctx* h, Model* M, const float* x_dev, int64_t m, cudaStream_t st) {
  Ctx* c = &h->c;
  const int n = (int)M->L.size();
  std::vector<uint8_t> b16((size_t)n, 16);
  int rc = adjust_pass(h, M, b16.data(), x_dev, m, nullptr, nullptr, false, st);
  const size_t bytes = (size_t)(m * M->L[n - 1].d.n_out) * 4;
  if (!rc) rc = M->search_ref.ensure(c, bytes);
  if (!rc) rc = check_cuda(c, cudaMemcpyAsync(M->search_ref.p, M->L[n - 1].yact.p, bytes, cudaMemcpyDeviceToDevice, st), "adjust: reference copy");
  return rc;
}

}  // namespace

int qcfg_scale_gradients(qcfg_ctx* ctx, qcfg_model* model, const uint8_t* bits, const float* x_dev, int64_t m,
                         double* d_scale_x, double* d_inv_scale_x, double* const* d_scale_w, double* const* d_inv_scale_w,
                         double* loss, void* stream) {
  if (!ctx || !model) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  Model* M = &model->m;
  int rc = adjust_check(c, M, bits, x_dev, m, "scale_gradients");
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const int n = (int)M->L.size();
  rc = adjust_reference(ctx, M, x_dev, m, st);
  if (!rc) rc = adjust_pass(ctx, M, bits, x_dev, m, (const float*)M->search_ref.p, loss, true, st);
  if (rc) return rc;
  std::vector<double> ds((size_t)2 * n);
  rc = check_cuda(c, cudaMemcpy(ds.data(), M->adj_dscal.p, ds.size() * 8, cudaMemcpyDeviceToHost), "scale_gradients: copy");
  for (int l = 0; l < n && !rc; ++l) {
    if (d_scale_x) d_scale_x[l] = bits[l] == 16 ? 0.0 : ds[2 * l];
    if (d_inv_scale_x) d_inv_scale_x[l] = bits[l] == 16 ? 0.0 : ds[2 * l + 1];
    const size_t bytes = (size_t)M->L[l].d.n_out * 8;
    if (d_scale_w && d_scale_w[l]) rc = check_cuda(c, cudaMemcpy(d_scale_w[l], M->L[l].dsw.p, bytes, cudaMemcpyDeviceToHost), "scale_gradients: copy");
    if (!rc && d_inv_scale_w && d_inv_scale_w[l]) rc = check_cuda(c, cudaMemcpy(d_inv_scale_w[l], M->L[l].diw.p, bytes, cudaMemcpyDeviceToHost), "scale_gradients: copy");
  }
  M->evaluated = true; M->last_m = m;
  return rc;
}

int qcfg_adjust_scales(qcfg_ctx* ctx, qcfg_model* model, const uint8_t* bits, const float* x_dev, int64_t m, int32_t steps,
                       double lr, double* losses_host, void* stream) {
  if (!ctx || !model) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  Model* M = &model->m;
  int rc = adjust_check(c, M, bits, x_dev, m, "adjust_scales");
  if (rc) return rc;
  if (steps < 0 || !(lr >= 0.0) || !std::isfinite(lr)) return set_error(c, QCFG_EINVAL, "adjust_scales: steps and lr must be >= 0");
  cudaStream_t st = (cudaStream_t)stream;
  const int n = (int)M->L.size();
  rc = adjust_reference(ctx, M, x_dev, m, st);
  if (rc) return rc;
  // from here on the scales of (layer, bits[layer]) live on their own: start from their current values
  for (int l = 0; l < n && !rc; ++l) {
    const int b = bits[l];
    if (b == 16) continue;
    LayerState& S = M->L[l];
    rc = ensure_weight_codes(c, S, b, st);
    S.wc[b].adjusted = true;
    if (!S.adj_act[b]) { host_scales(S.act_absmax, b, &S.adj_sx[b], &S.adj_ix[b]); S.adj_act[b] = true; }
  }
  std::vector<double> ds((size_t)2 * n);
  for (int step = 0; step < steps && !rc; ++step) {
    double loss = 0.0;
    rc = adjust_pass(ctx, M, bits, x_dev, m, (const float*)M->search_ref.p, &loss, true, st);
    if (rc) break;
    if (losses_host) losses_host[step] = loss;
    rc = check_cuda(c, cudaMemcpy(ds.data(), M->adj_dscal.p, ds.size() * 8, cudaMemcpyDeviceToHost), "adjust_scales: copy");
    for (int l = 0; l < n && !rc; ++l) {
      const int b = bits[l];
      if (b == 16) continue;
      LayerState& S = M->L[l];
      S.adj_sx[b] = (float)((double)S.adj_sx[b] - lr * ds[2 * l]);
      S.adj_ix[b] = (float)((double)S.adj_ix[b] - lr * ds[2 * l + 1]);
      rc = launch_sgd(c, (float*)S.wc[b].scale.p, (const double*)S.dsw.p, lr, S.d.n_out, st);
      if (!rc) rc = launch_sgd(c, (float*)S.wc[b].inv.p, (const double*)S.diw.p, lr, S.d.n_out, st);
      S.wc[b].ready = false;                    // the weight codes follow the new pre-rounding scales
    }
  }
  double loss = 0.0;
  if (!rc) rc = adjust_pass(ctx, M, bits, x_dev, m, (const float*)M->search_ref.p, &loss, false, st);
  if (!rc && losses_host) losses_host[steps] = loss;
  M->evaluated = true; M->last_m = m;
  M->reuse_valid = false;
  return rc;
}

int qcfg_model_scales(qcfg_model* model, int32_t layer, int bits, float* scale_x, float* inv_scale_x, float* scale_w_host,
                      float* inv_scale_w_host) {
  if (!model) return QCFG_EINVAL;
  Model* M = &model->m;
  Ctx* c = M->ctx;
  if (layer < 0 || layer >= (int)M->L.size()) return set_error(c, QCFG_EINVAL, "model_scales: bad layer index");
  if (!bits_int(bits)) return set_error(c, QCFG_EBITS, "model_scales: bits must be 2..8, got %d", bits);
  if (!M->calibrated) return set_error(c, QCFG_ESTATE, "model_scales: model is not calibrated");
  LayerState& S = M->L[layer];
  float sx, ix;
  act_scales(S, bits, &sx, &ix);
  if (scale_x) *scale_x = sx;
  if (inv_scale_x) *inv_scale_x = ix;
  if (scale_w_host || inv_scale_w_host) {
    int rc = ensure_weight_codes(c, S, bits, 0);
    if (!rc) rc = check_cuda(c, cudaStreamSynchronize(0), "model_scales: sync");
    const size_t bytes = (size_t)S.d.n_out * 4;
    if (!rc && scale_w_host) rc = check_cuda(c, cudaMemcpy(scale_w_host, S.wc[bits].scale.p, bytes, cudaMemcpyDeviceToHost), "model_scales: copy");
    if (!rc && inv_scale_w_host) rc = check_cuda(c, cudaMemcpy(inv_scale_w_host, S.wc[bits].inv.p, bytes, cudaMemcpyDeviceToHost), "model_scales: copy");
    return rc;
  }
  return QCFG_OK;
}

int qcfg_model_reset_scales(qcfg_model* model) {
  if (!model) return QCFG_EINVAL;
  cudaDeviceSynchronize();
  reset_adjusted_scales(&model->m);
  return QCFG_OK;
}

int qcfg_debug_dump(qcfg_ctx* ctx, qcfg_model* model, int32_t layer, int8_t* qx_dev, int8_t* qw_dev, int32_t* acc_dev,
                    void* stream) {
  if (!ctx || !model) return QCFG_EINVAL;
  Ctx* c = &ctx->c;
  Model* M = &model->m;
  if (!M->evaluated) return set_error(c, QCFG_ESTATE, "debug_dump: no evaluation has run");
  if (layer < 0 || layer >= (int)M->L.size()) return set_error(c, QCFG_EINVAL, "debug_dump: bad layer index");
  LayerState& S = M->L[layer];
  if (!bits_int(S.bits)) return set_error(c, QCFG_EBITS, "debug_dump: layer %d ran at %d bit", layer, S.bits);
  cudaStream_t st = (cudaStream_t)stream;
  if (qx_dev && S.implicit) {     // the patches were never materialised: gather them from the input's codes now
    const qcfg_layer& d = S.d;
    const int64_t opix = (int64_t)((d.in_h + 2 * d.pad - d.kh) / d.stride + 1) * ((d.in_w + 2 * d.pad - d.kw) / d.stride + 1);
    int rc = launch_im2col_codes(c, (const int8_t*)S.a_ptr, S.rows / opix, d.in_h, d.in_w, d.in_c, d.kh, d.kw, d.stride, d.pad, qx_dev, d.k_in, st);
    if (rc) return rc;
  } else if (qx_dev) {
    cudaError_t e = cudaMemcpy2DAsync(qx_dev, (size_t)S.d.k_in, S.a_ptr, (size_t)S.ldk, (size_t)S.d.k_in, (size_t)S.rows, cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) return check_cuda(c, e, "debug_dump qx copy");
  }
  if (qw_dev) {
    cudaError_t e = cudaMemcpy2DAsync(qw_dev, (size_t)S.d.k_in, S.wc[S.bits].codes.p, (size_t)S.ldk, (size_t)S.d.k_in, (size_t)S.d.n_out, cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) return check_cuda(c, e, "debug_dump qw copy");
  }
  if (acc_dev) {
    GemmArgs g{};
    g.a = S.a_ptr; g.lda = S.ldk; g.b = S.wc[S.bits].codes.p; g.ldb = S.ldk;
    g.m = S.rows; g.n = S.d.n_out; g.k = S.d.k_in; g.acc = acc_dev;
    if (S.implicit) {
      const qcfg_layer& d = S.d;
      g.lda = d.in_c;
      g.conv_kh = d.kh; g.conv_kw = d.kw; g.conv_stride = d.stride; g.conv_pad = d.pad;
      g.conv_h = d.in_h; g.conv_w = d.in_w; g.conv_c = d.in_c;
    }
    g.scale_x = 1.0f; g.scale_w = (const float*)S.wc[S.bits].scale.p;
    return launch_gemm(c, g, st);
  }
  return QCFG_OK;
}

}  // extern "C"
