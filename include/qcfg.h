/*
 * qcfg -- evaluation of candidate bit configurations and the quantization-error
 * sensitivity sweep for sensitivity-guided mixed-precision post-training quantization
 * (Schaefer et al., "Mixed Precision Post Training Quantization of Neural Networks with
 * Sensitivity Guided Search"), for one NVIDIA B200 (sm_100a).
 *
 * Conventions shared by every entry point
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; the library never
 *     frees or reallocates them.  Pointers without that suffix are HOST pointers.
 *   - `stream` is a cudaStream_t passed as void*.  Work is enqueued asynchronously on it
 *     unless stated otherwise.
 *   - Every call returns a status code (QCFG_OK = 0), never throws, aborts or prints.
 *     On a non-OK return no output has been written.  Errors detected on the device
 *     (a bounded wait that gave up, a non-finite calibration maximum) surface from
 *     qcfg_sync_status().
 *   - Matrices are row-major.  A weight is [n_out x k_in] fp32, row = output channel; for
 *     a convolution k_in = kh*kw*in_c in (kh, kw, cin) order (OHWI).  An activation is
 *     [m x k] fp32 (for convolutions: NHWC, i.e. [batch*h*w x c]).
 *   - Bit widths: 2..8 are symmetric signed integer grids with qmax = 2^(b-1)-1 (codes held
 *     in int8); 16 is bfloat16 operands with fp32 accumulation.
 *   - There is no CPU fallback: without an sm_100 device qcfg_create() fails.
 */
#ifndef QCFG_H_
#define QCFG_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qcfg_ctx qcfg_ctx;     /* device, workspace, tensor-map encoder, error word */
typedef struct qcfg_model qcfg_model; /* layer table, weight-code cache, calibration tables  */

enum {
  QCFG_OK = 0,
  QCFG_EINVAL = 1,     /* null pointer, bad enum, negative size                     */
  QCFG_EBITS = 2,      /* bit width outside {2..8, 16} (or outside 2..8 where stated) */
  QCFG_ESHAPE = 3,     /* inconsistent shapes / layer graph                         */
  QCFG_EALIGN = 4,     /* pointer or leading dimension alignment                    */
  QCFG_ENOMEM = 5,     /* device allocation failed                                  */
  QCFG_ENONFINITE = 6, /* a calibration maximum is NaN or Inf                       */
  QCFG_EARCH = 7,      /* device is not sm_100                                      */
  QCFG_ECUDA = 8,      /* a CUDA runtime/driver call failed; see qcfg_last_error    */
  QCFG_ETIMEOUT = 9,   /* a bounded device-side wait gave up                        */
  QCFG_ESTATE = 11     /* call order (e.g. evaluation before calibration)           */
};
enum { QCFG_PER_TENSOR = 0, QCFG_PER_ROW = 1 };
enum { QCFG_ACT_NONE = 0, QCFG_ACT_RELU = 1, QCFG_ACT_GELU_TANH = 2 };
enum { QCFG_POOL_NONE = 0, QCFG_POOL_MAX3S2 = 1, QCFG_POOL_GLOBAL_AVG = 2 };

/* One "tensor" of the bit configuration: a linear or convolution layer whose weight and
 * input activation share one bit width (Algorithms 1 and 2 index the configuration by
 * layer; Table 1's uniform rows likewise use one width for a layer's weight and input).  */
typedef struct qcfg_layer {
  const float* w_dev;    /* [n_out][k_in] fp32, borrowed for the model's lifetime          */
  int64_t n_out, k_in;
  int32_t src;           /* -1 = external input, else index of the producing layer (< own) */
  int32_t src_col0;      /* first column of the producer's output that is read             */
  int32_t act;           /* QCFG_ACT_*, applied to this layer's output after the residual  */
  int32_t kh, kw, stride, pad;  /* convolution geometry; all 0 for a linear layer          */
  int32_t in_h, in_w, in_c;     /* input size after pool_before (conv only)                */
  int32_t pool_before;          /* QCFG_POOL_*, applied in fp32 to the source              */
  int32_t src_h, src_w;         /* spatial size of the source before pool_before           */
  int32_t residual_from;        /* -1, or a layer whose fp32 output is added before act    */
} qcfg_layer;

/* ---- context ------------------------------------------------------------------------ */

/* Creates a context on CUDA device `device`.  QCFG_EARCH if it is not compute capability
 * 10.x, QCFG_ECUDA if the runtime fails.  The context allocates a small device error word
 * and grows scratch buffers on demand (cudaMalloc on first use of a larger size).        */
int qcfg_create(qcfg_ctx** out, int device);
int qcfg_destroy(qcfg_ctx* ctx);

/* Synchronises `stream`, then returns and clears the device error word:
 * QCFG_OK, QCFG_ETIMEOUT, QCFG_ENONFINITE or QCFG_ECUDA.                                  */
int qcfg_sync_status(qcfg_ctx* ctx, void* stream);
/* Self-test of the failure path of the kernels' bounded waits (every device-side wait, on a
 * barrier or on a counter in shared or global memory, gives up after a time limit instead of
 * hanging): enqueues a one-warp kernel that runs each kind of wait once on something nothing
 * ever signals, with a limit of limit_ns nanoseconds (1 .. 1e8) each.  Every wait has to run
 * out; then the kernel sets the time-out bit of the context's error word and ends normally;
 * the next qcfg_sync_status returns QCFG_ETIMEOUT and clears it.  Nothing else is touched.   */
int qcfg_selftest_wait_timeout(qcfg_ctx* ctx, uint64_t limit_ns, void* stream);
/* Library-owned, NUL-terminated description of the last non-OK status of this context.   */
const char* qcfg_last_error(qcfg_ctx* ctx);
/* Number of kernels this context has launched since creation (for accounting).            */
int64_t qcfg_launch_count(qcfg_ctx* ctx);

/* Switches the fusion of the consumer's quantize step into the producing GEMM's epilogue
 * (default on).  Off: every layer's fp32 output is written and re-read by a separate quantize
 * kernel; results are bit-identical either way for finite values (a NaN, which calibration
 * rejects, is clamped to a code of either sign depending on the path).                     */
int qcfg_set_fusion(qcfg_ctx* ctx, int enabled);
/* Switches the two-CTA GEMM tiles (256 rows per CTA pair, cta_group::2; default on, used for
 * outputs wider than 128 columns and more than 128 rows).  Off: every tile is 128 rows on one
 * CTA.  Results are bit-identical either way.                                               */
int qcfg_set_pair_tiles(qcfg_ctx* ctx, int enabled);
/* Switches grouped launches in model evaluations (default on): up to three layers that do not
 * depend on one another and share rows, reduction length, operand type and tile width run as
 * one kernel.  Results are bit-identical either way.                                        */
int qcfg_set_grouping(qcfg_ctx* ctx, int enabled);

/* Switches implicit-GEMM convolutions in model evaluations (default on): a convolution that is not a
 * plain row read (3x3, strided 1x1, ...) and whose input has channels in whole 16-byte chunks takes
 * the NHWC codes of its input (written by the producer's epilogue where fusion allows) and the GEMM
 * kernel gathers the patches itself, so no im2col matrix is written or read.  Off: every such
 * layer's patch matrix is materialised first.  Results are bit-identical either way.        */
int qcfg_set_implicit_conv(qcfg_ctx* ctx, int enabled);

/* Switches chained GEMM launches in model evaluations (default on): consecutive GEMMs of a
 * forward pass that use the two-CTA 256-column tiles, share rows and operand type and need no
 * other kernel in between (their operands come out of the producers' epilogues) run as ONE
 * cooperative launch of up to sixteen GEMMs.  Its CTA pairs work through the tiles of all layers
 * in one sequence; a tile starts once the row tiles it reads have been completed (per-row-tile
 * counters in device memory, every wait bounded).  Off: one launch per GEMM (or per group of
 * independent GEMMs).  Results are bit-identical either way.                                  */
int qcfg_set_gemm_chains(qcfg_ctx* ctx, int enabled);

/* Switches prefix reuse in model evaluations (default off).  On: qcfg_eval_config keeps every
 * layer's buffers from the previous evaluation and, when it is called again with the same x_dev,
 * the same m and no switch changed in between, recomputes only the layers whose bit width changed,
 * the layers whose output the caller asks for, and everything that reads a recomputed layer; the
 * other layers launch nothing.  This is what consecutive configurations of the searches allow:
 * Algorithm 2 changes one layer per evaluation, Algorithm 1 a slice of the ordering.  The CALLER
 * guarantees that the contents of x_dev did not change between such calls.  Results are
 * bit-identical to a full evaluation.  qcfg_calibrate_model, qcfg_latency_table and
 * qcfg_noise_sensitivity always run every layer.                                              */
int qcfg_set_prefix_reuse(qcfg_ctx* ctx, int enabled);

/* Per-launch timing, off by default.  Mode 1: CUDA events recorded around every launch on the
 * launching stream (a few microseconds of host time per launch; the event records keep
 * consecutive launches from overlapping, so a run in this mode is slower than an untimed one).
 * kernel_class 0 is the int8 GEMM, 1 the bf16 GEMM, 2 every other kernel of the library (except
 * the sweep's finalize step).  Mode 2: the GEMM kernels time themselves -- every CTA folds its
 * %globaltimer reading after the wait for the previous kernel and at its end into the launch's
 * slot of a ring in device memory (two atomics per CTA), so the duration of a launch is the span
 * from its first CTA's start to its last CTA's end, measured inside an otherwise untouched run;
 * classes 0 and 1 only, at most 65536 launches between two reads (later ones are not timed).
 * qcfg_profile_read waits for the recorded launches (mode 2: for the device), then returns the
 * summed kernel time (ms), the number of launches and the summed algorithmic operations
 * (2*m*n*k per launch) since the last reset.  Outputs may be NULL.                          */
int qcfg_profile_enable(qcfg_ctx* ctx, int mode);
int qcfg_profile_read(qcfg_ctx* ctx, int kernel_class, double* ms, int64_t* launches, double* ops,
                      int reset);

/* ---- tensor-level steps --------------------------------------------------------------- */

/* Max calibration (Section 3.1: the maximum value of each tensor; absolute value as in
 * Eq. 2).  x_dev is [rows x cols] fp32 with leading dimension ld (elements).
 * QCFG_PER_TENSOR writes 1 float, QCFG_PER_ROW writes `rows` floats to absmax_dev.  A NaN
 * or Inf input yields a non-finite maximum.                                               */
int qcfg_calibrate(qcfg_ctx* ctx, const float* x_dev, int64_t rows, int64_t cols, int64_t ld,
                   int granularity, float* absmax_dev, void* stream);

/* The two scales of Eq. 1 for a b-bit grid, b in 2..8: scale = A/qmax (applied after the
 * rounding, the paper's 2^-(b-1)*gamma) and inv_scale = qmax/A (applied before it, the
 * paper's alpha*2^(b-1)); one IEEE fp32 division each; A == 0 gives 1 and 1.  Either output
 * may be NULL.                                                                             */
int qcfg_scales_from_absmax(qcfg_ctx* ctx, const float* absmax_dev, int64_t n, int bits,
                            float* scale_dev, float* inv_scale_dev, void* stream);

/* Codes of Eq. 1: q = clamp(round_half_even(x * inv_scale), -qmax, +qmax) as int8 for bits
 * in 2..8; for bits == 16 the output is bfloat16 (round to nearest even) and inv_scale_dev
 * is ignored.  inv_scale_dev holds 1 float (QCFG_PER_TENSOR) or `rows` floats (QCFG_PER_ROW).
 * q_dev is [rows x ldq] elements (int8 or 2-byte bfloat16), 16-byte aligned, ldq a multiple
 * of 16 and >= cols; columns cols..ldq-1 are zeroed.                                       */
int qcfg_quantize(qcfg_ctx* ctx, const float* x_dev, int64_t rows, int64_t cols, int64_t ld,
                  const float* inv_scale_dev, int granularity, int bits, void* q_dev,
                  int64_t ldq, void* stream);

/* Quantization-error sensitivity (Eq. 2) of n_tensors weight tensors for every bit width
 * b_lo..b_hi (within 2..8) in ONE pass over the data.  w_dev, rows, cols are HOST arrays of
 * length n_tensors (w_dev[t] a device pointer to a dense [rows[t] x cols[t]] fp32 matrix).
 * Scales are max-calibrated per row (QCFG_PER_ROW) or per tensor.  Outputs, device memory:
 * sse_dev[t*(b_hi-b_lo+1) + (b-b_lo)] = sum over the tensor of (x - Q_b(x))^2 (double) and
 * absmax_dev[t] = max|x| over the tensor, so that
 * E_QE(t, b) = sqrt(sse / (rows*cols)) / absmax.  Per-tensor granularity takes a second
 * read of the tensor (the maximum must be known first).                                   */
int qcfg_quant_error_sweep(qcfg_ctx* ctx, const float* const* w_dev, const int64_t* rows,
                           const int64_t* cols, int32_t n_tensors, int granularity, int b_lo,
                           int b_hi, double* sse_dev, float* absmax_dev, void* stream);

/* The same sweep for callers that cannot allocate device memory when they call: code that
 * runs after a serving engine or training framework has reserved all of the GPU's memory for
 * its own pool (so cudaMalloc would fail), or inside a latency-critical loop where the implicit
 * device-wide synchronisation of cudaMalloc/cudaFree is not acceptable.  (The paper has no
 * counterpart; this is a deployment variant of qcfg_quant_error_sweep.)  Arguments, outputs and
 * results are those of qcfg_quant_error_sweep.  Differences:
 *   - Its scratch memory (partial sums and work tables) is a fixed array inside the library
 *     image, about 0.6 MiB on every GPU that loads the library, held until the process exits.
 *     The call itself performs no cudaMalloc, cudaFree or other device allocation.
 *   - Limits per call: at most 1024 tensors and at most 2^35 elements in total.  Anything larger
 *     returns QCFG_ENOMEM with a message and does nothing; split the tensors over several calls,
 *     one after the other.
 *   - The work tables are copied to the device from host memory the context reuses on the next
 *     call, so the call must not be recorded into a CUDA graph by stream capture.
 *   - ctx's device must be the current device (QCFG_ESTATE otherwise).  The first call on a
 *     device looks up the array's device address (cudaGetSymbolAddress) and keeps it; make
 *     that first call during start-up, before any stream capture begins.
 *   - All calls, from every context and stream of the process, share that one array per GPU.
 *     A call overwrites what the previous call left (nothing needs clearing: every value read is
 *     written first by the same call), so two calls must not overlap on the GPU: issue them on
 *     one stream, or order them with events.  Overlapping calls race and give wrong sums.     */
int qcfg_quant_error_sweep_static(qcfg_ctx* ctx, const float* const* w_dev, const int64_t* rows,
                                  const int64_t* cols, int32_t n_tensors, int granularity,
                                  int b_lo, int b_hi, double* sse_dev, float* absmax_dev,
                                  void* stream);

/* One quantized GEMM with its fused epilogue, the kernel a configuration evaluation is made
 * of: acc[m][n] = sum_k qx[m][k]*qw[n][k] (int8 x int8 -> int32, exact), then
 * y = float(acc) * (scale_x * scale_w[n]) (the rescale of Eq. 1 for both operands), then
 * the activation.  qx_dev is [m x ldx] int8, qw_dev [n x ldw] int8; ldx, ldw multiples of
 * 16, pointers 16-byte aligned; columns k..ld-1 must be zero.  Either output may be NULL:
 * y_dev [m x n] fp32, acc_dev [m x n] int32 (raw accumulators, for parity checks).         */
int qcfg_gemm_i8(qcfg_ctx* ctx, const int8_t* qx_dev, int64_t ldx, const int8_t* qw_dev,
                 int64_t ldw, int64_t m, int64_t n, int64_t k, float scale_x,
                 const float* scale_w_dev, int act, float* y_dev, int32_t* acc_dev,
                 void* stream);

/* The same GEMM with the consumer's quantize step (Eq. 1 at the consumer's bit width) fused
 * into the epilogue, as a configuration evaluation runs it between two quantized layers:
 * q_out = clamp(round_half_even(act(y) * next_inv_scale), +-qmax(next_bits)) as int8 for
 * next_bits in 2..8, or bfloat16(act(y)) for next_bits == 16 (next_inv_scale ignored).  The fp32
 * y is never written.  q_out_dev is [m x ldq] (int8 or 2-byte bfloat16), 16-byte aligned, ldq a
 * multiple of 16 and >= n; columns n..ldq-1 are left untouched.                              */
int qcfg_gemm_i8_requant(qcfg_ctx* ctx, const int8_t* qx_dev, int64_t ldx, const int8_t* qw_dev,
                         int64_t ldw, int64_t m, int64_t n, int64_t k, float scale_x,
                         const float* scale_w_dev, int act, float next_inv_scale, int next_bits,
                         void* q_out_dev, int64_t ldq, void* stream);

/* 16-bit layer (the paper's floating-point-16 baseline precision, Table 1):
 * y = act(sum_k x[m][k]*w[n][k]) with bfloat16 operands (2-byte elements, leading
 * dimensions multiples of 8 elements, padding zero) and fp32 accumulation.                */
int qcfg_gemm_bf16(qcfg_ctx* ctx, const void* x_bf16_dev, int64_t ldx, const void* w_bf16_dev,
                   int64_t ldw, int64_t m, int64_t n, int64_t k, int act, float* y_dev,
                   void* stream);

/* ---- model-level steps ---------------------------------------------------------------- */

/* Builds a model from a HOST array of layers (copied).  Checks the graph: src and
 * residual_from must point to earlier layers, k_in must fit the producer's slice.
 * Weight maxima per output channel are computed here (one pass over every weight).        */
int qcfg_model_create(qcfg_ctx* ctx, const qcfg_layer* layers, int32_t n_layers,
                      qcfg_model** out);
int qcfg_model_destroy(qcfg_model* model);

/* Max calibration of every activation tensor (Section 3.1): a forward of x_dev ([m x k] fp32,
 * or NHWC images with m = batch) with every layer at 16 bit -- the float model the searches
 * start from -- recording max|input| of every layer.  Synchronises the stream and keeps the
 * table on the host; QCFG_ENONFINITE if any maximum is NaN/Inf.                            */
int qcfg_calibrate_model(qcfg_ctx* ctx, qcfg_model* model, const float* x_dev, int64_t m,
                         void* stream);
/* Copies the calibrated activation maxima (n_layers floats) to a HOST array.              */
int qcfg_model_act_absmax(qcfg_model* model, float* absmax_host);
/* Copies layer `layer`'s per-row weight maxima (n_out floats) to a HOST array (syncs).    */
int qcfg_model_weight_absmax(qcfg_model* model, int32_t layer, float* absmax_host);

/* Evaluate f(x, w) (Algorithm 1 step "Evaluate f(x, lw)", Algorithm 2 "Evaluate f(x, w)"):
 * forward of x_dev under the bit configuration bits[n_layers] (HOST array, values in
 * {2..8, 16}).  Every layer quantizes its input with its calibrated activation scale at its
 * own bit width (the clip of Eq. 1 is live), multiplies by its weight codes at that bit
 * width (cached per (layer, b) after first use), rescales, adds the shortcut and applies the
 * activation.  y_dev is a HOST array of n_layers DEVICE pointers; y_dev[l] receives layer l's
 * fp32 output [rows_l x n_out] when non-NULL.  y_dev itself may be NULL (nothing returned;
 * used when only throughput matters).                                                      */
int qcfg_eval_config(qcfg_ctx* ctx, qcfg_model* model, const uint8_t* bits,
                     const float* x_dev, int64_t m, float* const* y_dev, void* stream);

/* Latency table of Section 4, "Compute Latency Estimates": the paper prices a configuration by
 * benchmarking every layer's kernel at every available precision and adding up the entries the
 * configuration selects.  For each bs[i] (values in {2..8, 16}) the model is run with every
 * layer at that width, `reps` times after one untimed pass, with a CUDA event pair around all
 * the kernels each layer launches (operand preparation and GEMM with its fused epilogue; codes
 * a producer writes for its consumer count towards the producer).  ms_host is a HOST array
 * [n_layers][n_bs] of mean milliseconds.  Synchronises the stream after every pass; event
 * pairs serialise the launches, so a column's sum exceeds the time of one untimed evaluation.
 * On this hardware every integer width 2..8 runs on the same int8 tensor path.               */
int qcfg_latency_table(qcfg_ctx* ctx, qcfg_model* model, const float* x_dev, int64_t m,
                       const uint8_t* bs, int32_t n_bs, int32_t reps, float* ms_host, void* stream);
/* The two deployment costs the searches minimise (Table 1 rows "Size" and "Latency"): size =
 * sum over layers of n_out * k_in * bits[l] / 8 bytes (weights only); latency = sum over layers of
 * the table entry of (l, bits[l]).  Host only.  latency_ms or size_bytes may be NULL; without
 * latency_ms the table arguments are ignored.  A bit width absent from bs gives QCFG_EBITS.  */
int qcfg_config_cost(qcfg_model* model, const uint8_t* bits, const uint8_t* bs, int32_t n_bs,
                     const float* ms_host, double* latency_ms, double* size_bytes);

/* Noise-injection sensitivity E_N (Section 3.1, Eqs. 3-5): for each layer i in turn, Gaussian
 * noise nu = sigma_i * noise_dev[i], sigma_i = lambda * max|w_i| (whole tensor), is added to that
 * layer's weights only, the model is run on x_dev and E_N(i) = L(x, W*) - L(x, W).  The loss needs
 * labels the library does not have: L is the relative distance ||y - y_0||_2 / ||y_0||_2 of the last
 * layer's fp32 output from the noise-free output y_0, so L(x, W) = 0.  The model runs with every
 * layer at 16 bit (the paper's floating-point baseline; the perturbed weights are rounded to bf16
 * like the clean ones).  The second argument of N(0, .) is read as the standard deviation.
 * noise_dev is a HOST array of n_layers DEVICE pointers to the caller's standard-normal draws,
 * [n_out x k_in] row-major like the weights (the generator is the caller's); a NULL entry skips
 * the layer (E_N = 0).  e_n_host receives n_layers doubles.  Costs one forward per perturbed layer
 * plus one; synchronises the stream after each.  No calibration needed.                        */
int qcfg_noise_sensitivity(qcfg_ctx* ctx, qcfg_model* model, const float* x_dev, int64_t m,
                           const float* const* noise_dev, float lambda, double* e_n_host, void* stream);

/* The paper's two configuration searches as host drivers over qcfg_eval_config.
 * QCFG_SEARCH_BISECTION is Algorithm 1, QCFG_SEARCH_GREEDY Algorithm 2.  order[n_layers] lists
 * the layers by ascending sensitivity (e.g. the E_QE ranking from qcfg_quant_error_sweep);
 * bs[n_bs] are the available bit widths.  The working configuration starts at max(bs); the
 * other widths are visited from high to low; the halving steps of Algorithm 1 use floor
 * division and the prefix finally written is the largest one that met the target.
 * "Accuracy" needs data and labels the library does not have; the drivers use the fidelity
 * a = 1 - ||y - y_ref||_2 / ||y_ref||_2 of the LAST layer's fp32 output, y_ref being the output
 * with every layer at max(bs), and accept a candidate when a >= target.
 * Outputs (HOST): bits_out[n_layers] the final configuration; optionally visited
 * [capacity x n_layers] the configurations evaluated, in order, and accuracies[capacity] their
 * fidelities (the first `capacity` evaluations are recorded); n_evals the number of
 * evaluations.  Synchronises the stream after every evaluation.                              */
enum { QCFG_SEARCH_BISECTION = 0, QCFG_SEARCH_GREEDY = 1 };
int qcfg_search(qcfg_ctx* ctx, qcfg_model* model, int algorithm, const int32_t* order,
                const uint8_t* bs, int32_t n_bs, double target, const float* x_dev, int64_t m,
                uint8_t* bits_out, uint8_t* visited, double* accuracies, int32_t capacity,
                int32_t* n_evals, void* stream);

/* Scale adjustment (Section 3.1, second step of the scale estimation; Section 4 gives the
 * learning rate 1e-5): after max calibration the quantization scales are adapted by
 * backpropagation, the model's own parameters staying fixed.  The loss needs labels the library
 * does not have: L = sum (y - y_ref)^2 / sum y_ref^2 on the LAST layer's fp32 output, y_ref being
 * the output with every layer at 16 bit.  The rounding of Eq. 1 is differentiated straight through
 * (derivative 1 inside the clip range, 0 outside).  All four kinds of scale of every layer that
 * runs at an integer width under bits[] are adapted: the activation's scale and inv_scale (one pair
 * per layer) and the weight's per output channel.  Each of `steps` steps is one forward, one
 * backward (two bf16 tensor-core GEMMs per layer) and scale <- float(scale - lr * gradient) on the
 * whole batch x_dev; losses_host (HOST, steps + 1 doubles, may be NULL) receives the loss before
 * every step and after the last.  From then on qcfg_eval_config uses the adapted scales wherever a
 * layer runs at the width it was adapted at; qcfg_calibrate_model and qcfg_model_reset_scales go
 * back to max calibration.  Linear layers only (QCFG_ESHAPE for a convolutional table).
 * Synchronises the stream several times per step.                                              */
int qcfg_adjust_scales(qcfg_ctx* ctx, qcfg_model* model, const uint8_t* bits, const float* x_dev,
                       int64_t m, int32_t steps, double lr, double* losses_host, void* stream);
/* The gradients one step of qcfg_adjust_scales would use, at the model's current scales (HOST
 * outputs, any may be NULL): d_scale_x[n_layers], d_inv_scale_x[n_layers] (0 for 16-bit layers);
 * d_scale_w / d_inv_scale_w are HOST arrays of n_layers HOST pointers to n_out doubles each (a NULL
 * entry skips the layer; 16-bit layers give zeros); *loss the loss.  Changes no scale.          */
int qcfg_scale_gradients(qcfg_ctx* ctx, qcfg_model* model, const uint8_t* bits, const float* x_dev,
                         int64_t m, double* d_scale_x, double* d_inv_scale_x,
                         double* const* d_scale_w, double* const* d_inv_scale_w, double* loss,
                         void* stream);
/* The scales layer `layer` uses at `bits` (2..8) right now: the activation pair and, to HOST arrays
 * of n_out floats, the weight's per-channel pairs.  Outputs may be NULL.                        */
int qcfg_model_scales(qcfg_model* model, int32_t layer, int bits, float* scale_x,
                      float* inv_scale_x, float* scale_w_host, float* inv_scale_w_host);
/* Discards every adapted scale: all layers are back at their max-calibrated scales.             */
int qcfg_model_reset_scales(qcfg_model* model);

/* Parity taps for layer `layer` of the LAST qcfg_eval_config call (same stream order):
 * the int8 codes of its GEMM input (qx_dev, [rows x k_in] dense, or NULL), of its weight
 * (qw_dev, [n_out x k_in] dense, or NULL) and its raw int32 accumulators (acc_dev,
 * [rows x n_out], or NULL; recomputed by a second GEMM launch).  QCFG_EBITS if that layer
 * ran at 16 bit.                                                                           */
int qcfg_debug_dump(qcfg_ctx* ctx, qcfg_model* model, int32_t layer, int8_t* qx_dev,
                    int8_t* qw_dev, int32_t* acc_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QCFG_H_ */
