/*
 * aiq.h - C ABI of the B200 (sm_100a) scheme evaluator for Arithmetic-Intensity-Aware
 * Quantization (AIQ).
 *
 * The paper (Section 2.1) assigns every layer i of a trained CNN a bit-width q_i from a
 * small set Q, forming a scheme q = (q_1 .. q_L), and scores a scheme by (i) its global
 * arithmetic intensity AI(q), computed analytically, and (ii) its accuracy, measured by
 * running the quantized model (Section 1).  Both search loops of Section 2.2 spend their
 * time in (ii).  This library is that evaluation path:
 *
 *   aiq_fold_bn          fold batch-norm into the preceding convolution
 *   aiq_quantize_layer   quantize + pack one layer's weights at 4 / 8 / 16 / 32 bits
 *   aiq_qlinear          y = x * dequant(W)^T for a packed weight matrix (small batch)
 *   aiq_model_create     fold, then build the L x {4,8,16,32} bank of packed weights
 *   aiq_forward          logits of one scheme on one image batch
 *   aiq_eval_schemes     top-1 agreement of many schemes on an image set
 *   aiq_scheme_ai        AI(q), on the host
 *   aiq_search_greedy / aiq_search_coordinate_descent   the searches of Section 2.2
 *
 * Conventions
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are
 *     ordinary host memory.  The library never allocates or frees device memory: the
 *     caller provides model memory and workspace and keeps them alive while they are used.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Every function returns an aiq_status_t (0 = AIQ_OK) unless stated; nothing throws.
 *     aiq_last_error() gives a thread-local detail string for the last non-zero status.
 *   - Bit-widths: 4 and 8 are symmetric integer codes with one float32 scale per output
 *     channel; 16 is IEEE half; 32 is float32.  Anything else: AIQ_ERR_UNSUPPORTED_BITS.
 *   - There is no CPU fallback: on a device that is not compute capability 10.x every
 *     entry point that would launch a kernel returns AIQ_ERR_NOT_SM100.
 */
#ifndef AIQ_H_
#define AIQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int aiq_status_t;
enum {
  AIQ_OK = 0,
  AIQ_ERR_INVALID_ARG = 1,       /* null pointer, non-positive size, bad wiring              */
  AIQ_ERR_UNSUPPORTED_BITS = 2,  /* bit-width outside {4, 8, 16, 32}                         */
  AIQ_ERR_SHAPE = 3,             /* layer shapes inconsistent with the wiring                */
  AIQ_ERR_WORKSPACE_TOO_SMALL = 4,
  AIQ_ERR_CUDA = 5,              /* a CUDA runtime call failed; see aiq_last_error()         */
  AIQ_ERR_NOT_SM100 = 6,
  AIQ_ERR_NONFINITE = 7,         /* a weight was NaN or infinite                             */
  AIQ_ERR_TIMEOUT = 8            /* a bounded device-side wait expired                       */
};

/* Static description of a status code. Never NULL. */
const char* aiq_status_string(aiq_status_t status);
/* Thread-local detail of the last failure on this thread ("" if none). */
const char* aiq_last_error(void);

/* ------------------------------------------------------------------------------------
 * Batch-norm folding.  The paper evaluates a trained model as-is (Section 3); folding the
 * inference batch-norm into the convolution before quantizing is this library's stated
 * reading.  Per output channel n:
 *     g = gamma[n] / sqrt(var[n] + eps);   Wf[n][k] = W[n][k] * g;   bf[n] = beta[n] - mean[n] * g
 * float32, every operation rounded once (no fused multiply-add, IEEE division and sqrt).
 * W, Wf: device [N][K] row-major (K = cin/groups * kh * kw in (c, r, t) order);
 * gamma, beta, mean, var, bf: device [N].  Wf may alias W.  Asynchronous on `stream`.
 */
aiq_status_t aiq_fold_bn(const float* W, const float* gamma, const float* beta,
                         const float* mean, const float* var, int N, int K, float eps,
                         float* Wf, float* bf, void* stream);

/* ------------------------------------------------------------------------------------
 * Quantize + pack (Section 2.1: layer i is stored at q_i bits; the paper prints no
 * quantizer formula, so the rule is: symmetric, per output channel, max-abs scale, round
 * half to even).  For row n of W [N][K]:
 *   bits 4 / 8: qmax = 2^(bits-1) - 1; amax = max_k |W[n][k]|; s_n = amax / qmax (IEEE
 *               float32 division; s_n = 1 when amax == 0);
 *               code = clamp(rint(W[n][k] / s_n), -2^(bits-1), 2^(bits-1) - 1)
 *   bits 16:    IEEE half, round to nearest even;  s_n = 1
 *   bits 32:    bit copy;                          s_n = 1
 * Packed layout: row-major, row stride aiq_packed_row_bytes(K, bits) = Kpad * bits / 8 with
 * Kpad = K rounded up to a multiple of 32 elements; padding elements are zero.  At 4 bits
 * byte j of a row holds element 2j in its low nibble and element 2j+1 in its high nibble,
 * two's complement.  16- and 32-bit elements are little endian.
 *
 * W: device float32 [N][K].  packed_out: device, N * row_bytes, 16-byte aligned.
 * scales_out: device float32 [N].  nonfinite_flag: optional device int32; set to 1 when a
 * NaN or infinity is met (outputs are then unspecified), to 2 if a bounded wait inside the
 * kernel for large matrices expired (should not happen; outputs invalid); never cleared by
 * the call.  Asynchronous on `stream`.
 */
size_t aiq_packed_row_bytes(int K, int bits);   /* 0 for an unsupported bits or K <= 0 */
aiq_status_t aiq_quantize_layer(const float* W, int N, int K, int bits, void* packed_out,
                                float* scales_out, int32_t* nonfinite_flag, void* stream);

/* The same quantizer with ONE scale for the whole tensor instead of one per output channel:
 * amax = max |W[n][k]| over all n and k, s = amax / qmax, every entry of scales_out holds s (so the
 * forward kernels need no second code path).  The paper prints no quantizer and lists per-channel
 * effects as future work (Section 6), which makes this the granularity its own experiments most
 * likely used; the per-channel rule above is this library's default.  16 and 32 bits do not
 * depend on the granularity.  scratch: device, 4 bytes, 4-byte aligned (holds the tensor maximum
 * during the call).  Otherwise as aiq_quantize_layer. */
aiq_status_t aiq_quantize_layer_per_tensor(const float* W, int N, int K, int bits, void* packed_out,
                                           float* scales_out, int32_t* nonfinite_flag, void* scratch,
                                           void* stream);

/* Scale granularity of the weight banks of models created after the call (process-wide; default
 * AIQ_SCALE_PER_CHANNEL).  The analytic AI of a scheme does not depend on it. */
enum { AIQ_SCALE_PER_CHANNEL = 0, AIQ_SCALE_PER_TENSOR = 1 };
void aiq_set_scale_granularity(int granularity);

/* ------------------------------------------------------------------------------------
 * Small-batch quantized linear layer - the memory-bound case the method targets
 * (Abstract; Section 5, Roofline paragraph): weight bytes N*K*bits/8 dominate the traffic.
 *     y[m][n] = s_n * sum_k code[n][k] * x[m][k] + bias[n]
 * (16 / 32 bits: the stored element itself, s_n = 1).  packed / scales: as written by
 * aiq_quantize_layer (device).  bias: device [N] or NULL.  x: device float32 [M][K]
 * row-major, 16-byte aligned; y: device float32 [M][N].  M >= 1.  Asynchronous on `stream`.
 *
 * Three kernels.  The plain one expands weights to float32 in registers and accumulates in
 * float32 (any shape, any bit-width).  For 4- / 8-bit weights two faster ones exist:
 *   M <= 8, K a multiple of 512, N*K >= 2^20: the codes stay integer and feed the int8
 *     warp-level tensor cores; the activations of each group of 512 k become three int8
 *     digits with a shared exponent (21 bits below the group's largest |x|), the int32 sums
 *     are exact.
 *   M >= 9, K a multiple of 8, K >= 64, N >= 32: a tcgen05 GEMM with the weight matrix as the
 *     MMA's M operand (codes expanded to bfloat16 in shared memory, exact) and the batch as
 *     its N operand; the activations enter as the sum of two bfloat16 (relative rounding
 *     2^-17), accumulation is float32.
 * Both split K over thread blocks where the matrix has too few rows to fill the GPU; the
 * partial sums then meet in y through float atomics (run-to-run differences in the last
 * bit).  Both need scratch memory: pass `workspace` (device, 16-byte aligned) of at least
 * aiq_qlinear_workspace_bytes(...) bytes; with workspace == NULL, or where that function
 * returns 0, the plain kernel runs.
 * Device-side failure: the tcgen05 kernel bounds every wait on its copy / MMA pipeline (about
 * 2 s of SM clocks).  Should one expire, the kernel stops early and y is invalid; the call has
 * long returned AIQ_OK by then, so the record is on the device: the int32 at byte offset
 * aiq_qlinear_workspace_bytes(...) - 16 of `workspace` is set to 0 by every call that uses the
 * tcgen05 kernel and to 1 by a kernel whose wait expired.  Read it after synchronising.
 */
size_t aiq_qlinear_workspace_bytes(int N, int K, int bits, int M);
aiq_status_t aiq_qlinear(const void* packed, const float* scales, const float* bias, int N,
                         int K, int bits, const float* x, int M, float* y, void* workspace,
                         size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * Model description.  Layers are listed in scheme order: entry i of a scheme is the
 * bit-width of layers[i] (Section 2.1).  A layer reads the output of layer `input`
 * (-1 = the network input) and, before its activation, adds the output of layer
 * `residual` (-1 = none).  `input` / `residual` may refer to a later entry (a block's
 * projection shortcut is listed after the convolution that adds it); the wiring must be
 * acyclic.  An AIQ_LAYER_FC layer consumes the global average pool of its input layer.
 * The last layer produces the logits.
 */
enum { AIQ_LAYER_CONV = 0, AIQ_LAYER_DEPTHWISE = 1, AIQ_LAYER_FC = 2 };
enum { AIQ_ACT_NONE = 0, AIQ_ACT_RELU = 1, AIQ_ACT_RELU6 = 2 };

typedef struct aiq_layer_desc {
  int32_t kind;      /* AIQ_LAYER_*                                        */
  int32_t cin;       /* input channels (depthwise: == cout)                */
  int32_t cout;      /* output channels / classes                          */
  int32_t ksize;     /* square kernel: 1 or 3 (fc: 1)                      */
  int32_t stride;    /* 1 or 2                                             */
  int32_t pad;       /* zero padding on each side                          */
  int32_t act;       /* AIQ_ACT_*, applied after bias and residual         */
  int32_t input;     /* producing layer, -1 = network input                */
  int32_t residual;  /* layer added before the activation, -1 = none       */
  int32_t has_bn;    /* 1: gamma/beta/mean/var given and folded; 0: bias   */
} aiq_layer_desc_t;

typedef struct aiq_arch_desc {
  int32_t n_layers;
  int32_t in_c, in_h, in_w;        /* network input, NCHW                  */
  const aiq_layer_desc_t* layers;  /* host [n_layers]                      */
} aiq_arch_desc_t;

/* Host pointers to one layer's trained float32 parameters.  W: [cout][cin/groups][k][k]
 * (fc: [cout][cin]).  has_bn: gamma, beta, mean, var [cout], bias ignored.  Otherwise
 * bias [cout] (NULL = zeros) and the batch-norm pointers are ignored. */
typedef struct aiq_layer_weights {
  const float* W;
  const float* gamma;
  const float* beta;
  const float* mean;
  const float* var;
  const float* bias;
} aiq_layer_weights_t;

typedef struct aiq_model aiq_model_t;   /* opaque host object */

/* Device bytes aiq_model_create needs for `arch` (folded weights, biases, the packed
 * weight bank at all four bit-widths, scales).  0 on an invalid description. */
size_t aiq_model_bytes(const aiq_arch_desc_t* arch);

/* Uploads the weights, folds batch-norm (eps = 1e-5) and quantizes every layer at 4, 8,
 * 16 and 32 bits into `dev_mem` (device, 256-byte aligned, >= aiq_model_bytes(arch)).
 * A layer's quantized weights depend only on (layer, bits), so a scheme is an index vector
 * into this bank.  Synchronises `stream` before returning.  The model refers to `dev_mem`
 * until aiq_model_destroy; the arch and weight arrays are copied and may be freed.
 * Errors: AIQ_ERR_INVALID_ARG / AIQ_ERR_SHAPE (wiring, shapes), AIQ_ERR_WORKSPACE_TOO_SMALL
 * (dev_bytes), AIQ_ERR_NONFINITE, AIQ_ERR_NOT_SM100, AIQ_ERR_CUDA.  *out is NULL on error. */
aiq_status_t aiq_model_create(const aiq_arch_desc_t* arch, const aiq_layer_weights_t* weights,
                              void* dev_mem, size_t dev_bytes, void* stream, aiq_model_t** out);
/* Frees the host object only (device memory belongs to the caller). NULL is accepted. */
void aiq_model_destroy(aiq_model_t* model);
int aiq_model_num_layers(const aiq_model_t* model);   /* L, the scheme length; -1 if NULL */
int aiq_model_num_classes(const aiq_model_t* model);  /* cout of the last layer           */
/* Synchronises `stream` and reports a device-side failure recorded by an earlier
 * asynchronous call on this model (AIQ_ERR_TIMEOUT: a bounded wait inside a kernel expired;
 * the outputs of that call are then invalid).  AIQ_OK otherwise.  Clears the record. */
aiq_status_t aiq_model_status(const aiq_model_t* model, void* stream);

/* Test aid for the failure path above (no counterpart in the paper).  Launches a one-thread
 * kernel that waits, with the same bounded-wait routine as the tensor-core kernels, on a
 * barrier nothing arrives at.  After `limit_cycles` SM clocks (0 < limit_cycles <= 2e9) the
 * wait gives up, records the failure in the model's device status word and the kernel returns
 * normally; the next aiq_model_status / aiq_eval_schemes on this model then reports
 * AIQ_ERR_TIMEOUT and clears the record.  Asynchronous on `stream`. */
aiq_status_t aiq_debug_expire_wait(const aiq_model_t* model, int64_t limit_cycles, void* stream);

/* Device views into the model memory, for inspection: folded weights Wf [cout][K] and bias
 * [cout] of `layer`; packed rows and scales of (`layer`, `bits`) in the layout of
 * aiq_quantize_layer.  Any output pointer may be NULL. */
aiq_status_t aiq_model_layer_folded(const aiq_model_t* model, int layer, const float** Wf,
                                    const float** bias, int* N, int* K);
aiq_status_t aiq_model_layer_packed(const aiq_model_t* model, int layer, int bits,
                                    const void** packed, const float** scales);

/* Workspace bytes sufficient for aiq_forward with batch <= max_batch and for
 * aiq_eval_schemes with n_schemes <= max_schemes processing max_batch images at a time. */
size_t aiq_workspace_bytes(const aiq_model_t* model, int max_batch, int max_schemes);

/* ------------------------------------------------------------------------------------
 * One scheme, one batch (Section 1 (ii): the quantized model is run).  scheme_bits: host
 * uint8 [L].  x: device float32 NCHW [batch][in_c][in_h][in_w].  logits: device float32
 * [batch][n_classes].  Layer l uses the bank entry (l, scheme_bits[l]); weights are
 * expanded from their packed form inside the kernels, products accumulate in float32, the
 * per-channel scale multiplies the finished sum.  workspace: device, 256-byte aligned.
 * Asynchronous on `stream` (the scheme is consumed before the call returns).
 */
aiq_status_t aiq_forward(const aiq_model_t* model, const uint8_t* scheme_bits, const float* x,
                         int batch, float* logits, void* workspace, size_t workspace_bytes,
                         void* stream);

/* ------------------------------------------------------------------------------------
 * aiq_forward without a caller-provided workspace.  (The paper has no counterpart: this is
 * a packaging variant of aiq_forward, not a step of the method.)
 *
 * Some callers cannot obtain device memory at the moment they need a forward pass: code
 * that runs inside another framework's callback where cudaMalloc (which synchronises the
 * whole device) is forbidden, services that received a fixed memory budget at start-up and
 * have already handed all of it out, or plug-ins that are given input and output buffers
 * and nothing else.  For them the library carries its own workspace: a fixed device array
 * of AIQ_STATIC_WORKSPACE_BYTES that belongs to the library image.  Every GPU that loads
 * the library holds that array until the process exits, whether or not this call is used.
 *
 * Same arguments, results and asynchrony as aiq_forward, minus the workspace.  The call
 * makes no cudaMalloc / cudaFree and uses no allocating library routine.
 *   - Limit: if the model at this batch needs more than AIQ_STATIC_WORKSPACE_BYTES in its own
 *     activation format (aiq_workspace_bytes(model, batch, 1) after aiq_set_small_pass_images(0)) the call returns AIQ_ERR_WORKSPACE_TOO_SMALL
 *     and launches nothing; lower the batch or use aiq_forward.  8 MiB fits, e.g.,
 *     ResNet-20 up to batch 32.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress with that device current).  Like aiq_forward, the call plans on
 *     the host and copies its job records from host memory: make no call of it while the
 *     stream is being captured.
 *   - All calls on a device share the one array and it keeps whatever the previous call
 *     left there.  A forward pass needs nothing zeroed, so nothing is cleared; but two calls
 *     whose kernels overlap on the GPU (different streams, or different host threads) write
 *     the same scratch and race.  Issue them on one stream, or order them yourself.
 */
#define AIQ_STATIC_WORKSPACE_BYTES (8u * 1024u * 1024u)
aiq_status_t aiq_forward_static(const aiq_model_t* model, const uint8_t* scheme_bits,
                                const float* x, int batch, float* logits, void* stream);

/* ------------------------------------------------------------------------------------
 * Many candidate schemes, whole evaluation set - the inner loop of greedy search and
 * coordinate descent (Section 2.2), which evaluates L(q; lambda) for every candidate move
 * and so needs each candidate's accuracy on the validation images.
 * schemes: host uint8 [n_schemes][L].  x: device float32 NCHW [n_images][...].  labels:
 * device int32 [n_images].  acc: host float32 [n_schemes] = correct / n_images, where a
 * prediction is the lowest index attaining the maximum logit.  correct_counts: optional
 * host int32 [n_schemes].  preds: optional device int32 [n_schemes][n_images].
 * Images are processed in chunks sized to the workspace; within a chunk, work shared by
 * candidates (equal bit-widths on a common prefix of the network) is done once, which
 * does not change any result.  Synchronises `stream` before returning.
 */
aiq_status_t aiq_eval_schemes(const aiq_model_t* model, const uint8_t* schemes, int n_schemes,
                              const float* x, const int32_t* labels, int n_images, float* acc,
                              int32_t* correct_counts, int32_t* preds, void* workspace,
                              size_t workspace_bytes, void* stream);

/* Evaluation knobs (process-wide, for experiments and tests; results never depend on
 * them).  chunk: images per pass, 0 = choose from the workspace size.  share_prefix: 0
 * evaluates every scheme independently. */
void aiq_set_eval_options(int chunk, int share_prefix);

/* Kernel fusion on networks stored for the row-streaming kernel (process-wide, both default on; the
 * paper's searches only pay off if a candidate evaluation is cheap, Section 2.2).
 *   blocks: bit 0 (default on): a basic block out = relu(conv2(relu(conv1(x))) + x) with two 3x3
 *           convolutions of 16 or 32 channels runs as one kernel whenever every scheme of the call gives
 *           both convolutions 4 or 8 bits: the intermediate tensor stays in shared memory.  Results are
 *           bit-identical to the layer-by-layer path.
 *           bit 2 (default on) / bit 1 (default off): a MobileNetV2 inverted-residual block (expansion 1x1 -> depthwise 3x3 ->
 *           projection 1x1, optional shortcut) runs as one kernel whenever every scheme gives both 1x1
 *           layers 4 or 8 bits: the six-fold hidden tensor stays in shared memory (float32 there, so the
 *           results differ from the layer-by-layer path by that path's rounding of the hidden tensor).
 *           Bit 2 fuses a block only where the fused kernel was measured faster than the three layer kernels
 *           (maps at most 8 columns wide, or stride 2 on maps up to 56 wide, and at least 128 bands of
 *           128 output pixels in the pass); bit 1 fuses every eligible block.
 *   pool:   the classifier's global average pool is taken in the epilogue of the convolution that
 *           produces its input; that tensor is then never stored.  Sums are formed in a fixed order
 *           (run-to-run identical); they differ from the separate pooling kernel's in the last bits. */
void aiq_set_fusion(int blocks, int pool);

/* Small passes (process-wide; evaluation cost, Section 2.2).  The row-streaming kernels work on groups of 8 or
 * 16 images, so a pass of a few hundred images leaves most SMs idle.  A model created under
 * AIQ_PATH_AUTO that stores its activations in the row-streaming format also keeps the pixel-tile view of
 * the same weights; aiq_forward and aiq_eval_schemes run a pass of fewer than `image_schemes` (images of the
 * pass x schemes; default 1024) on that view.  0: always the row-streaming kernels.  Both views meet the same
 * tolerances; their logits differ in the last bits.  aiq_forward_static always uses the model's own format. */
void aiq_set_small_pass_images(int image_schemes);

/* Compute path of models created after the call (process-wide; the paper has no kernels,
 * Section 3 runs stock PyTorch, so this is an implementation choice, not a step of AIQ):
 *   AIQ_PATH_FP32    every layer on float32 multiply-add kernels, activations stored as
 *                    float32.  Logits agree with a float64 reference to ~1e-5 relative.
 *   AIQ_PATH_TENSOR  dense 3x3 / 1x1 convolutions with 4- or 8-bit weights and 16/32/64
 *                    channels run on the bf16 tensor cores (tcgen05, float32 accumulation
 *                    in tensor memory); activations are stored as the sum of two bfloat16
 *                    (17-18 significant bits).  Other layers use the float32 kernels on the
 *                    same storage.
 *                    Networks that consist of a 3x3 stem and dense 3x3 / 1x1 convolutions with
 *                    16, 32 or 64 channels on maps 8 to 64 columns wide (the CIFAR ResNets) are
 *                    stored image-interleaved and run on the row-streaming tensor-core kernel,
 *                    which folds the three vertical taps into the width of one MMA.
 *   AIQ_PATH_TENSOR_TILES  AIQ_PATH_TENSOR without the row-streaming kernel: every tensor-core
 *                    layer runs on the kernels that tile the output pixels.
 *   AIQ_PATH_AUTO    AIQ_PATH_TENSOR when the model has at least one layer the tensor
 *                    kernels accept, else AIQ_PATH_FP32.  This is the default.
 */
enum { AIQ_PATH_AUTO = 0, AIQ_PATH_FP32 = 1, AIQ_PATH_TENSOR = 2, AIQ_PATH_TENSOR_TILES = 3 };
void aiq_set_compute_path(int path);

/* Counters of the last aiq_forward / aiq_eval_schemes call on this thread: kernels
 * launched, and layer evaluations executed vs. n_schemes * L * chunks without sharing. */
void aiq_last_call_stats(int64_t* kernel_launches, int64_t* layer_evals, int64_t* layer_evals_unshared);

/* ------------------------------------------------------------------------------------
 * Analytic global arithmetic intensity (Section 1 (i); Section 2.2: "AI can be recomputed
 * analytically").  The paper gives no formula; this one is used:
 *     FLOPs_l = 2 * cout * K * Ho * Wo * ai_batch
 *     Bytes_l = cout * K * q_l / 8 + 4 * ai_batch * (cin * Hi * Wi + cout * Ho * Wo)
 *     AI(q)   = sum_l FLOPs_l / sum_l Bytes_l          [FLOP / byte]
 * over every weight layer; biases, scales, activations functions, residual adds and
 * pooling count for nothing.  Host only, no CUDA call.  ai, flops, bytes: host doubles
 * (each may be NULL).
 */
aiq_status_t aiq_scheme_ai(const aiq_model_t* model, const uint8_t* scheme_bits, int ai_batch,
                           double* ai, double* flops, double* bytes);

/* ------------------------------------------------------------------------------------
 * The two searches of Section 2.2 over the AIQ objective of Section 2.1,
 *     L(q; lambda) = -lambda * AI(q) + (1 - lambda) * AccLoss(q),
 * as host loops over aiq_eval_schemes and aiq_scheme_ai (every candidate of an iteration is
 * scored in one aiq_eval_schemes call).  The paper fixes neither the units of AccLoss nor a
 * normalisation of AI; used here: AccLoss(q) = 100 * (acc(q_FP32) - acc(q)) (percentage
 * points, both accuracies measured on the given images) and AI in FLOP per byte at batch 1.
 *
 * Both start from the all-32-bit scheme.  `layers`: host int32 list of the layers that may
 * move (NULL = all L layers), visited in the given order.  `options`: host uint8 list of
 * bit-widths, in the order in which ties are broken.  x, labels, workspace, stream: as for
 * aiq_eval_schemes; the workspace must cover n_layers * n_options schemes.
 *
 * aiq_search_greedy: per iteration the candidate moves are "set a selectable layer that is
 *   still at 32 bits to an option below 32"; the move with the smallest Delta L is applied
 *   when Delta L < 0 (first candidate in (layer, option) order on ties); n_layers iterations
 *   at most, ending early once no move lowers L (the scheme could not change any more).
 * aiq_search_coordinate_descent: passes over the selectable layers; each layer takes the
 *   option with the smallest L, the others held fixed (the current value stays unless an
 *   option is strictly better); passes repeat until one changes nothing, max_passes at most.
 *
 * scheme_out: host uint8 [L].  trace (optional): one record per iteration (greedy) or per
 * layer visit (coordinate descent), the first trace_capacity of them; *n_trace = how many
 * there were.  Synchronous (every iteration reads accuracies back).
 */
typedef struct aiq_search_step {
  int32_t layer;       /* layer of the best move of this iteration / the layer visited      */
  int32_t bits;        /* its new bit-width (coordinate descent: its bit-width afterwards)   */
  int32_t accepted;    /* 1 if the scheme changed                                            */
  int32_t candidates;  /* schemes evaluated in this iteration                                */
  double loss;         /* L of the scheme after the iteration                                */
  double acc;          /* accuracy of the scheme after the iteration (greedy, rejected move: */
                       /* of the rejected candidate)                                         */
  double ai;           /* AI of that scheme                                                  */
} aiq_search_step_t;
aiq_status_t aiq_search_greedy(const aiq_model_t* model, const int32_t* layers, int n_layers,
                               const uint8_t* options, int n_options, double lambda, const float* x,
                               const int32_t* labels, int n_images, uint8_t* scheme_out,
                               aiq_search_step_t* trace, int trace_capacity, int* n_trace,
                               void* workspace, size_t workspace_bytes, void* stream);
aiq_status_t aiq_search_coordinate_descent(const aiq_model_t* model, const int32_t* layers, int n_layers,
                                           const uint8_t* options, int n_options, double lambda,
                                           int max_passes, const float* x, const int32_t* labels,
                                           int n_images, uint8_t* scheme_out, aiq_search_step_t* trace,
                                           int trace_capacity, int* n_trace, void* workspace,
                                           size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * Per-kernel timing.  The paper measures throughput by wall clock (Section 3, experiment
 * 3); this is the device-side equivalent for the kernels of this library.  Between
 * aiq_profile_start and aiq_profile_stop every kernel launch made by the calling thread is
 * bracketed by CUDA events on its stream.  aiq_profile_stop synchronises those events and
 * fills out[kind] with the number of launches, their summed duration in milliseconds, and
 * the algorithmic work they were asked to do: floating-point operations (2 per
 * multiply-add) and bytes (packed weights + scales once, input and output tensors once).
 * Event records cost about a microsecond each on the host; leave profiling off otherwise.
 */
enum {
  AIQ_KERNEL_FOLD = 0,
  AIQ_KERNEL_QUANTIZE = 1,
  AIQ_KERNEL_QLINEAR = 2,
  AIQ_KERNEL_CONV = 3,
  AIQ_KERNEL_DEPTHWISE = 4,
  AIQ_KERNEL_POOL = 5,
  AIQ_KERNEL_ARGMAX = 6,
  AIQ_KERNEL_CONV_TC = 7,   /* tensor-core convolution */
  AIQ_KERNEL_KINDS = 8
};
typedef struct aiq_kernel_profile {
  int64_t launches;
  double ms;
  double flops;
  double bytes;
} aiq_kernel_profile_t;
aiq_status_t aiq_profile_start(void);
aiq_status_t aiq_profile_stop(aiq_kernel_profile_t* out /* host [AIQ_KERNEL_KINDS] */);

#ifdef __cplusplus
}
#endif
#endif /* AIQ_H_ */
