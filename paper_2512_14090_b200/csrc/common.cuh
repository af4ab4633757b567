// Shared declarations of the AIQ CUDA library (internal; the public ABI is include/aiq.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include <atomic>

#include "../../include/aiq.h"

namespace aiq {

// ---- host-side error plumbing -------------------------------------------------------
aiq_status_t set_error(aiq_status_t status, const char* fmt, ...);
aiq_status_t check_device_sm100();          // AIQ_OK or AIQ_ERR_NOT_SM100 / AIQ_ERR_CUDA
void count_launch();                         // per-thread launch counter (aiq_last_call_stats)

#define AIQ_CUDA_TRY(expr)                                                              \
  do {                                                                                  \
    cudaError_t e__ = (expr);                                                           \
    if (e__ != cudaSuccess)                                                             \
      return ::aiq::set_error(AIQ_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

#define AIQ_LAUNCH_CHECK(what)                                                          \
  do {                                                                                  \
    cudaError_t e__ = cudaGetLastError();                                               \
    if (e__ != cudaSuccess)                                                             \
      return ::aiq::set_error(AIQ_ERR_CUDA, "launch %s: %s", what, cudaGetErrorString(e__)); \
    ::aiq::count_launch();                                                              \
  } while (0)

// Properties of the current device (looked up once per device, then cached).
struct DeviceProps { int dev, n_sms, smem_optin; };
aiq_status_t current_device_props(DeviceProps* out);

// Opt-in of `kernel` to `bytes` of dynamic shared memory.  The attribute belongs to the
// (kernel, device) pair, so the record of what has been set is kept per device; it is only
// written after the runtime call succeeded.  `kernel` must name one kernel per call site.
#define AIQ_ENSURE_DYNAMIC_SMEM(kernel, bytes)                                                   \
  do {                                                                                           \
    static std::atomic<int> set_bytes__[64];                                                     \
    int dev__ = 0;                                                                               \
    AIQ_CUDA_TRY(cudaGetDevice(&dev__));                                                         \
    const bool cached__ = dev__ >= 0 && dev__ < 64;                                              \
    if (!cached__ || set_bytes__[dev__].load(std::memory_order_acquire) < (int)(bytes)) {        \
      AIQ_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(bytes))); \
      if (cached__) set_bytes__[dev__].store((int)(bytes), std::memory_order_release);           \
    }                                                                                            \
  } while (0)

// Brackets one kernel launch with CUDA events while profiling is on (see aiq_profile_start),
// and adds the launch's algorithmic work to the per-kind totals.
struct LaunchScope {
  LaunchScope(int kind, cudaStream_t stream, double flops, double bytes);
  ~LaunchScope();
  int slot_;
  cudaStream_t stream_;
};

inline bool bits_ok(int bits) { return bits == 4 || bits == 8 || bits == 16 || bits == 32; }
inline int padded_k(int K) { return (K + 31) / 32 * 32; }
inline size_t row_bytes(int K, int bits) { return (size_t)padded_k(K) * bits / 8; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- device-side element decode -----------------------------------------------------
// Element k of a packed row as a float: the integer code (4 / 8 bits, unscaled), the half
// (16) or the float (32).
__device__ __forceinline__ float load_element(const uint8_t* __restrict__ row, int k, int bits) {
  switch (bits) {
    case 4: {
      int byte = row[k >> 1];
      int nib = (k & 1) ? (byte >> 4) : (byte & 0xF);
      return (float)((nib ^ 8) - 8);
    }
    case 8:
      return (float)(((const int8_t*)row)[k]);
    case 16:
      return __half2float(((const __half*)row)[k]);
    default:
      return ((const float*)row)[k];
  }
}

__device__ __forceinline__ float apply_act(float v, int act) {
  if (act == AIQ_ACT_RELU) return fmaxf(v, 0.0f);
  if (act == AIQ_ACT_RELU6) return fminf(fmaxf(v, 0.0f), 6.0f);
  return v;
}

// ---- internal activation formats ----------------------------------------------------
// Activation tensors between layers are [B][H+2][W][pixel] with Cs = channels rounded up to
// a multiple of 16 and 4*Cs bytes per pixel.  Rows 0 and H+1 of every image are zero
// (vertical padding stored physically, so that (image, row) is one uniform dimension);
// channels >= C are zero.  Two pixel formats:
//   ACT_F32   Cs floats.  Used when every layer of the model runs on the float32 path.
//   ACT_SPLIT [hi(Cs) | lo(Cs)] bfloat16, value = float(hi) + float(lo) with
//             hi = bf16_rn(v), lo = bf16_rn(v - hi): 16+ significant bits in the same bytes,
//             in the form the bf16 tensor cores consume without conversion (the two halves
//             are two K-slices of the GEMM).  Used when the model has tensor-core layers.
//   ACT_RS    the hi / lo bfloat16 pairs of ACT_SPLIT in the image-interleaved layout of the
//             row-streaming tensor-core convolution (conv_rs.cu):
//             [group][row][column][plane][image][8 bfloat16], G = rs_group_images(width) images per
//             group, plane p < C/8 = hi halves of channels 8p .. 8p+7, plane C/8 + p = their lo
//             halves; no padding rows; the batch is padded to a multiple of 16 images.
enum { ACT_F32 = 0, ACT_SPLIT = 1, ACT_RS = 2 };
inline int rs_group_images(int W) { return W % 16 == 0 ? 8 : 16; }
inline int rs_padded_batch(int B) { return (B + 15) / 16 * 16; }
inline size_t rs_image_bytes(int H, int W, int C) { return (size_t)H * W * 4 * C; }
inline int padded_channels(int C) { return (C + 15) / 16 * 16; }
inline size_t split_image_bytes(int H, int W, int C) {
  return (size_t)(H + 2) * W * 2 * padded_channels(C) * 2;
}

__device__ __forceinline__ void split_bf16(float v, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(v);
  lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// ---- job records: one evaluation of one layer under one weight choice ---------------
// Device-resident arrays of these let a single launch cover every distinct version of a
// layer that a group of schemes needs (gridDim.z = number of jobs).
struct LayerJob {
  const void* in;       // split activations (nullptr: the float32 NCHW network input, a kernel argument);
                        // head jobs: float32 pooled features / logits
  const void* res;      // residual operand (split), or nullptr
  void* out;            // split activations; head jobs: float32
  const uint8_t* w;     // packed rows (aiq_quantize_layer layout)
  const float* scale;   // [cout]
  const float* bias;    // [cout]
  int32_t bits;
  int32_t label_slot;   // head jobs: index of the count / prediction row
  int32_t in_version;   // index of `in` along the version dimension of its slot
  int32_t out_version;  // index of `out` along the version dimension of its slot
  // fused basic block (conv_rs_block_kernel): the block's first convolution; `in` / `in_version` are
  // then that convolution's input, which is also the shortcut
  const uint8_t* w_pre;
  const float* scale_pre;
  const float* bias_pre;
  int32_t bits_pre;
  int32_t bits_mid;
  // fused inverted-residual block (mb_block_kernel): w_pre / scale_pre = operand images / coefficients of the
  // expansion, scale_mid = coefficients of the depthwise layer, w = operand images of the projection
  const uint8_t* w_mid;
  const float* scale_mid;
  const float* bias_mid;
  float* pool;          // fused global average pool: float32 [batch][cout] written instead of `out`, or nullptr
};

struct ConvGeom {
  int B, H, W, Cin, Ho, Wo, Cout, ks, stride, pad, act;
  int K;              // Cin/groups * ks * ks
  int Cs_in, Cs_out;  // padded channel counts of the split tensors
  int in_is_nchw;     // 1: the input is the float32 NCHW network input
  int act_format;     // ACT_F32 or ACT_SPLIT, for input, residual and output alike
};

// ---- launchers (defined in the .cu files) --------------------------------------------
aiq_status_t launch_fold_bn(const float* W, const float* gamma, const float* beta, const float* mean,
                            const float* var, int N, int K, float eps, float* Wf, float* bf,
                            cudaStream_t s);
// tensor_amax: nullptr = one scale per row; else device scratch word and one scale for the whole tensor
aiq_status_t launch_quantize(const float* W, int N, int K, int bits, void* packed, float* scales,
                             int32_t* nonfinite_flag, uint32_t* tensor_amax, cudaStream_t s);
// all four widths (4, 8, 16, 32 bits, in that order) of one layer from one read of W; tensor_amax as above, for the 4- and 8-bit codes
aiq_status_t launch_quantize_bank(const float* W, int N, int K, void* const* packed, float* const* scales,
                                  int32_t* nonfinite_flag, uint32_t* tensor_amax, cudaStream_t s);
// y[m][n] for every job: in = x [M][K], out = y [M][N]
aiq_status_t launch_qlinear(const LayerJob* jobs_dev, const LayerJob* single_host, int n_jobs, int N,
                            int K, int M, cudaStream_t s);
// warp-level tensor-core path of the linear layer (4- / 8-bit weights, M <= 16, large N*K)
bool qlinear_mma_applicable(int N, int K, int bits, int M);
size_t qlinear_mma_workspace_bytes(int K, int M);
aiq_status_t launch_qlinear_mma(const LayerJob& job, int N, int K, int M, void* workspace, cudaStream_t s);
// tcgen05 path of the linear layer (4- / 8-bit weights, M >= 9): weights as the MMA's M operand,
// the batch as its N operand; needs workspace for the activations as two bfloat16 planes
bool qlinear_tc_applicable(int N, int K, int bits, int M);
size_t qlinear_tc_workspace_bytes(int K, int M);
aiq_status_t launch_qlinear_tc(const LayerJob& job, int N, int K, int M, void* workspace, int32_t* error_flag,
                               cudaStream_t s);
// weight_bytes: packed weights + scales + biases of all jobs (for the profile's byte count)
aiq_status_t launch_conv(const ConvGeom& g, const LayerJob* jobs_dev, int n_jobs,
                         const float* net_input, double weight_bytes, cudaStream_t s);
aiq_status_t launch_depthwise(const ConvGeom& g, const LayerJob* jobs_dev, int n_jobs,
                              const float* net_input, double weight_bytes, cudaStream_t s);
// Tensor-core convolution (conv_tc.cu).  `map` points to a 128-byte CUtensorMap over the input
// slot: dims (2*Cs, W, batch_capacity*(H+2), versions).
bool conv_tc_eligible(const ConvGeom& g);
aiq_status_t conv_tc_encode_map(const ConvGeom& g, const void* slot_base, int batch_capacity, int n_versions,
                                void* map_out);
// All jobs of one launch have weights of one class: weight_bits = 8 (4- or 8-bit codes), 16 or 32.
// 16- / 32-bit weights enter as two bfloat16 pieces (hi + lo); conv_tc_bits_ok says whether the kernel takes them.
bool conv_tc_bits_ok(const ConvGeom& g, int bits);
aiq_status_t launch_conv_tc(const ConvGeom& g, const void* map, const LayerJob* jobs_dev, int n_jobs,
                            int batch_capacity, int32_t* error_flag, double weight_bytes, int weight_bits,
                            cudaStream_t s);
// Row-streaming tensor-core convolution on ACT_RS tensors (conv_rs.cu).  `maps`: two CUtensorMaps
// (256 bytes) over the input slot written by conv_rs_encode_maps.  weight_bits as for launch_conv_tc.
bool conv_rs_eligible(const ConvGeom& g);
aiq_status_t conv_rs_encode_maps(const ConvGeom& g, const void* slot_base, int batch_capacity, int n_versions,
                                 void* maps_out);
// pool_jobs: the jobs carry LayerJob::pool; the kernel then writes the global average of its output
// (float32 [batch][Cout]) instead of the output tensor.  Only where conv_rs_pool_fusable(g).
bool conv_rs_pool_fusable(const ConvGeom& g);
aiq_status_t launch_conv_rs(const ConvGeom& g, const void* maps, const LayerJob* jobs_dev, int n_jobs, int batch_capacity,
                            int32_t* error_flag, double weight_bytes, int weight_bits, bool pool_jobs, cudaStream_t s);
// A whole identity-shortcut basic block (two 3x3 convolutions of C -> C channels) in one kernel; `g`
// describes either convolution.  Jobs carry both weight sets (LayerJob::w_pre ...).
// fused MobileNetV2 inverted-residual block (expansion 1x1 -> depthwise 3x3 -> projection 1x1 [+ shortcut]) on split
// activations; the three geometries are those of the block's layers
// hidden channels per chunk (32 or 64) the kernel would use for this block on the current device, 0 = not eligible
int mb_block_chunk_channels(const ConvGeom& ge, const ConvGeom& gd, const ConvGeom& gp);
// bytes of one chunk's operand image: expansion (Cs_in / 8 planes of nh rows), projection (nh / 8 planes of Cs_out rows)
__host__ __device__ inline size_t mb_etile_bytes(int cs_in, int nh) { return (size_t)(cs_in / 8) * (nh * 16); }
__host__ __device__ inline size_t mb_ptile_bytes(int cs_out, int nh) { return (size_t)(nh / 8) * (cs_out * 16); }
// role 0: expansion, 1: projection, 2: depthwise (coefficients only); see mb_block.cu
aiq_status_t launch_mb_build_tiles(int role, const uint8_t* packed, const float* scale, const float* bias, int bits, int N,
                                   int K, int nh, int cs, void* tile_out, float* coef_out, cudaStream_t s);
// whether the fused kernel is expected to beat the layer kernels for this block at this batch (measured policy)
bool mb_block_pays(const ConvGeom& gd, const ConvGeom& gp);
// nh: the chunk width the jobs' operand images were built for
aiq_status_t launch_mb_block(const ConvGeom& ge, const ConvGeom& gd, const ConvGeom& gp, int nh, const LayerJob* jobs_dev, int n_jobs,
                             int32_t* error_flag, double weight_bytes, cudaStream_t s);
bool conv_rs_block_eligible(const ConvGeom& g);
aiq_status_t launch_conv_rs_block(const ConvGeom& g, const void* maps, const LayerJob* jobs_dev, int n_jobs, int batch_capacity,
                                  int32_t* error_flag, double weight_bytes, cudaStream_t s);
// Pointwise (1x1, stride 1) tensor-core convolution for any channel count that is a multiple
// of 8 (conv_pw_tc.cuh).  `map`: CUtensorMap over the input slot, dims (Cs, 2, pixels of all versions).
bool conv_pw_tc_eligible(const ConvGeom& g);
aiq_status_t conv_pw_tc_encode_map(const ConvGeom& g, const void* slot_base, int batch_capacity, int n_versions,
                                   void* map_out);
// store map over the output slot: dims (Cs_out, 2, pixels per version, versions)
aiq_status_t conv_pw_tc_encode_out_map(const ConvGeom& g, const void* slot_base, int batch_capacity, int n_versions,
                                       void* map_out);
// weight_bits: 8 (4- or 8-bit codes), 16 or 32 (two bfloat16 pieces per weight); one class per launch
aiq_status_t launch_conv_pw_tc(const ConvGeom& g, const void* map, const void* out_map, const LayerJob* jobs_dev, int n_jobs,
                               int batch_capacity, int32_t* error_flag, double weight_bytes, int weight_bits, cudaStream_t s);
// Test aid: a one-thread kernel whose bounded wait runs out after `limit_cycles` SM clocks; it sets
// *error_flag to 1 and *observed (optional) to 2, then returns.
aiq_status_t launch_expire_wait(int32_t* error_flag, long long limit_cycles, int32_t* observed, cudaStream_t s);
// pooled[b][c] = mean over the H x W interior of a split tensor, per job (in -> out float32 [B][C])
aiq_status_t launch_avgpool(const LayerJob* jobs_dev, int n_jobs, int B, int H, int W, int C, int act_format,
                            cudaStream_t s);
// pred = lowest index of the max logit; preds[slot][img0 + b] = pred; counts[slot] += (pred == label)
aiq_status_t launch_argmax_count(const LayerJob* jobs_dev, int n_jobs, int B, int n_classes,
                                 const int32_t* labels, int32_t* counts, int32_t* preds,
                                 long long preds_stride, long long img0, cudaStream_t s);

}  // namespace aiq
