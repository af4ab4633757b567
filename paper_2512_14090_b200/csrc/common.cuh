// Shared declarations of the AIQ CUDA library (internal; the public ABI is include/aiq.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

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

// ---- job records: one evaluation of one layer under one weight choice ---------------
// Device-resident arrays of these let a single launch cover every distinct version of a
// layer that a group of schemes needs (gridDim.z = number of jobs).
struct LayerJob {
  const float* in;      // activations NHWC (nullptr: the network input passed as a kernel argument)
  const float* res;     // residual operand NHWC, or nullptr
  float* out;           // NHWC
  const uint8_t* w;     // packed rows (aiq_quantize_layer layout)
  const float* scale;   // [cout]
  const float* bias;    // [cout]
  int32_t bits;
  int32_t label_slot;   // head jobs: index of the count / prediction row
};

struct ConvGeom {
  int B, H, W, Cin, Ho, Wo, Cout, ks, stride, pad, act;
  int K;            // Cin/groups * ks * ks
  int row_bytes;    // packed row stride at the job's bit-width is computed per job
  long long in_sb, in_sy, in_sx, in_sc;   // element strides of the input tensor
};

// ---- launchers (defined in the .cu files) --------------------------------------------
aiq_status_t launch_fold_bn(const float* W, const float* gamma, const float* beta, const float* mean,
                            const float* var, int N, int K, float eps, float* Wf, float* bf,
                            cudaStream_t s);
aiq_status_t launch_quantize(const float* W, int N, int K, int bits, void* packed, float* scales,
                             int32_t* nonfinite_flag, cudaStream_t s);
// y[m][n] for every job: in = x [M][K], out = y [M][N]
aiq_status_t launch_qlinear(const LayerJob* jobs_dev, const LayerJob* single_host, int n_jobs, int N,
                            int K, int M, cudaStream_t s);
// weight_bytes: packed weights + scales + biases of all jobs (for the profile's byte count)
aiq_status_t launch_conv(const ConvGeom& g, const LayerJob* jobs_dev, int n_jobs,
                         const float* net_input, double weight_bytes, cudaStream_t s);
aiq_status_t launch_depthwise(const ConvGeom& g, const LayerJob* jobs_dev, int n_jobs,
                              const float* net_input, double weight_bytes, cudaStream_t s);
// pooled[b][c] = mean over HW of in[b][hw][c], per job (in -> out)
aiq_status_t launch_avgpool(const LayerJob* jobs_dev, int n_jobs, int B, int HW, int C, cudaStream_t s);
// pred = lowest index of the max logit; preds[slot][img0 + b] = pred; counts[slot] += (pred == label)
aiq_status_t launch_argmax_count(const LayerJob* jobs_dev, int n_jobs, int B, int n_classes,
                                 const int32_t* labels, int32_t* counts, int32_t* preds,
                                 long long preds_stride, long long img0, cudaStream_t s);

}  // namespace aiq
