// Depthwise 3x3 convolution (stride 1 or 2, pad 1) with bias, residual and activation.
//
// The layer moves 8 bytes per output element for 18 FLOP: it is bound by memory traffic, so
// the kernel is organised around wide, coalesced accesses and input reuse in registers:
//   - a thread owns 8 consecutive channels (16-byte loads: one for the hi and one for the lo
//     half of a split pixel, two for a float32 pixel) and 4 consecutive output columns;
//   - for each of the 3 input rows it loads the 6 (stride 1) or 9 (stride 2) input columns
//     its 4 outputs need once and feeds all taps from registers;
//   - work items (output row, column group, channel octet) are flattened with the channel
//     octet fastest, so consecutive lanes touch consecutive 16-byte units whatever the
//     channel count (32 .. 960 in MobileNetV2);
//   - the 9 x C expanded weights, scales and biases sit in shared memory; blocks are
//     persistent (grid-stride over items).
// Rows 0 and Ho+1 of every output image (the physical padding rows) are written as zeros.
#include "common.cuh"

namespace aiq {

namespace {

constexpr int kDwThreads = 256;
constexpr int kDwCols = 2;        // output columns per thread

template <int FMT>
__device__ __forceinline__ void load8(const void* __restrict__ base, size_t pixel, int c, int Cs, float* v) {
  if (FMT == ACT_SPLIT) {
    const __nv_bfloat16* px = static_cast<const __nv_bfloat16*>(base) + pixel * 2 * Cs;
    const uint4 h = __ldg(reinterpret_cast<const uint4*>(px + c));
    const uint4 l = __ldg(reinterpret_cast<const uint4*>(px + Cs + c));
    const uint32_t hw[4] = {h.x, h.y, h.z, h.w}, lw[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {          // a bfloat16 is the upper half of a float
      v[2 * i] = __uint_as_float(hw[i] << 16) + __uint_as_float(lw[i] << 16);
      v[2 * i + 1] = __uint_as_float(hw[i] & 0xFFFF0000u) + __uint_as_float(lw[i] & 0xFFFF0000u);
    }
  } else {
    const float* px = static_cast<const float*>(base) + pixel * Cs + c;
    const float4 a = __ldg(reinterpret_cast<const float4*>(px)), b = __ldg(reinterpret_cast<const float4*>(px) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}

template <int FMT>
__device__ __forceinline__ void store8(void* __restrict__ base, size_t pixel, int c, int Cs, const float* v) {
  if (FMT == ACT_SPLIT) {
    __nv_bfloat16* px = static_cast<__nv_bfloat16*>(base) + pixel * 2 * Cs;
    uint32_t hw[4], lw[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat16 h0, l0, h1, l1;
      split_bf16(v[2 * i], h0, l0);
      split_bf16(v[2 * i + 1], h1, l1);
      hw[i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
      lw[i] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
    }
    *reinterpret_cast<uint4*>(px + c) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
    *reinterpret_cast<uint4*>(px + Cs + c) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
  } else {
    float* px = static_cast<float*>(base) + pixel * Cs + c;
    *reinterpret_cast<float4*>(px) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(px + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
}

template <int FMT, int STRIDE>
__global__ void __launch_bounds__(kDwThreads, 4)
depthwise3x3_kernel(ConvGeom g, const LayerJob* __restrict__ jobs) {
  extern __shared__ __align__(16) float dsm[];          // [9][Cs] weights, [Cs] scale, [Cs] bias
  const LayerJob job = jobs[blockIdx.y];
  const int Cs = g.Cs_out;                               // == Cs_in
  float* wsm = dsm;
  float* ssm = dsm + 9 * Cs;
  float* bsm = ssm + Cs;
  const int wrow_bytes = 32 * job.bits / 8;              // K = 9 pads to 32 elements
  for (int i = threadIdx.x; i < 9 * Cs; i += kDwThreads) {
    const int tap = i / Cs, c = i - tap * Cs;
    wsm[i] = c < g.Cout ? load_element(job.w + (size_t)c * wrow_bytes, tap, job.bits) : 0.f;
  }
  for (int c = threadIdx.x; c < Cs; c += kDwThreads) {
    ssm[c] = c < g.Cout ? job.scale[c] : 0.f;
    bsm[c] = c < g.Cout ? job.bias[c] : 0.f;
  }
  __syncthreads();

  constexpr int IN_COLS = (kDwCols - 1) * STRIDE + 3;    // 6 or 9 input columns per thread
  const int octs = Cs / 8;
  const int col_groups = (g.Wo + kDwCols - 1) / kDwCols;
  const int rows_out = g.B * (g.Ho + 2);
  const long long n_items = (long long)rows_out * col_groups * octs;
  for (long long item = (long long)blockIdx.x * kDwThreads + threadIdx.x; item < n_items;
       item += (long long)gridDim.x * kDwThreads) {
    const int oct = (int)(item % octs);
    const long long rest = item / octs;
    const int cg = (int)(rest % col_groups);
    const int jr = (int)(rest / col_groups);             // padded output row (image, y')
    const int b = jr / (g.Ho + 2), oyp = jr - b * (g.Ho + 2);
    const int c = oct * 8, ox0 = cg * kDwCols;
    float acc[kDwCols][8];
#pragma unroll
    for (int x = 0; x < kDwCols; ++x)
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[x][i] = 0.f;
    const bool interior = oyp >= 1 && oyp <= g.Ho;
    if (interior) {
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        const int iy = (oyp - 1) * STRIDE - 1 + r;       // unpadded input row
        if (iy < 0 || iy >= g.H) continue;
        const size_t row_pix = (size_t)(b * (g.H + 2) + iy + 1) * g.W;
        float in[IN_COLS][8];
#pragma unroll
        for (int xx = 0; xx < IN_COLS; ++xx) {
          const int ix = ox0 * STRIDE - 1 + xx;
          if (ix >= 0 && ix < g.W) {
            load8<FMT>(job.in, row_pix + ix, c, Cs, in[xx]);
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) in[xx][i] = 0.f;
          }
        }
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const float4 w0 = *reinterpret_cast<const float4*>(wsm + (r * 3 + t) * Cs + c);
          const float4 w1 = *reinterpret_cast<const float4*>(wsm + (r * 3 + t) * Cs + c + 4);
          const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
          for (int x = 0; x < kDwCols; ++x)
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[x][i] = fmaf(in[x * STRIDE + t][i], wv[i], acc[x][i]);
        }
      }
    }
    const float4 s0 = *reinterpret_cast<const float4*>(ssm + c), s1 = *reinterpret_cast<const float4*>(ssm + c + 4);
    const float4 b0 = *reinterpret_cast<const float4*>(bsm + c), b1 = *reinterpret_cast<const float4*>(bsm + c + 4);
    const float sc[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    const float bi[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
    for (int x = 0; x < kDwCols; ++x) {
      const int ox = ox0 + x;
      if (ox >= g.Wo) break;
      const size_t opix = (size_t)jr * g.Wo + ox;
      float v[8];
      if (interior) {
        float rs[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (job.res) load8<FMT>(job.res, opix, c, Cs, rs);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          v[i] = (c + i < g.Cout) ? apply_act(fmaf(acc[x][i], sc[i], bi[i]) + rs[i], g.act) : 0.f;
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
      }
      store8<FMT>(job.out, opix, c, Cs, v);
    }
  }
}

}  // namespace

aiq_status_t launch_depthwise(const ConvGeom& g, const LayerJob* jobs_dev, int n_jobs,
                              const float* /*net_input*/, double weight_bytes, cudaStream_t s) {
  if (g.stride != 1 && g.stride != 2) return set_error(AIQ_ERR_SHAPE, "depthwise: stride %d is not supported", g.stride);
  const int Cs = g.Cs_out;
  const size_t smem = (size_t)11 * Cs * sizeof(float);
  static int n_sms = 0;
  if (!n_sms) {
    int dev = 0;
    AIQ_CUDA_TRY(cudaGetDevice(&dev));
    AIQ_CUDA_TRY(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev));
  }
  if (smem > 48 * 1024) return set_error(AIQ_ERR_SHAPE, "depthwise: %d channels need %zu bytes of shared memory", g.Cout, smem);
  const long long n_items = (long long)g.B * (g.Ho + 2) * ((g.Wo + kDwCols - 1) / kDwCols) * (Cs / 8);
  long long blocks = (n_items + kDwThreads - 1) / kDwThreads;
  const long long cap = (long long)n_sms * 4;                 // persistent: as many blocks as are resident (4 per SM)
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  dim3 grid((unsigned)blocks, n_jobs);
  LaunchScope scope(AIQ_KERNEL_DEPTHWISE, s, 18.0 * g.B * g.Ho * g.Wo * g.Cout * n_jobs,
                    weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W +
                                                   (double)g.B * g.Ho * g.Wo * g.Cout));
#define AIQ_DW(FMT_, ST_) depthwise3x3_kernel<FMT_, ST_><<<grid, kDwThreads, smem, s>>>(g, jobs_dev)
  if (g.act_format == ACT_SPLIT) { if (g.stride == 1) AIQ_DW(ACT_SPLIT, 1); else AIQ_DW(ACT_SPLIT, 2); }
  else { if (g.stride == 1) AIQ_DW(ACT_F32, 1); else AIQ_DW(ACT_F32, 2); }
#undef AIQ_DW
  AIQ_LAUNCH_CHECK("depthwise3x3");
  return AIQ_OK;
}

}  // namespace aiq
