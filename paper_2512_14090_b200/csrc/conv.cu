// Forward kernels on the float32 multiply-add path: dense convolution as an implicit GEMM,
// global average pool, arg-max + agreement count (the depthwise kernel lives in depthwise.cu).
//
// Every kernel takes an array of LayerJob records and covers all of them in one launch
// (gridDim.z = job), so one launch evaluates a layer for every distinct weight choice a
// group of candidate schemes needs (Section 2.2: each candidate move needs its own
// accuracy measurement).  Weights are read in their packed form and expanded while they
// are staged; the per-channel scale multiplies the finished float32 sum; bias, residual
// add and activation are applied before the single store of the output tensor.
// Activations are read and written in the split bfloat16 format described in common.cuh.
#include "common.cuh"

namespace aiq {

namespace {

__device__ __forceinline__ int rs_group_images_dev(int W) { return (W & 15) == 0 ? 8 : 16; }

constexpr int kConvThreads = 256;
constexpr int BK = 16;

enum { IN_NCHW = 0, IN_SPLIT_VEC = 1, IN_SPLIT_SCALAR = 2 };

__device__ __forceinline__ float4 load_split4(const __nv_bfloat16* __restrict__ pix, int c, int Cs) {
  // 4 consecutive channels of one pixel: hi and lo halves are 8-byte loads
  const uint2 h = __ldg(reinterpret_cast<const uint2*>(pix + c));
  const uint2 l = __ldg(reinterpret_cast<const uint2*>(pix + Cs + c));
  const __nv_bfloat162 h0 = *reinterpret_cast<const __nv_bfloat162*>(&h.x);
  const __nv_bfloat162 h1 = *reinterpret_cast<const __nv_bfloat162*>(&h.y);
  const __nv_bfloat162 l0 = *reinterpret_cast<const __nv_bfloat162*>(&l.x);
  const __nv_bfloat162 l1 = *reinterpret_cast<const __nv_bfloat162*>(&l.y);
  const float2 a = __bfloat1622float2(h0), b = __bfloat1622float2(h1);
  const float2 c0 = __bfloat1622float2(l0), c1 = __bfloat1622float2(l1);
  return make_float4(a.x + c0.x, a.y + c0.y, b.x + c1.x, b.y + c1.y);
}

__device__ __forceinline__ void store_split4(__nv_bfloat16* __restrict__ pix, int c, int Cs, float4 v) {
  __nv_bfloat16 h[4], l[4];
  split_bf16(v.x, h[0], l[0]);
  split_bf16(v.y, h[1], l[1]);
  split_bf16(v.z, h[2], l[2]);
  split_bf16(v.w, h[3], l[3]);
  uint2 hv, lv;
  hv.x = (uint32_t)__bfloat16_as_ushort(h[0]) | ((uint32_t)__bfloat16_as_ushort(h[1]) << 16);
  hv.y = (uint32_t)__bfloat16_as_ushort(h[2]) | ((uint32_t)__bfloat16_as_ushort(h[3]) << 16);
  lv.x = (uint32_t)__bfloat16_as_ushort(l[0]) | ((uint32_t)__bfloat16_as_ushort(l[1]) << 16);
  lv.y = (uint32_t)__bfloat16_as_ushort(l[2]) | ((uint32_t)__bfloat16_as_ushort(l[3]) << 16);
  *reinterpret_cast<uint2*>(pix + c) = hv;
  *reinterpret_cast<uint2*>(pix + Cs + c) = lv;
}

// Element access of an activation tensor in either storage format.  A pixel is 4*Cs bytes
// in both: Cs floats (ACT_F32) or [hi Cs | lo Cs] bfloat16 (ACT_SPLIT).
template <int FMT>
__device__ __forceinline__ float4 act_load4(const void* __restrict__ base, size_t pixel, int c, int Cs) {
  if (FMT == ACT_SPLIT)
    return load_split4(static_cast<const __nv_bfloat16*>(base) + pixel * 2 * Cs, c, Cs);
  return __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(base) + pixel * Cs + c));
}
template <int FMT>
__device__ __forceinline__ float act_load1(const void* __restrict__ base, size_t pixel, int c, int Cs) {
  if (FMT == ACT_SPLIT) {
    const __nv_bfloat16* px = static_cast<const __nv_bfloat16*>(base) + pixel * 2 * Cs;
    return __bfloat162float(px[c]) + __bfloat162float(px[Cs + c]);
  }
  return __ldg(static_cast<const float*>(base) + pixel * Cs + c);
}
template <int FMT>
__device__ __forceinline__ void act_store4(void* __restrict__ base, size_t pixel, int c, int Cs, float4 v) {
  if (FMT == ACT_SPLIT)
    store_split4(static_cast<__nv_bfloat16*>(base) + pixel * 2 * Cs, c, Cs, v);
  else
    *reinterpret_cast<float4*>(static_cast<float*>(base) + pixel * Cs + c) = v;
}

// Implicit GEMM:  out[p][n] = act( s_n * sum_k code[n][k] * patch[p][k] + b_n + res[p][n] )
// p runs over the *padded* output pixel space (image, row 0..Ho+1, column): border rows are
// written as zeros.  k = (tap, channel) with the channel fastest.
// Block tile BM pixels x BN channels, thread tile TM x TN, K consumed in slices of 16
// through a double-buffered shared-memory stage.
//   As[k][p ^ ((k >> 2) << 3)]   (XOR keeps groups of 4 pixels contiguous and makes the
//                                 transposing stores of the vector path conflict-free)
//   Bs[k][n]
template <int BM, int BN, int TM, int TN, int IN_MODE, int FMT>
__global__ void __launch_bounds__(kConvThreads)
conv_igemm_kernel(ConvGeom g, const LayerJob* __restrict__ jobs, const float* __restrict__ net_input) {
  static_assert((BM / TM) * (BN / TN) == kConvThreads, "thread tile must cover the block tile");
  static_assert(TM % 4 == 0 && TN == 4, "thread tile shape");
  constexpr bool VEC = IN_MODE == IN_SPLIT_VEC;
  const LayerJob job = jobs[blockIdx.z];
  const int tid = threadIdx.x;
  const int rows_out = g.Ho + 2;
  const int M = g.B * rows_out * g.Wo;            // padded output pixels
  const int p_base = blockIdx.x * BM;
  const int n_base = blockIdx.y * BN;
  const int Kt = g.ks * g.ks * g.Cin;
  const int n_slices = (Kt + BK - 1) / BK;
  const int taps = g.ks * g.ks;

  __shared__ __align__(16) float As[2][BK][BM];
  __shared__ __align__(16) float Bs[2][BK][BN];

  // ---- A loader state: the pixel(s) a thread fetches never change over the K loop
  constexpr int A_VEC_PER_THREAD = BM * BK / 4 / kConvThreads;   // float4 fetches (VEC)
  constexpr int A_SCL_PER_THREAD = BM * BK / kConvThreads;       // scalar fetches (!VEC)
  constexpr int NPIX = VEC ? A_VEC_PER_THREAD : 1;
  int pix_b[NPIX], pix_iy0[NPIX], pix_ix0[NPIX];
  bool pix_ok[NPIX];
#pragma unroll
  for (int i = 0; i < NPIX; ++i) {
    const int pl = VEC ? (tid >> 2) + i * (kConvThreads >> 2) : (tid % BM);
    const int p = p_base + pl;
    const int pp = p < M ? p : 0;
    const int b = pp / (rows_out * g.Wo);
    const int rem = pp - b * (rows_out * g.Wo);
    const int oyp = rem / g.Wo;                     // padded row 0..Ho+1
    const int ox = rem - oyp * g.Wo;
    pix_ok[i] = p < M && oyp >= 1 && oyp <= g.Ho;
    pix_b[i] = b;
    pix_iy0[i] = (oyp - 1) * g.stride - g.pad;
    pix_ix0[i] = ox * g.stride - g.pad;
  }

  float a_reg[VEC ? A_VEC_PER_THREAD * 4 : A_SCL_PER_THREAD];
  constexpr int B_PER_THREAD = (BK * BN + kConvThreads - 1) / kConvThreads;
  float b_reg[B_PER_THREAD];
  const int wrow_bytes = ((g.K + 31) / 32 * 32) * job.bits / 8;

  auto fetch = [&](int slice) {
    const int k0 = slice * BK;
    if (VEC) {
      const int kq = tid & 3;
      const int kk = k0 + kq * 4;
      const int tap = kk / g.Cin;
      const int c = kk - tap * g.Cin;
      const int r = tap / g.ks;
      const int t = tap - r * g.ks;
#pragma unroll
      for (int i = 0; i < A_VEC_PER_THREAD; ++i) {
        const int iy = pix_iy0[i] + r, ix = pix_ix0[i] + t;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (pix_ok[i] && kk < Kt && iy >= 0 && iy < g.H && ix >= 0 && ix < g.W)
          v = act_load4<FMT>(job.in, (size_t)(pix_b[i] * (g.H + 2) + iy + 1) * g.W + ix, c, g.Cs_in);
        a_reg[4 * i] = v.x; a_reg[4 * i + 1] = v.y; a_reg[4 * i + 2] = v.z; a_reg[4 * i + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < A_SCL_PER_THREAD; ++i) {
        const int kl = tid / BM + i * (kConvThreads / BM);
        const int kk = k0 + kl;
        const int tap = kk / g.Cin;
        const int c = kk - tap * g.Cin;
        const int r = tap / g.ks;
        const int t = tap - r * g.ks;
        const int iy = pix_iy0[0] + r, ix = pix_ix0[0] + t;
        float v = 0.f;
        if (pix_ok[0] && kk < Kt && iy >= 0 && iy < g.H && ix >= 0 && ix < g.W) {
          if (IN_MODE == IN_NCHW) {
            v = __ldg(net_input + (((size_t)pix_b[0] * g.Cin + c) * g.H + iy) * g.W + ix);
          } else {
            v = act_load1<FMT>(job.in, (size_t)(pix_b[0] * (g.H + 2) + iy + 1) * g.W + ix, c, g.Cs_in);
          }
        }
        a_reg[i] = v;
      }
    }
#pragma unroll
    for (int i = 0; i < B_PER_THREAD; ++i) {
      const int idx = tid + i * kConvThreads;
      const int kl = idx / BN, nl = idx - kl * BN;
      const int kk = k0 + kl;
      const int n = n_base + nl;
      float v = 0.f;
      if (idx < BK * BN && kk < Kt && n < g.Cout) {
        const int tap = kk / g.Cin;
        const int c = kk - tap * g.Cin;
        v = load_element(job.w + (size_t)n * wrow_bytes, c * taps + tap, job.bits);
      }
      b_reg[i] = v;
    }
  };

  auto stash = [&](int buf) {
    if (VEC) {
      const int kq = tid & 3;
#pragma unroll
      for (int i = 0; i < A_VEC_PER_THREAD; ++i) {
        const int pl = (tid >> 2) + i * (kConvThreads >> 2);
        const int ps = pl ^ (kq << 3);
#pragma unroll
        for (int j = 0; j < 4; ++j) As[buf][kq * 4 + j][ps] = a_reg[4 * i + j];
      }
    } else {
      const int pl = tid % BM;
#pragma unroll
      for (int i = 0; i < A_SCL_PER_THREAD; ++i) {
        const int kl = tid / BM + i * (kConvThreads / BM);
        As[buf][kl][pl ^ ((kl >> 2) << 3)] = a_reg[i];
      }
    }
#pragma unroll
    for (int i = 0; i < B_PER_THREAD; ++i) {
      const int idx = tid + i * kConvThreads;
      if (idx < BK * BN) (&Bs[buf][0][0])[idx] = b_reg[i];
    }
  };

  // ---- compute
  constexpr int NTX = BN / TN;
  const int tx = tid % NTX;
  const int ty = tid / NTX;
  constexpr int PGROUPS = TM / 4;                    // groups of 4 pixels per thread
  constexpr int PG_STRIDE = BM / PGROUPS;
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  fetch(0);
  stash(0);
  __syncthreads();
  for (int s = 0; s < n_slices; ++s) {
    const int buf = s & 1;
    if (s + 1 < n_slices) fetch(s + 1);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[TM];
#pragma unroll
      for (int pg = 0; pg < PGROUPS; ++pg) {
        const int pl = (pg * PG_STRIDE + ty * 4) ^ ((k >> 2) << 3);
        const float4 v = *reinterpret_cast<const float4*>(&As[buf][k][pl]);
        a[4 * pg] = v.x; a[4 * pg + 1] = v.y; a[4 * pg + 2] = v.z; a[4 * pg + 3] = v.w;
      }
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * TN]);
      const float b[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (s + 1 < n_slices) {
      stash(buf ^ 1);
      __syncthreads();
    }
  }

  // ---- epilogue: scale, bias, residual, activation, split, one store.  Border rows and
  // padded channels are written as zeros.
  const int n = n_base + tx * TN;
  if (n >= g.Cs_out) return;
  float sc[TN], bi[TN];
  bool ch_ok[TN];
#pragma unroll
  for (int j = 0; j < TN; ++j) {
    ch_ok[j] = n + j < g.Cout;
    sc[j] = ch_ok[j] ? job.scale[n + j] : 0.f;
    bi[j] = ch_ok[j] ? job.bias[n + j] : 0.f;
  }
#pragma unroll
  for (int pg = 0; pg < PGROUPS; ++pg) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int p = p_base + pg * PG_STRIDE + ty * 4 + i;
      if (p >= M) continue;
      const int oyp = (p / g.Wo) % rows_out;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (oyp >= 1 && oyp <= g.Ho) {
        float u[TN];
#pragma unroll
        for (int j = 0; j < TN; ++j) u[j] = fmaf(acc[4 * pg + i][j], sc[j], bi[j]);
        if (job.res) {
          const float4 r = act_load4<FMT>(job.res, (size_t)p, n, g.Cs_out);
          u[0] += r.x; u[1] += r.y; u[2] += r.z; u[3] += r.w;
        }
        v = make_float4(ch_ok[0] ? apply_act(u[0], g.act) : 0.f, ch_ok[1] ? apply_act(u[1], g.act) : 0.f,
                        ch_ok[2] ? apply_act(u[2], g.act) : 0.f, ch_ok[3] ? apply_act(u[3], g.act) : 0.f);
      }
      act_store4<FMT>(job.out, (size_t)p, n, g.Cs_out, v);
    }
  }
}

template <int BM, int BN, int TM, int TN>
aiq_status_t launch_conv_tile(const ConvGeom& g, const LayerJob* jobs, int n_jobs, const float* net_input,
                              int in_mode, double weight_bytes, cudaStream_t s) {
  const int M = g.B * (g.Ho + 2) * g.Wo;
  dim3 grid((M + BM - 1) / BM, (g.Cs_out + BN - 1) / BN, n_jobs);
  LaunchScope scope(AIQ_KERNEL_CONV, s,
                    2.0 * g.B * g.Ho * g.Wo * g.Cout * (double)(g.ks * g.ks * g.Cin) * n_jobs,
                    weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W +
                                                   (double)g.B * g.Ho * g.Wo * g.Cout));
#define AIQ_CONV_LAUNCH(MODE)                                                                        \
  do {                                                                                              \
    if (g.act_format == ACT_SPLIT)                                                                  \
      conv_igemm_kernel<BM, BN, TM, TN, MODE, ACT_SPLIT><<<grid, kConvThreads, 0, s>>>(g, jobs, net_input); \
    else                                                                                            \
      conv_igemm_kernel<BM, BN, TM, TN, MODE, ACT_F32><<<grid, kConvThreads, 0, s>>>(g, jobs, net_input);   \
  } while (0)
  if (in_mode == IN_SPLIT_VEC) AIQ_CONV_LAUNCH(IN_SPLIT_VEC);
  else if (in_mode == IN_SPLIT_SCALAR) AIQ_CONV_LAUNCH(IN_SPLIT_SCALAR);
  else AIQ_CONV_LAUNCH(IN_NCHW);
#undef AIQ_CONV_LAUNCH
  AIQ_LAUNCH_CHECK("conv_igemm");
  return AIQ_OK;
}

// ---------------------------------------------------------------------------------------
// Stem convolution: 3x3, pad 1, a few input channels read straight from the float32 NCHW
// network input.  K = 9 * Cin = 27 is too short for the tiled GEMM above (one 16-deep slice
// and a half-empty one, two block barriers per 16 multiply-adds per thread), so a thread
// owns one padded output pixel and all COUT channels: its 27 inputs sit in registers, the
// expanded weights [k][COUT] in shared memory (read as warp-wide broadcasts), and the result
// leaves as 16-byte stores.  Border rows are written as zeros.
// ---------------------------------------------------------------------------------------
constexpr int kStemThreads = 256;

template <int COUT, int FMT>
__global__ void __launch_bounds__(kStemThreads)
conv_stem_kernel(ConvGeom g, const LayerJob* __restrict__ jobs, const float* __restrict__ net_input) {
  extern __shared__ __align__(16) float stem_sm[];            // [Kt][COUT] weights, [COUT] scale, [COUT] bias
  const LayerJob job = jobs[blockIdx.z];
  const int Kt = 9 * g.Cin;
  float* wsm = stem_sm;
  float* ssm = wsm + Kt * COUT;
  float* bsm = ssm + COUT;
  const int wrow_bytes = ((g.K + 31) / 32 * 32) * job.bits / 8;
  for (int i = threadIdx.x; i < Kt * COUT; i += kStemThreads) {
    const int k = i / COUT, n = i - k * COUT;                // k = (tap, channel), channel fastest
    const int tap = k / g.Cin, c = k - tap * g.Cin;
    wsm[i] = n < g.Cout ? load_element(job.w + (size_t)n * wrow_bytes, c * 9 + tap, job.bits) : 0.f;
  }
  for (int n = threadIdx.x; n < COUT; n += kStemThreads) {
    ssm[n] = n < g.Cout ? job.scale[n] : 0.f;
    bsm[n] = n < g.Cout ? job.bias[n] : 0.f;
  }
  __syncthreads();

  const int rows_out = g.Ho + 2;
  const long long M = (long long)g.B * rows_out * g.Wo;      // padded output pixels
  const long long p = (long long)blockIdx.x * kStemThreads + threadIdx.x;
  if (p >= M) return;
  const int b = (int)(p / (rows_out * g.Wo));
  const int rem = (int)(p - (long long)b * rows_out * g.Wo);
  const int oyp = rem / g.Wo, ox = rem - oyp * g.Wo;
  float acc[COUT];
#pragma unroll
  for (int n = 0; n < COUT; ++n) acc[n] = 0.f;
  const bool interior = oyp >= 1 && oyp <= g.Ho;
  if (interior) {
    const int iy0 = (oyp - 1) * g.stride - 1, ix0 = ox * g.stride - 1;
    for (int c = 0; c < g.Cin; ++c) {
      const float* plane = net_input + ((size_t)b * g.Cin + c) * g.H * g.W;
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        const int iy = iy0 + r;
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const int ix = ix0 + t;
          const float xv = (iy >= 0 && iy < g.H && ix >= 0 && ix < g.W) ? __ldg(plane + (size_t)iy * g.W + ix) : 0.f;
          const float* wk = wsm + ((r * 3 + t) * g.Cin + c) * COUT;
#pragma unroll
          for (int n = 0; n < COUT; n += 4) {
            const float4 wv = *reinterpret_cast<const float4*>(wk + n);
            acc[n] = fmaf(xv, wv.x, acc[n]);
            acc[n + 1] = fmaf(xv, wv.y, acc[n + 1]);
            acc[n + 2] = fmaf(xv, wv.z, acc[n + 2]);
            acc[n + 3] = fmaf(xv, wv.w, acc[n + 3]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int n = 0; n < COUT; n += 4) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (interior) {
      v.x = n < g.Cout ? apply_act(fmaf(acc[n], ssm[n], bsm[n]), g.act) : 0.f;
      v.y = n + 1 < g.Cout ? apply_act(fmaf(acc[n + 1], ssm[n + 1], bsm[n + 1]), g.act) : 0.f;
      v.z = n + 2 < g.Cout ? apply_act(fmaf(acc[n + 2], ssm[n + 2], bsm[n + 2]), g.act) : 0.f;
      v.w = n + 3 < g.Cout ? apply_act(fmaf(acc[n + 3], ssm[n + 3], bsm[n + 3]), g.act) : 0.f;
    }
    act_store4<FMT>(job.out, (size_t)p, n, g.Cs_out, v);
  }
}

// The same stem writing the image-interleaved ACT_RS layout: consecutive threads own consecutive
// images of a group at one output position, so the 16-byte plane stores of a warp are contiguous.
template <int COUT>
__global__ void __launch_bounds__(kStemThreads)
conv_stem_rs_kernel(ConvGeom g, const LayerJob* __restrict__ jobs, const float* __restrict__ net_input) {
  extern __shared__ __align__(16) float stem_sm[];            // [Kt][COUT] weights, [COUT] scale, [COUT] bias
  const LayerJob job = jobs[blockIdx.z];
  const int Kt = 9 * g.Cin;
  float* wsm = stem_sm;
  float* ssm = wsm + Kt * COUT;
  float* bsm = ssm + COUT;
  const int wrow_bytes = ((g.K + 31) / 32 * 32) * job.bits / 8;
  for (int i = threadIdx.x; i < Kt * COUT; i += kStemThreads) {
    const int k = i / COUT, n = i - k * COUT;
    const int tap = k / g.Cin, c = k - tap * g.Cin;
    wsm[i] = load_element(job.w + (size_t)n * wrow_bytes, c * 9 + tap, job.bits);
  }
  for (int n = threadIdx.x; n < COUT; n += kStemThreads) { ssm[n] = job.scale[n]; bsm[n] = job.bias[n]; }
  __syncthreads();

  const int G = rs_group_images_dev(g.Wo);
  const int Bp = (g.B + 15) / 16 * 16;
  const long long M = (long long)Bp * g.Ho * g.Wo;
  const long long p = (long long)blockIdx.x * kStemThreads + threadIdx.x;
  if (p >= M) return;
  const int img = (int)(p % G);
  const int ox = (int)((p / G) % g.Wo);
  const int oy = (int)((p / ((long long)G * g.Wo)) % g.Ho);
  const int grp = (int)(p / ((long long)G * g.Wo * g.Ho));
  const int b = grp * G + img;
  float acc[COUT];
#pragma unroll
  for (int n = 0; n < COUT; ++n) acc[n] = 0.f;
  if (b < g.B) {                                               // padding images of the last group see a zero input
    const int iy0 = oy * g.stride - 1, ix0 = ox * g.stride - 1;
    for (int c = 0; c < g.Cin; ++c) {
      const float* plane = net_input + ((size_t)b * g.Cin + c) * g.H * g.W;
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        const int iy = iy0 + r;
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const int ix = ix0 + t;
          const float xv = (iy >= 0 && iy < g.H && ix >= 0 && ix < g.W) ? __ldg(plane + (size_t)iy * g.W + ix) : 0.f;
          const float* wk = wsm + ((r * 3 + t) * g.Cin + c) * COUT;
#pragma unroll
          for (int n = 0; n < COUT; n += 4) {
            const float4 wv = *reinterpret_cast<const float4*>(wk + n);
            acc[n] = fmaf(xv, wv.x, acc[n]);
            acc[n + 1] = fmaf(xv, wv.y, acc[n + 1]);
            acc[n + 2] = fmaf(xv, wv.z, acc[n + 2]);
            acc[n + 3] = fmaf(xv, wv.w, acc[n + 3]);
          }
        }
      }
    }
  }
  const size_t plane_bytes = (size_t)G * 16;
  uint8_t* dst = static_cast<uint8_t*>(job.out) +
                 ((((size_t)grp * g.Ho + oy) * g.Wo + ox) * (COUT / 4)) * plane_bytes + (size_t)img * 16;
#pragma unroll
  for (int n = 0; n < COUT; n += 8) {
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      const float u0 = apply_act(fmaf(acc[n + e], ssm[n + e], bsm[n + e]), g.act);
      const float u1 = apply_act(fmaf(acc[n + e + 1], ssm[n + e + 1], bsm[n + e + 1]), g.act);
      __nv_bfloat16 h0, l0, h1, l1;
      split_bf16(u0, h0, l0);
      split_bf16(u1, h1, l1);
      hi[e >> 1] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
      lo[e >> 1] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
    }
    *reinterpret_cast<uint4*>(dst + (size_t)(n / 8) * plane_bytes) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(dst + (size_t)(COUT / 8 + n / 8) * plane_bytes) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
}

// Stride-1 stem for ACT_RS with the input staged in shared memory.  A block owns kStemRows output
// rows of one group of G images: the kStemRows + 2 input rows of every channel and image arrive
// by coalesced 16-byte loads (the kernel above gathers 27 scattered words per thread) and are
// held as [channel][row][image][column + 1 zero column on both sides], 4 words of slack per
// row so that the 8 images x 4 columns of a warp read 32 different banks.  A thread owns one
// (image, column) and walks down the rows.  Same arithmetic order as the gathering kernel.
constexpr int kStemRows = 4;

template <int COUT>
__global__ void __launch_bounds__(256)
conv_stem_rs_rows_kernel(ConvGeom g, const LayerJob* __restrict__ jobs, const float* __restrict__ net_input) {
  extern __shared__ __align__(16) float stem_sm[];            // weights, scale, bias, input tile
  const LayerJob job = jobs[blockIdx.z];
  const int Kt = 9 * g.Cin;
  float* wsm = stem_sm;
  float* ssm = wsm + Kt * COUT;
  float* bsm = ssm + COUT;
  float* tile = bsm + COUT;
  const int G = rs_group_images_dev(g.Wo);
  const int RS = g.W + 4;                                      // words of a tile row
  const int n_threads = blockDim.x;
  const int wrow_bytes = ((g.K + 31) / 32 * 32) * job.bits / 8;
  for (int i = threadIdx.x; i < Kt * COUT; i += n_threads) {
    const int k = i / COUT, n = i - k * COUT;
    const int tap = k / g.Cin, c = k - tap * g.Cin;
    wsm[i] = load_element(job.w + (size_t)n * wrow_bytes, c * 9 + tap, job.bits);
  }
  for (int n = threadIdx.x; n < COUT; n += n_threads) { ssm[n] = job.scale[n]; bsm[n] = job.bias[n]; }
  const int row_blocks = g.Ho / kStemRows;
  const int grp = blockIdx.x / row_blocks, oy0 = (blockIdx.x - grp * row_blocks) * kStemRows;
  // input rows oy0 - 1 .. oy0 + kStemRows of every channel and image of the group
  const int W4 = g.W / 4;
  const int n_quads = g.Cin * (kStemRows + 2) * G * W4;
  for (int i = threadIdx.x; i < n_quads; i += n_threads) {
    const int x4 = i % W4, img = (i / W4) % G, r = (i / (W4 * G)) % (kStemRows + 2), c = i / (W4 * G * (kStemRows + 2));
    const int iy = oy0 - 1 + r, b = grp * G + img;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (iy >= 0 && iy < g.H && b < g.B)
      v = __ldg(reinterpret_cast<const float4*>(net_input + (((size_t)b * g.Cin + c) * g.H + iy) * g.W) + x4);
    float* dst = tile + ((size_t)(c * (kStemRows + 2) + r) * G + img) * RS + 1 + 4 * x4;
    dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
  }
  for (int i = threadIdx.x; i < g.Cin * (kStemRows + 2) * G * 2; i += n_threads)    // the zero columns
    tile[(size_t)(i >> 1) * RS + ((i & 1) ? g.W + 1 : 0)] = 0.f;
  __syncthreads();

  const int img = threadIdx.x % G, ox = threadIdx.x / G;
  const size_t plane_bytes = (size_t)G * 16;
  for (int ry = 0; ry < kStemRows; ++ry) {
    float acc[COUT];
#pragma unroll
    for (int n = 0; n < COUT; ++n) acc[n] = 0.f;
    for (int c = 0; c < g.Cin; ++c) {
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        const float* row = tile + ((size_t)(c * (kStemRows + 2) + ry + r) * G + img) * RS + ox;
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const float xv = row[t];
          const float* wk = wsm + ((r * 3 + t) * g.Cin + c) * COUT;
#pragma unroll
          for (int n = 0; n < COUT; n += 4) {
            const float4 wv = *reinterpret_cast<const float4*>(wk + n);
            acc[n] = fmaf(xv, wv.x, acc[n]);
            acc[n + 1] = fmaf(xv, wv.y, acc[n + 1]);
            acc[n + 2] = fmaf(xv, wv.z, acc[n + 2]);
            acc[n + 3] = fmaf(xv, wv.w, acc[n + 3]);
          }
        }
      }
    }
    uint8_t* dst = static_cast<uint8_t*>(job.out) +
                   ((((size_t)grp * g.Ho + oy0 + ry) * g.Wo + ox) * (COUT / 4)) * plane_bytes + (size_t)img * 16;
#pragma unroll
    for (int n = 0; n < COUT; n += 8) {
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 8; e += 2) {
        const float u0 = apply_act(fmaf(acc[n + e], ssm[n + e], bsm[n + e]), g.act);
        const float u1 = apply_act(fmaf(acc[n + e + 1], ssm[n + e + 1], bsm[n + e + 1]), g.act);
        __nv_bfloat16 h0, l0, h1, l1;
        split_bf16(u0, h0, l0);
        split_bf16(u1, h1, l1);
        hi[e >> 1] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
        lo[e >> 1] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
      }
      *reinterpret_cast<uint4*>(dst + (size_t)(n / 8) * plane_bytes) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *reinterpret_cast<uint4*>(dst + (size_t)(COUT / 8 + n / 8) * plane_bytes) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
  }
}

template <int COUT>
aiq_status_t launch_stem(const ConvGeom& g, const LayerJob* jobs, int n_jobs, const float* net_input,
                         double weight_bytes, cudaStream_t s) {
  const long long M = g.act_format == ACT_RS ? (long long)rs_padded_batch(g.B) * g.Ho * g.Wo
                                             : (long long)g.B * (g.Ho + 2) * g.Wo;
  dim3 grid((unsigned)((M + kStemThreads - 1) / kStemThreads), 1, n_jobs);
  const size_t smem = (size_t)(9 * g.Cin * COUT + 2 * COUT) * sizeof(float);
  LaunchScope scope(AIQ_KERNEL_CONV, s,
                    2.0 * g.B * g.Ho * g.Wo * g.Cout * (double)(9 * g.Cin) * n_jobs,
                    weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W +
                                                   (double)g.B * g.Ho * g.Wo * g.Cout));
  const int G = rs_group_images(g.Wo);
  const size_t tile_bytes = (size_t)g.Cin * (kStemRows + 2) * G * (g.W + 4) * sizeof(float);
  if (g.act_format == ACT_RS && g.stride == 1 && g.W == g.Wo && g.H == g.Ho && g.W % 4 == 0 && g.Ho % kStemRows == 0 &&
      G * g.Wo <= 256 && (G * g.Wo) % 32 == 0 && smem + tile_bytes <= 100 * 1024) {
    AIQ_ENSURE_DYNAMIC_SMEM((conv_stem_rs_rows_kernel<COUT>), 100 * 1024);
    const dim3 rgrid((unsigned)(rs_padded_batch(g.B) / G * (g.Ho / kStemRows)), 1, n_jobs);
    conv_stem_rs_rows_kernel<COUT><<<rgrid, G * g.Wo, smem + tile_bytes, s>>>(g, jobs, net_input);
  } else if (g.act_format == ACT_RS)
    conv_stem_rs_kernel<COUT><<<grid, kStemThreads, smem, s>>>(g, jobs, net_input);
  else if (g.act_format == ACT_SPLIT)
    conv_stem_kernel<COUT, ACT_SPLIT><<<grid, kStemThreads, smem, s>>>(g, jobs, net_input);
  else
    conv_stem_kernel<COUT, ACT_F32><<<grid, kStemThreads, smem, s>>>(g, jobs, net_input);
  AIQ_LAUNCH_CHECK("conv_stem");
  return AIQ_OK;
}

// ---------------------------------------------------------------------------------------
// Global average pool over the interior of a split tensor: pooled[b][c] float32
// ---------------------------------------------------------------------------------------
// One block per (image, job).  A thread owns 4 consecutive channels and every PL-th pixel
// (8-byte loads of the hi and the lo half); the PL partial sums of a channel meet in shared
// memory in a fixed order, so the result does not depend on timing.
constexpr int kPoolThreads = 256;

template <int FMT>
__global__ void __launch_bounds__(kPoolThreads)
avgpool_kernel(const LayerJob* __restrict__ jobs, int H, int W, int C, int Cs) {
  __shared__ float4 s_sum[kPoolThreads];
  const LayerJob job = jobs[blockIdx.z];
  const int b = blockIdx.x;
  const float inv = 1.0f / (float)(H * W);
  float* __restrict__ out = static_cast<float*>(job.out);
  const size_t p0 = ((size_t)b * (H + 2) + 1) * W;       // first interior pixel of image b
  const int quads = Cs / 4;                               // groups of 4 channels
  const int qb = quads < kPoolThreads ? quads : kPoolThreads;   // quads handled per pass
  const int PL = kPoolThreads / qb;                       // pixel lanes
  const int ql = threadIdx.x % qb, pl = threadIdx.x / qb;
  for (int q0 = 0; q0 < quads; q0 += qb) {
    const int q = q0 + ql;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q < quads && pl < PL)
      for (int i = pl; i < H * W; i += PL) {
        const float4 v = act_load4<FMT>(job.in, p0 + i, 4 * q, Cs);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
    s_sum[threadIdx.x] = acc;
    __syncthreads();
    if (pl == 0 && q < quads) {
      float4 t = s_sum[ql];
      for (int j = 1; j < PL; ++j) {
        const float4 u = s_sum[j * qb + ql];
        t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
      }
      const float r[4] = {t.x * inv, t.y * inv, t.z * inv, t.w * inv};
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (4 * q + j < C) out[(size_t)b * C + 4 * q + j] = r[j];
    }
    __syncthreads();
  }
}

// Global average pool of an ACT_RS tensor.  One block per (group, job); a thread owns 8
// consecutive channels of one image and every PL-th position; partial sums meet in a fixed order.
__global__ void __launch_bounds__(kPoolThreads)
avgpool_rs_kernel(const LayerJob* __restrict__ jobs, int B, int H, int W, int C) {
  __shared__ float s_sum[kPoolThreads][8];
  const LayerJob job = jobs[blockIdx.z];
  const int G = rs_group_images_dev(W);
  const int grp = blockIdx.x;
  const int octets = C / 8;
  const int units = octets * G;                           // (image, channel octet) pairs: at most 128
  const int PL = kPoolThreads / units;
  const int unit = threadIdx.x % units, pl = threadIdx.x / units;
  const int img = unit % G, oc = unit / G;
  const size_t plane_bytes = (size_t)G * 16;
  const size_t px_bytes = (size_t)(C / 4) * plane_bytes;
  const uint8_t* base = static_cast<const uint8_t*>(job.in) + (size_t)grp * H * W * px_bytes + (size_t)img * 16;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (pl < PL)
    for (int i = pl; i < H * W; i += PL) {
      const uint4 hv = __ldg(reinterpret_cast<const uint4*>(base + (size_t)i * px_bytes + (size_t)oc * plane_bytes));
      const uint4 lv = __ldg(reinterpret_cast<const uint4*>(base + (size_t)i * px_bytes + (size_t)(octets + oc) * plane_bytes));
      const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w}, lw[4] = {lv.x, lv.y, lv.z, lv.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        acc[2 * j] += __uint_as_float(hw[j] << 16) + __uint_as_float(lw[j] << 16);
        acc[2 * j + 1] += __uint_as_float(hw[j] & 0xFFFF0000u) + __uint_as_float(lw[j] & 0xFFFF0000u);
      }
    }
#pragma unroll
  for (int j = 0; j < 8; ++j) s_sum[threadIdx.x][j] = acc[j];
  __syncthreads();
  const int b = grp * G + img;
  if (pl == 0 && b < B) {
    float* out = static_cast<float*>(job.out) + (size_t)b * C + oc * 8;
    const float inv = 1.0f / (float)(H * W);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float t = s_sum[unit][j];
      for (int k = 1; k < PL; ++k) t += s_sum[k * units + unit][j];
      out[j] = t * inv;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Arg-max (lowest index on ties) and agreement count.  One warp per image.
// ---------------------------------------------------------------------------------------
__global__ void argmax_count_kernel(const LayerJob* __restrict__ jobs, int B, int n_classes,
                                    const int32_t* __restrict__ labels, int32_t* __restrict__ counts,
                                    int32_t* __restrict__ preds, long long preds_stride, long long img0) {
  const LayerJob job = jobs[blockIdx.z];
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int correct = 0;
  if (b < B) {
    const float* lg = static_cast<const float*>(job.in) + (size_t)b * n_classes;
    float best = -INFINITY;
    int arg = 0x7fffffff;
    for (int j = lane; j < n_classes; j += 32) {
      const float v = lg[j];
      if (v > best || (v == best && j < arg) || arg == 0x7fffffff) { best = v; arg = j; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
      if (oa != 0x7fffffff && (arg == 0x7fffffff || ob > best || (ob == best && oa < arg))) {
        best = ob;
        arg = oa;
      }
    }
    if (lane == 0) {
      if (preds) preds[(long long)job.label_slot * preds_stride + img0 + b] = arg;
      if (labels && labels[img0 + b] == arg) correct = 1;
    }
  }
  if (counts) {
    __shared__ int s_cnt;
    if (threadIdx.x == 0) s_cnt = 0;
    __syncthreads();
    if (correct) atomicAdd(&s_cnt, 1);
    __syncthreads();
    if (threadIdx.x == 0 && s_cnt) atomicAdd(&counts[job.label_slot], s_cnt);
  }
}

}  // namespace

aiq_status_t launch_conv(const ConvGeom& g, const LayerJob* jobs_dev, int n_jobs, const float* net_input,
                         double weight_bytes, cudaStream_t s) {
  if (g.in_is_nchw && g.ks == 3 && g.pad == 1 && g.Cin <= 4 && (g.stride == 1 || g.stride == 2)) {
    if (g.Cs_out == 16) return launch_stem<16>(g, jobs_dev, n_jobs, net_input, weight_bytes, s);
    if (g.Cs_out == 32) return launch_stem<32>(g, jobs_dev, n_jobs, net_input, weight_bytes, s);
    if (g.Cs_out == 64) return launch_stem<64>(g, jobs_dev, n_jobs, net_input, weight_bytes, s);
  }
  const int in_mode = g.in_is_nchw ? IN_NCHW : ((g.Cin % 4 == 0) ? IN_SPLIT_VEC : IN_SPLIT_SCALAR);
  auto waste = [&](int bn) { return (g.Cs_out + bn - 1) / bn * bn - g.Cs_out; };
  int bn = 64;
  if (waste(32) < waste(bn)) bn = 32;
  if (waste(16) < waste(bn)) bn = 16;
  if (bn == 64) return launch_conv_tile<128, 64, 8, 4>(g, jobs_dev, n_jobs, net_input, in_mode, weight_bytes, s);
  if (bn == 32) return launch_conv_tile<128, 32, 4, 4>(g, jobs_dev, n_jobs, net_input, in_mode, weight_bytes, s);
  return launch_conv_tile<256, 16, 4, 4>(g, jobs_dev, n_jobs, net_input, in_mode, weight_bytes, s);
}

aiq_status_t launch_avgpool(const LayerJob* jobs_dev, int n_jobs, int B, int H, int W, int C, int act_format,
                            cudaStream_t s) {
  const int threads = kPoolThreads;
  LaunchScope scope(AIQ_KERNEL_POOL, s, (double)n_jobs * B * H * W * C,
                    4.0 * n_jobs * B * ((double)H * W * C + C));
  if (act_format == ACT_RS)
    avgpool_rs_kernel<<<dim3(rs_padded_batch(B) / rs_group_images(W), 1, n_jobs), threads, 0, s>>>(jobs_dev, B, H, W, C);
  else if (act_format == ACT_SPLIT)
    avgpool_kernel<ACT_SPLIT><<<dim3(B, 1, n_jobs), threads, 0, s>>>(jobs_dev, H, W, C, padded_channels(C));
  else
    avgpool_kernel<ACT_F32><<<dim3(B, 1, n_jobs), threads, 0, s>>>(jobs_dev, H, W, C, padded_channels(C));
  AIQ_LAUNCH_CHECK("avgpool");
  return AIQ_OK;
}

aiq_status_t launch_argmax_count(const LayerJob* jobs_dev, int n_jobs, int B, int n_classes,
                                 const int32_t* labels, int32_t* counts, int32_t* preds,
                                 long long preds_stride, long long img0, cudaStream_t s) {
  const int warps = 8;
  LaunchScope scope(AIQ_KERNEL_ARGMAX, s, 0.0, 4.0 * n_jobs * B * ((double)n_classes + 2));
  argmax_count_kernel<<<dim3((B + warps - 1) / warps, 1, n_jobs), warps * 32, 0, s>>>(
      jobs_dev, B, n_classes, labels, counts, preds, preds_stride, img0);
  AIQ_LAUNCH_CHECK("argmax_count");
  return AIQ_OK;
}

}  // namespace aiq
