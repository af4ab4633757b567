// Forward kernels on the float32 multiply-add path: dense convolution as an implicit GEMM,
// depthwise 3x3, global average pool, arg-max + agreement count.
//
// Every kernel takes an array of LayerJob records and covers all of them in one launch
// (gridDim.z = job), so one launch evaluates a layer for every distinct weight choice a
// group of candidate schemes needs (Section 2.2: each candidate move needs its own
// accuracy measurement).  Weights are read in their packed form and expanded while they
// are staged; the per-channel scale multiplies the finished float32 sum; bias, residual
// add and activation are applied before the single store of the output tensor.
#include "common.cuh"

namespace aiq {

namespace {

constexpr int kConvThreads = 256;
constexpr int BK = 16;

// Implicit GEMM:  out[p][n] = act( s_n * sum_k code[n][k] * patch[p][k] + b_n + res[p][n] )
// p = (image, oy, ox) flattened, k = (tap, channel) with the channel fastest.
// Block tile BM pixels x BN channels, thread tile TM x TN, K consumed in slices of 16
// through a double-buffered shared-memory stage.
//   As[k][p ^ ((k >> 2) << 3)]   (XOR keeps groups of 4 pixels contiguous and makes the
//                                 transposing stores of the vector path conflict-free)
//   Bs[k][n]
template <int BM, int BN, int TM, int TN, bool VEC>
__global__ void __launch_bounds__(kConvThreads)
conv_igemm_kernel(ConvGeom g, const LayerJob* __restrict__ jobs, const float* __restrict__ net_input) {
  static_assert((BM / TM) * (BN / TN) == kConvThreads, "thread tile must cover the block tile");
  static_assert(TM % 4 == 0 && TN == 4, "thread tile shape");
  const LayerJob job = jobs[blockIdx.z];
  const float* __restrict__ in = job.in ? job.in : net_input;
  const int tid = threadIdx.x;
  const int M = g.B * g.Ho * g.Wo;
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
  long long pix_off[NPIX];
  int pix_iy0[NPIX], pix_ix0[NPIX];
  bool pix_ok[NPIX];
#pragma unroll
  for (int i = 0; i < NPIX; ++i) {
    const int pl = VEC ? (tid >> 2) + i * (kConvThreads >> 2) : (tid % BM);
    const int p = p_base + pl;
    pix_ok[i] = p < M;
    const int pp = pix_ok[i] ? p : 0;
    const int b = pp / (g.Ho * g.Wo);
    const int rem = pp - b * (g.Ho * g.Wo);
    const int oy = rem / g.Wo;
    const int ox = rem - oy * g.Wo;
    pix_iy0[i] = oy * g.stride - g.pad;
    pix_ix0[i] = ox * g.stride - g.pad;
    pix_off[i] = (long long)b * g.in_sb;
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
          v = __ldg(reinterpret_cast<const float4*>(in + pix_off[i] + (long long)iy * g.in_sy +
                                                    (long long)ix * g.in_sx + c));
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
        if (pix_ok[0] && kk < Kt && iy >= 0 && iy < g.H && ix >= 0 && ix < g.W)
          v = __ldg(in + pix_off[0] + (long long)iy * g.in_sy + (long long)ix * g.in_sx +
                    (long long)c * g.in_sc);
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

  // ---- epilogue: scale, bias, residual, activation, one store
  const int n = n_base + tx * TN;
  if (n >= g.Cout) return;
  float sc[TN], bi[TN];
#pragma unroll
  for (int j = 0; j < TN; ++j) {
    const bool ok = n + j < g.Cout;
    sc[j] = ok ? job.scale[n + j] : 0.f;
    bi[j] = ok ? job.bias[n + j] : 0.f;
  }
  const bool full = (n + TN <= g.Cout) && ((g.Cout & 3) == 0);
#pragma unroll
  for (int pg = 0; pg < PGROUPS; ++pg) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int p = p_base + pg * PG_STRIDE + ty * 4 + i;
      if (p >= M) continue;
      float v[TN];
#pragma unroll
      for (int j = 0; j < TN; ++j) v[j] = fmaf(acc[4 * pg + i][j], sc[j], bi[j]);
      float* o = job.out + (size_t)p * g.Cout + n;
      if (full) {
        if (job.res) {
          const float4 r = *reinterpret_cast<const float4*>(job.res + (size_t)p * g.Cout + n);
          v[0] += r.x; v[1] += r.y; v[2] += r.z; v[3] += r.w;
        }
        *reinterpret_cast<float4*>(o) = make_float4(apply_act(v[0], g.act), apply_act(v[1], g.act),
                                                    apply_act(v[2], g.act), apply_act(v[3], g.act));
      } else {
#pragma unroll
        for (int j = 0; j < TN; ++j) {
          if (n + j >= g.Cout) break;
          float u = v[j];
          if (job.res) u += job.res[(size_t)p * g.Cout + n + j];
          o[j] = apply_act(u, g.act);
        }
      }
    }
  }
}

template <int BM, int BN, int TM, int TN>
aiq_status_t launch_conv_tile(const ConvGeom& g, const LayerJob* jobs, int n_jobs, const float* net_input,
                              bool vec, double weight_bytes, cudaStream_t s) {
  const int M = g.B * g.Ho * g.Wo;
  dim3 grid((M + BM - 1) / BM, (g.Cout + BN - 1) / BN, n_jobs);
  LaunchScope scope(AIQ_KERNEL_CONV, s, 2.0 * M * g.Cout * (double)(g.ks * g.ks * g.Cin) * n_jobs,
                    weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W + (double)M * g.Cout));
  if (vec)
    conv_igemm_kernel<BM, BN, TM, TN, true><<<grid, kConvThreads, 0, s>>>(g, jobs, net_input);
  else
    conv_igemm_kernel<BM, BN, TM, TN, false><<<grid, kConvThreads, 0, s>>>(g, jobs, net_input);
  AIQ_LAUNCH_CHECK("conv_igemm");
  return AIQ_OK;
}

// ---------------------------------------------------------------------------------------
// Depthwise 3x3 (NHWC).  A block owns a slice of up to 128 channels and a tile of pixels;
// a lane owns 4 consecutive channels, so a warp reads 512 contiguous bytes per tap.
// ---------------------------------------------------------------------------------------
constexpr int kDwPixPerBlock = 64;

__global__ void __launch_bounds__(256)
depthwise3x3_kernel(ConvGeom g, const LayerJob* __restrict__ jobs) {
  const LayerJob job = jobs[blockIdx.z];
  const int c_base = blockIdx.y * 128;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __shared__ __align__(16) float wsm[9][128];
  __shared__ __align__(16) float ssm[128], bsm[128];
  const int wrow_bytes = 32 * job.bits / 8;            // K = 9 pads to 32 elements
  for (int i = threadIdx.x; i < 9 * 128; i += blockDim.x) {
    const int tap = i / 128, cl = i - tap * 128;
    const int c = c_base + cl;
    wsm[tap][cl] = c < g.Cout ? load_element(job.w + (size_t)c * wrow_bytes, tap, job.bits) : 0.f;
  }
  for (int i = threadIdx.x; i < 128; i += blockDim.x) {
    const int c = c_base + i;
    ssm[i] = c < g.Cout ? job.scale[c] : 0.f;
    bsm[i] = c < g.Cout ? job.bias[c] : 0.f;
  }
  __syncthreads();
  const int c = c_base + lane * 4;
  if (c >= g.Cout) return;
  const int M = g.B * g.Ho * g.Wo;
  const int C = g.Cout;
  const float4 sc = *reinterpret_cast<const float4*>(&ssm[lane * 4]);
  const float4 bi = *reinterpret_cast<const float4*>(&bsm[lane * 4]);
  for (int pi = warp; pi < kDwPixPerBlock; pi += 8) {
    const int p = blockIdx.x * kDwPixPerBlock + pi;
    if (p >= M) break;
    const int b = p / (g.Ho * g.Wo);
    const int rem = p - b * (g.Ho * g.Wo);
    const int oy = rem / g.Wo, ox = rem - (rem / g.Wo) * g.Wo;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const int iy = oy * g.stride - 1 + r;
      if (iy < 0 || iy >= g.H) continue;
#pragma unroll
      for (int t = 0; t < 3; ++t) {
        const int ix = ox * g.stride - 1 + t;
        if (ix < 0 || ix >= g.W) continue;
        const float4 xv = __ldg(reinterpret_cast<const float4*>(
            job.in + ((size_t)(b * g.H + iy) * g.W + ix) * C + c));
        const float4 wv = *reinterpret_cast<const float4*>(&wsm[r * 3 + t][lane * 4]);
        acc.x = fmaf(xv.x, wv.x, acc.x);
        acc.y = fmaf(xv.y, wv.y, acc.y);
        acc.z = fmaf(xv.z, wv.z, acc.z);
        acc.w = fmaf(xv.w, wv.w, acc.w);
      }
    }
    float4 v = make_float4(fmaf(acc.x, sc.x, bi.x), fmaf(acc.y, sc.y, bi.y), fmaf(acc.z, sc.z, bi.z),
                           fmaf(acc.w, sc.w, bi.w));
    if (job.res) {
      const float4 rr = *reinterpret_cast<const float4*>(job.res + (size_t)p * C + c);
      v.x += rr.x; v.y += rr.y; v.z += rr.z; v.w += rr.w;
    }
    *reinterpret_cast<float4*>(job.out + (size_t)p * C + c) =
        make_float4(apply_act(v.x, g.act), apply_act(v.y, g.act), apply_act(v.z, g.act),
                    apply_act(v.w, g.act));
  }
}

// ---------------------------------------------------------------------------------------
// Global average pool: pooled[b][c] = (1/HW) * sum_hw in[b][hw][c]
// ---------------------------------------------------------------------------------------
__global__ void avgpool_kernel(const LayerJob* __restrict__ jobs, int HW, int C) {
  const LayerJob job = jobs[blockIdx.z];
  const int b = blockIdx.x;
  const float inv = 1.0f / (float)HW;
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    const float* p = job.in + (size_t)b * HW * C + c;
    float s = 0.f;
    for (int i = 0; i < HW; ++i) s += p[(size_t)i * C];
    job.out[(size_t)b * C + c] = s * inv;
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
    const float* lg = job.in + (size_t)b * n_classes;
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
  // vector path: channel-contiguous (NHWC) input with a channel count that keeps float4
  // groups inside one tap
  const bool vec = (g.in_sc == 1) && (g.Cin % 4 == 0) && (g.in_sx % 4 == 0) && (g.in_sy % 4 == 0) &&
                   (g.in_sb % 4 == 0);
  auto waste = [&](int bn) { return (g.Cout + bn - 1) / bn * bn - g.Cout; };
  int bn = 64;
  if (waste(32) < waste(bn)) bn = 32;
  if (waste(16) < waste(bn)) bn = 16;
  if (bn == 64) return launch_conv_tile<128, 64, 8, 4>(g, jobs_dev, n_jobs, net_input, vec, weight_bytes, s);
  if (bn == 32) return launch_conv_tile<128, 32, 4, 4>(g, jobs_dev, n_jobs, net_input, vec, weight_bytes, s);
  return launch_conv_tile<256, 16, 4, 4>(g, jobs_dev, n_jobs, net_input, vec, weight_bytes, s);
}

aiq_status_t launch_depthwise(const ConvGeom& g, const LayerJob* jobs_dev, int n_jobs,
                              const float* /*net_input*/, double weight_bytes, cudaStream_t s) {
  const int M = g.B * g.Ho * g.Wo;
  dim3 grid((M + kDwPixPerBlock - 1) / kDwPixPerBlock, (g.Cout + 127) / 128, n_jobs);
  LaunchScope scope(AIQ_KERNEL_DEPTHWISE, s, 18.0 * M * g.Cout * n_jobs,
                    weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W + (double)M * g.Cout));
  depthwise3x3_kernel<<<grid, 256, 0, s>>>(g, jobs_dev);
  AIQ_LAUNCH_CHECK("depthwise3x3");
  return AIQ_OK;
}

aiq_status_t launch_avgpool(const LayerJob* jobs_dev, int n_jobs, int B, int HW, int C, cudaStream_t s) {
  int threads = C >= 256 ? 256 : (C >= 128 ? 128 : 64);
  LaunchScope scope(AIQ_KERNEL_POOL, s, (double)n_jobs * B * HW * C, 4.0 * n_jobs * B * ((double)HW * C + C));
  avgpool_kernel<<<dim3(B, 1, n_jobs), threads, 0, s>>>(jobs_dev, HW, C);
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
