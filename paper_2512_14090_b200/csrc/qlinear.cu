// Small-batch quantized linear layer: y[m][n] = s_n * sum_k code[n][k] * x[m][k] + bias[n].
//
// The memory-bound case the method targets (Abstract; Section 5, Roofline paragraph): the
// packed weight matrix is streamed once with 128-bit loads, expanded to float32 in
// registers, multiplied against activations held in registers, and reduced across the
// warp with shuffles.  The per-channel scale multiplies the finished sum.
#include "common.cuh"

namespace aiq {

namespace {

constexpr int kRowsPerWarp = 4;
constexpr int kWarps = 8;

// 8 consecutive elements starting at element offset `e0` (a multiple of 8) inside a 16-byte
// packed chunk, as floats.
template <int BITS>
__device__ __forceinline__ void decode8(const uint4& q, int sub, float* f) {
  if (BITS == 4) {
    const uint32_t w = sub == 0 ? q.x : sub == 1 ? q.y : sub == 2 ? q.z : q.w;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      // offset-binary nibble in the mantissa of 2^23: exact integer-to-float without I2F
      const uint32_t u = (((w >> (4 * j)) & 0xFu) ^ 0x8u) | 0x4B000000u;
      f[j] = __uint_as_float(u) - 8388616.0f;
    }
  } else if (BITS == 8) {
    const uint32_t w0 = sub == 0 ? q.x : q.z;
    const uint32_t w1 = sub == 0 ? q.y : q.w;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t a = (((w0 >> (8 * j)) & 0xFFu) ^ 0x80u) | 0x4B000000u;
      const uint32_t b = (((w1 >> (8 * j)) & 0xFFu) ^ 0x80u) | 0x4B000000u;
      f[j] = __uint_as_float(a) - 8388736.0f;
      f[j + 4] = __uint_as_float(b) - 8388736.0f;
    }
  } else if (BITS == 16) {
    const __half2 h0 = *reinterpret_cast<const __half2*>(&q.x);
    const __half2 h1 = *reinterpret_cast<const __half2*>(&q.y);
    const __half2 h2 = *reinterpret_cast<const __half2*>(&q.z);
    const __half2 h3 = *reinterpret_cast<const __half2*>(&q.w);
    const float2 a = __half22float2(h0), b = __half22float2(h1), c = __half22float2(h2),
                 d = __half22float2(h3);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
  }
}

// One warp: kRowsPerWarp output channels x MT batch rows.  Lanes stride over 16-byte chunks
// of the packed rows.
template <int BITS, int MT>
__global__ void __launch_bounds__(kWarps * 32)
qlinear_kernel(LayerJob single, const LayerJob* __restrict__ jobs, int N, int K, int M) {
  const LayerJob job = jobs ? jobs[blockIdx.z] : single;
  constexpr int E = 128 / BITS;                 // elements per 16-byte chunk
  constexpr int SUBS = (E >= 8) ? E / 8 : 1;    // 8-element sub-chunks (fp32: one of 4)
  constexpr int SE = (E >= 8) ? 8 : 4;          // elements per sub-chunk
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int n0 = (blockIdx.x * kWarps + warp) * kRowsPerWarp;
  const int m0 = blockIdx.y * MT;
  if (n0 >= N) return;
  const int Kpad = (K + 31) / 32 * 32;
  const size_t rb = (size_t)Kpad * BITS / 8;
  const int n_chunks = Kpad / E;
  const float* __restrict__ x = static_cast<const float*>(job.in);
  const bool xvec = ((K & 3) == 0) && ((((uintptr_t)x) & 15) == 0);

  float acc[kRowsPerWarp][MT];
#pragma unroll
  for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
    for (int m = 0; m < MT; ++m) acc[r][m] = 0.0f;

  const uint8_t* rows[kRowsPerWarp];
#pragma unroll
  for (int r = 0; r < kRowsPerWarp; ++r) rows[r] = job.w + (size_t)min(n0 + r, N - 1) * rb;

  for (int ci = lane; ci < n_chunks; ci += 32) {
    uint4 q[kRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r) q[r] = __ldg(reinterpret_cast<const uint4*>(rows[r]) + ci);
#pragma unroll
    for (int sub = 0; sub < SUBS; ++sub) {
      const int k0 = ci * E + sub * SE;
      float xv[MT][SE];
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        const int mm = min(m0 + m, M - 1);
        const float* xp = x + (size_t)mm * K + k0;
        if (xvec && k0 + SE <= K) {
#pragma unroll
          for (int v = 0; v < SE / 4; ++v) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(xp) + v);
            xv[m][4 * v] = t.x; xv[m][4 * v + 1] = t.y; xv[m][4 * v + 2] = t.z; xv[m][4 * v + 3] = t.w;
          }
        } else {
#pragma unroll
          for (int j = 0; j < SE; ++j) xv[m][j] = (k0 + j < K) ? __ldg(xp + j) : 0.0f;
        }
      }
#pragma unroll
      for (int r = 0; r < kRowsPerWarp; ++r) {
        float wf[SE];
        if (BITS == 32) {
          wf[0] = __uint_as_float(q[r].x); wf[1] = __uint_as_float(q[r].y);
          wf[2] = __uint_as_float(q[r].z); wf[3] = __uint_as_float(q[r].w);
        } else {
          decode8<BITS>(q[r], sub, wf);
        }
#pragma unroll
        for (int j = 0; j < SE; ++j)
#pragma unroll
          for (int m = 0; m < MT; ++m) acc[r][m] = fmaf(wf[j], xv[m][j], acc[r][m]);
      }
    }
  }

#pragma unroll
  for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      float v = acc[r][m];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      acc[r][m] = v;
    }
  if (lane == 0) {
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r) {
      const int n = n0 + r;
      if (n >= N) break;
      const float s = job.scale[n];
      const float b = job.bias ? job.bias[n] : 0.0f;
#pragma unroll
      for (int m = 0; m < MT; ++m)
        if (m0 + m < M) static_cast<float*>(job.out)[(size_t)(m0 + m) * N + n] = fmaf(acc[r][m], s, b);
    }
  }
}

template <int BITS>
aiq_status_t launch_bits(const LayerJob* jobs_dev, const LayerJob& single, int n_jobs, int N, int K,
                         int M, cudaStream_t s) {
  const int gx = (N + kWarps * kRowsPerWarp - 1) / (kWarps * kRowsPerWarp);
  LaunchScope scope(AIQ_KERNEL_QLINEAR, s, 2.0 * M * N * K * n_jobs,
                    n_jobs * ((double)N * row_bytes(K, BITS) + 4.0 * N + 4.0 * M * ((double)K + N)));
  if (M == 1) {
    qlinear_kernel<BITS, 1><<<dim3(gx, 1, n_jobs), kWarps * 32, 0, s>>>(single, jobs_dev, N, K, M);
  } else if (M == 2) {
    qlinear_kernel<BITS, 2><<<dim3(gx, 1, n_jobs), kWarps * 32, 0, s>>>(single, jobs_dev, N, K, M);
  } else {
    qlinear_kernel<BITS, 4><<<dim3(gx, (M + 3) / 4, n_jobs), kWarps * 32, 0, s>>>(single, jobs_dev, N, K, M);
  }
  AIQ_LAUNCH_CHECK("qlinear");
  return AIQ_OK;
}

}  // namespace

aiq_status_t launch_qlinear(const LayerJob* jobs_dev, const LayerJob* single_host, int n_jobs, int N,
                            int K, int M, cudaStream_t s) {
  LayerJob single = {};
  int bits;
  if (jobs_dev) {
    // all jobs of one launch share a bit-width: the caller groups them
    bits = single_host->bits;
  } else {
    single = *single_host;
    bits = single.bits;
  }
  switch (bits) {
    case 4: return launch_bits<4>(jobs_dev, single, n_jobs, N, K, M, s);
    case 8: return launch_bits<8>(jobs_dev, single, n_jobs, N, K, M, s);
    case 16: return launch_bits<16>(jobs_dev, single, n_jobs, N, K, M, s);
    case 32: return launch_bits<32>(jobs_dev, single, n_jobs, N, K, M, s);
  }
  return set_error(AIQ_ERR_UNSUPPORTED_BITS, "qlinear: bits=%d", bits);
}

}  // namespace aiq

extern "C" size_t aiq_qlinear_workspace_bytes(int N, int K, int bits, int M) {
  if (N <= 0 || K <= 0 || M <= 0) return 0;
  if (aiq::qlinear_tc_applicable(N, K, bits, M)) return aiq::qlinear_tc_workspace_bytes(K, M) + 16;   // + status word
  if (aiq::qlinear_mma_applicable(N, K, bits, M)) return aiq::qlinear_mma_workspace_bytes(K, M);
  return 0;
}

extern "C" aiq_status_t aiq_qlinear(const void* packed, const float* scales, const float* bias, int N,
                                    int K, int bits, const float* x, int M, float* y, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  if (!aiq::bits_ok(bits)) return aiq::set_error(AIQ_ERR_UNSUPPORTED_BITS, "aiq_qlinear: bits=%d", bits);
  if (!packed || !scales || !x || !y) return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_qlinear: null pointer");
  if (N <= 0 || K <= 0 || M <= 0)
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_qlinear: N=%d K=%d M=%d", N, K, M);
  if (((uintptr_t)packed) & 15)
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_qlinear: packed not 16-byte aligned");
  aiq_status_t st = aiq::check_device_sm100();
  if (st != AIQ_OK) return st;
  aiq::LayerJob job = {};
  job.in = x;
  job.out = y;
  job.w = static_cast<const uint8_t*>(packed);
  job.scale = scales;
  job.bias = bias;
  job.bits = bits;
  // the tensor-core kernels need scratch for the converted activations
  if (workspace && aiq::qlinear_tc_applicable(N, K, bits, M)) {
    if (((uintptr_t)workspace) & 15)
      return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_qlinear: workspace not 16-byte aligned");
    const size_t scratch = aiq::qlinear_tc_workspace_bytes(K, M);
    if (workspace_bytes >= scratch + 16) {
      // device status word behind the scratch: 0, or 1 once a bounded wait of the kernel expired
      int32_t* status = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + scratch);
      AIQ_CUDA_TRY(cudaMemsetAsync(status, 0, 16, (cudaStream_t)stream));
      return aiq::launch_qlinear_tc(job, N, K, M, workspace, status, (cudaStream_t)stream);
    }
  } else if (workspace && aiq::qlinear_mma_applicable(N, K, bits, M)) {
    if (((uintptr_t)workspace) & 15)
      return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_qlinear: workspace not 16-byte aligned");
    if (workspace_bytes >= aiq::qlinear_mma_workspace_bytes(K, M))
      return aiq::launch_qlinear_mma(job, N, K, M, workspace, (cudaStream_t)stream);
  }
  return aiq::launch_qlinear(nullptr, &job, 1, N, K, M, (cudaStream_t)stream);
}
