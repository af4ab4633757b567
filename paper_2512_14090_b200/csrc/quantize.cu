// Batch-norm folding and the per-output-channel weight quantizer + packer.
//
// Quantizer rule (the paper assigns per-layer bit-widths in Section 2.1 and leaves the
// formula open): symmetric, per output channel, max-abs scale, round half to even.
// Every float32 step is a single correctly rounded IEEE operation (explicit _rn
// intrinsics), so codes and scales are reproducible bit for bit.
#include "common.cuh"

namespace aiq {

// ---------------------------------------------------------------------------------------
// fold: one block per output channel
// ---------------------------------------------------------------------------------------
__global__ void fold_bn_kernel(const float* __restrict__ W, const float* __restrict__ gamma,
                               const float* __restrict__ beta, const float* __restrict__ mean,
                               const float* __restrict__ var, int K, float eps,
                               float* __restrict__ Wf, float* __restrict__ bf) {
  const int n = blockIdx.x;
  const float g = __fdiv_rn(gamma[n], __fsqrt_rn(__fadd_rn(var[n], eps)));
  const float* src = W + (size_t)n * K;
  float* dst = Wf + (size_t)n * K;
  for (int k = threadIdx.x; k < K; k += blockDim.x) dst[k] = __fmul_rn(src[k], g);
  if (threadIdx.x == 0) bf[n] = __fsub_rn(beta[n], __fmul_rn(mean[n], g));
}

aiq_status_t launch_fold_bn(const float* W, const float* gamma, const float* beta, const float* mean,
                            const float* var, int N, int K, float eps, float* Wf, float* bf,
                            cudaStream_t s) {
  int threads = K >= 256 ? 256 : (K >= 128 ? 128 : (K >= 64 ? 64 : 32));
  {
    LaunchScope scope(AIQ_KERNEL_FOLD, s, (double)N * K, 8.0 * N * K + 20.0 * N);
    fold_bn_kernel<<<N, threads, 0, s>>>(W, gamma, beta, mean, var, K, eps, Wf, bf);
  }
  AIQ_LAUNCH_CHECK("fold_bn");
  return AIQ_OK;
}

// ---------------------------------------------------------------------------------------
// quantize + pack: one block per row.  A thread owns granules of 8 consecutive elements
// (two float4 loads); up to CACHE granules per thread stay in registers between the
// max-abs pass and the rounding pass, so a row of up to blockDim * 8 * CACHE elements is
// read from memory once.
// ---------------------------------------------------------------------------------------
template <int CACHE>
__global__ void __launch_bounds__(256, CACHE == 1 ? 4 : 3)
quantize_rows_kernel(const float* __restrict__ W, int K, int Kpad, int bits,
                     uint8_t* __restrict__ packed, float* __restrict__ scales,
                     int32_t* __restrict__ nonfinite_flag) {
  const int n = blockIdx.x;
  const float* row = W + (size_t)n * K;
  const int n_gran = Kpad >> 3;
  const bool vec_ok = ((K & 3) == 0) && ((((uintptr_t)row) & 15) == 0);

  float v[CACHE][8];
  float amax = 0.0f;
  float poison = 0.0f;           // stays 0 unless an element is NaN or infinite (x * 0 is then NaN)

  auto load_granule = [&](int gi, float* dstv) {
    const int k0 = gi << 3;
    if (vec_ok && k0 + 8 <= K) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(row + k0));
      const float4 b = __ldg(reinterpret_cast<const float4*>(row + k0 + 4));
      dstv[0] = a.x; dstv[1] = a.y; dstv[2] = a.z; dstv[3] = a.w;
      dstv[4] = b.x; dstv[5] = b.y; dstv[6] = b.z; dstv[7] = b.w;
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) dstv[j] = (k0 + j < K) ? __ldg(row + k0 + j) : 0.0f;
    }
  };

#pragma unroll
  for (int c = 0; c < CACHE; ++c) {
    const int gi = threadIdx.x + c * blockDim.x;
    if (gi < n_gran) {
      load_granule(gi, v[c]);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        poison = fmaf(v[c][j], 0.0f, poison);
        amax = fmaxf(amax, fabsf(v[c][j]));
      }
    }
  }
  // rows longer than the register cache: stream the remainder (re-read in pass 2)
  for (int gi = threadIdx.x + CACHE * blockDim.x; gi < n_gran; gi += blockDim.x) {
    float t[8];
    load_granule(gi, t);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      poison = fmaf(t[j], 0.0f, poison);
      amax = fmaxf(amax, fabsf(t[j]));
    }
  }

  __shared__ float s_max[8];
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
  if (poison != 0.0f) s_bad = 1;                 // NaN compares unequal to everything
  __syncthreads();
  amax = 0.0f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) amax = fmaxf(amax, s_max[w]);
  if (s_bad) {
    if (threadIdx.x == 0 && nonfinite_flag) *nonfinite_flag = 1;
    return;
  }

  float s = 1.0f;
  float lo = 0.f, hi = 0.f;
  if (bits <= 8) {
    const float qmax = (float)((1 << (bits - 1)) - 1);
    if (amax != 0.0f) s = __fdiv_rn(amax, qmax);
    lo = -(float)(1 << (bits - 1));
    hi = qmax;
  }
  if (threadIdx.x == 0) scales[n] = s;

  uint8_t* out_row = packed + (size_t)n * ((size_t)Kpad * bits / 8);
  // code = rint(w / s) with the IEEE quotient.  A true division costs ~10 instructions, so the
  // quotient is first estimated as w * (1/s): the estimate and the correctly rounded quotient
  // differ by at most 1.5 * 2^-23 relative, hence they round to the same integer unless the
  // estimate lies within that distance of a tie.  Only then (about one element in 10^4) is
  // the exact division evaluated, so the result is bit-identical to always dividing.
  const bool estimate_ok = s >= 1e-30f;        // a tiny scale would overflow the reciprocal: always divide
  const float rs = estimate_ok ? __frcp_rn(s) : 0.f;
  // Rounding without the conversion unit: adding 1.5 * 2^23 rounds the estimate to the nearest
  // integer (ties to even) in the adder, and leaves that integer, in two's complement, in the
  // low mantissa bits of the sum.  |estimate| <= 128, far inside the range where this holds.
  // Codes cannot leave [-qmax, qmax]: |w| <= amax and s = fl(amax / qmax).
  auto code_of = [&](float wv) -> uint32_t {
    const float tq = wv * rs;
    const float m = tq + 12582912.0f;
    const float q = m - 12582912.0f;
    uint32_t code = (uint32_t)__float_as_int(m);
    if (!estimate_ok || fabsf(fabsf(tq - q) - 0.5f) <= fabsf(tq) * 4.8e-7f)   // 2^-21: near a tie
      code = (uint32_t)(int)fminf(fmaxf(rintf(__fdiv_rn(wv, s)), lo), hi);
    return code;
  };
  auto store_granule = [&](int gi, const float* val) {
    if (bits == 4) {
      uint32_t word = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        word |= (code_of(val[j]) & 0xFu) << (4 * j);
      }
      reinterpret_cast<uint32_t*>(out_row)[gi] = word;
    } else if (bits == 8) {
      uint32_t w0 = 0, w1 = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        w0 |= (code_of(val[j]) & 0xFFu) << (8 * j);
        w1 |= (code_of(val[j + 4]) & 0xFFu) << (8 * j);
      }
      reinterpret_cast<uint2*>(out_row)[gi] = make_uint2(w0, w1);
    } else if (bits == 16) {
      __half2 h0 = __floats2half2_rn(val[0], val[1]);
      __half2 h1 = __floats2half2_rn(val[2], val[3]);
      __half2 h2 = __floats2half2_rn(val[4], val[5]);
      __half2 h3 = __floats2half2_rn(val[6], val[7]);
      uint4 o;
      o.x = *reinterpret_cast<uint32_t*>(&h0);
      o.y = *reinterpret_cast<uint32_t*>(&h1);
      o.z = *reinterpret_cast<uint32_t*>(&h2);
      o.w = *reinterpret_cast<uint32_t*>(&h3);
      reinterpret_cast<uint4*>(out_row)[gi] = o;
    } else {
      float4* o = reinterpret_cast<float4*>(out_row) + 2 * (size_t)gi;
      o[0] = make_float4(val[0], val[1], val[2], val[3]);
      o[1] = make_float4(val[4], val[5], val[6], val[7]);
    }
  };

#pragma unroll
  for (int c = 0; c < CACHE; ++c) {
    const int gi = threadIdx.x + c * blockDim.x;
    if (gi < n_gran) store_granule(gi, v[c]);
  }
  for (int gi = threadIdx.x + CACHE * blockDim.x; gi < n_gran; gi += blockDim.x) {
    float t[8];
    load_granule(gi, t);
    store_granule(gi, t);
  }
}

aiq_status_t launch_quantize(const float* W, int N, int K, int bits, void* packed, float* scales,
                             int32_t* nonfinite_flag, cudaStream_t s) {
  const int Kpad = padded_k(K);
  const int n_gran = Kpad / 8;
  int threads = 32;
  while (threads < 256 && threads < n_gran) threads <<= 1;
  uint8_t* p = static_cast<uint8_t*>(packed);
  {
    LaunchScope scope(AIQ_KERNEL_QUANTIZE, s, 2.0 * N * K,
                      4.0 * N * K + (double)N * row_bytes(K, bits) + 4.0 * N);
    if (n_gran <= threads) {
      quantize_rows_kernel<1><<<N, threads, 0, s>>>(W, K, Kpad, bits, p, scales, nonfinite_flag);
    } else {
      quantize_rows_kernel<4><<<N, threads, 0, s>>>(W, K, Kpad, bits, p, scales, nonfinite_flag);
    }
  }
  AIQ_LAUNCH_CHECK("quantize_rows");
  return AIQ_OK;
}

}  // namespace aiq

// ---------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------
extern "C" size_t aiq_packed_row_bytes(int K, int bits) {
  if (K <= 0 || !aiq::bits_ok(bits)) return 0;
  return aiq::row_bytes(K, bits);
}

extern "C" aiq_status_t aiq_fold_bn(const float* W, const float* gamma, const float* beta,
                                    const float* mean, const float* var, int N, int K, float eps,
                                    float* Wf, float* bf, void* stream) {
  if (!W || !gamma || !beta || !mean || !var || !Wf || !bf)
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_fold_bn: null pointer");
  if (N <= 0 || K <= 0) return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_fold_bn: N=%d K=%d", N, K);
  aiq_status_t st = aiq::check_device_sm100();
  if (st != AIQ_OK) return st;
  return aiq::launch_fold_bn(W, gamma, beta, mean, var, N, K, eps, Wf, bf, (cudaStream_t)stream);
}

extern "C" aiq_status_t aiq_quantize_layer(const float* W, int N, int K, int bits, void* packed_out,
                                           float* scales_out, int32_t* nonfinite_flag, void* stream) {
  if (!aiq::bits_ok(bits))
    return aiq::set_error(AIQ_ERR_UNSUPPORTED_BITS, "aiq_quantize_layer: bits=%d", bits);
  if (!W || !packed_out || !scales_out)
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_quantize_layer: null pointer");
  if (N <= 0 || K <= 0)
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_quantize_layer: N=%d K=%d", N, K);
  if (((uintptr_t)packed_out) & 15)
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_quantize_layer: packed_out not 16-byte aligned");
  aiq_status_t st = aiq::check_device_sm100();
  if (st != AIQ_OK) return st;
  return aiq::launch_quantize(W, N, K, bits, packed_out, scales_out, nonfinite_flag, (cudaStream_t)stream);
}
