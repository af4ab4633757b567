// Batch-norm folding and the per-output-channel weight quantizer + packer.
//
// Quantizer rule (the paper assigns per-layer bit-widths in Section 2.1 and leaves the
// formula open): symmetric, per output channel, max-abs scale, round half to even.
// Every float32 step is a single correctly rounded IEEE operation (explicit _rn
// intrinsics), so codes and scales are reproducible bit for bit.
#include "common.cuh"

#include <type_traits>

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
// quantize + pack
// ---------------------------------------------------------------------------------------
// code = rint(w / s) with the IEEE quotient, without dividing.  A true division costs ~10
// instructions, so the quotient is estimated as e = w * (1/s) inside one fused multiply-add
// with the constant 768: the sum lies in [512, 1024), where a float32 has 14 fraction bits,
// so the adder rounds e to the nearest multiple of 2^-14 and leaves that fixed-point number
// in the mantissa.  e and the correctly rounded quotient differ by at most 2^-23 relative
// (< 1.6e-5 absolute, |e| <= 128), so both round to the same integer unless the fixed-point
// value sits exactly on k + 1/2 (e within 2^-15 of a tie; one element in 2^14).  Only then is
// the exact division evaluated, which makes the result bit-identical to always dividing.
// Codes cannot leave [-qmax, qmax]: |w| <= amax and s = fl(amax / qmax).
struct RowQuantizer {
  float s, rs, lo, hi;
  bool estimate_ok;
  __device__ __forceinline__ RowQuantizer(float amax, int bits) {
    s = 1.0f; lo = 0.f; hi = 0.f;
    if (bits <= 8) {
      const float qmax = (float)((1 << (bits - 1)) - 1);
      if (amax != 0.0f) s = __fdiv_rn(amax, qmax);
      lo = -(float)(1 << (bits - 1));
      hi = qmax;
    }
    estimate_ok = s >= 1e-30f;           // a tiny scale would overflow the reciprocal: always divide
    rs = estimate_ok ? __frcp_rn(s) : 0.f;
  }
  __device__ __forceinline__ uint32_t code(float wv) const {
    // 768 = 1.5 * 2^9: bits = 0x44000000 + 0x400000 + round(2^14 e); u = round(2^14 e) + 2^13
    const uint32_t u = (uint32_t)__float_as_int(fmaf(wv, rs, 768.0f)) - 0x443FE000u;
    uint32_t c = (uint32_t)((int32_t)u >> 14);                      // floor(e + 1/2)
    if (!estimate_ok || (u & 16383u) == 0u)                          // on (or too close to) a tie
      c = (uint32_t)(int)fminf(fmaxf(rintf(__fdiv_rn(wv, s)), lo), hi);
    return c;
  }
};

// 8 consecutive elements -> packed output at granule index gi of the row
template <int BITS>
__device__ __forceinline__ void store_granule(uint8_t* out_row, int gi, const float* val, const RowQuantizer& rq) {
  if (BITS == 4) {
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) word |= (rq.code(val[j]) & 0xFu) << (4 * j);
    reinterpret_cast<uint32_t*>(out_row)[gi] = word;
  } else if (BITS == 8) {
    uint32_t w0 = 0, w1 = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      w0 |= (rq.code(val[j]) & 0xFFu) << (8 * j);
      w1 |= (rq.code(val[j + 4]) & 0xFFu) << (8 * j);
    }
    reinterpret_cast<uint2*>(out_row)[gi] = make_uint2(w0, w1);
  } else if (BITS == 16) {
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
}

// max |v| as an integer maximum of the sign-stripped bit patterns: NaN and infinity have
// the largest patterns, so they survive the reduction and the row maximum itself tells
// whether the row holds a non-finite element.
__device__ __forceinline__ uint32_t absbits(float v) { return (uint32_t)__float_as_int(v) & 0x7FFFFFFFu; }
constexpr uint32_t kInfBits = 0x7F800000u;

// --- general kernel: one block per row.  A thread owns granules of 8 consecutive elements
// (two float4 loads); up to CACHE granules per thread stay in registers between the max-abs
// pass and the rounding pass, so a row of up to blockDim * 8 * CACHE elements is read from
// memory once.
template <int CACHE, int BITS>
__global__ void __launch_bounds__(256, CACHE == 1 ? 4 : 3)
quantize_rows_kernel(const float* __restrict__ W, int K, int Kpad,
                     uint8_t* __restrict__ packed, float* __restrict__ scales,
                     int32_t* __restrict__ nonfinite_flag, const uint32_t* __restrict__ tensor_amax) {
  const int n = blockIdx.x;
  const float* row = W + (size_t)n * K;
  const int n_gran = Kpad >> 3;
  const bool vec_ok = ((K & 3) == 0) && ((((uintptr_t)row) & 15) == 0);

  float v[CACHE][8];
  uint32_t amax_bits = 0;

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
      for (int j = 0; j < 8; ++j) amax_bits = max(amax_bits, absbits(v[c][j]));
    }
  }
  // rows longer than the register cache: stream the remainder (re-read in pass 2)
  for (int gi = threadIdx.x + CACHE * blockDim.x; gi < n_gran; gi += blockDim.x) {
    float t[8];
    load_granule(gi, t);
#pragma unroll
    for (int j = 0; j < 8; ++j) amax_bits = max(amax_bits, absbits(t[j]));
  }

  __shared__ uint32_t s_max[8];
  amax_bits = __reduce_max_sync(0xffffffffu, amax_bits);
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax_bits;
  __syncthreads();
  amax_bits = 0;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) amax_bits = max(amax_bits, s_max[w]);
  if (amax_bits >= kInfBits) {
    if (threadIdx.x == 0 && nonfinite_flag) *nonfinite_flag = 1;
    return;
  }
  // per-tensor variant: the maximum over the whole tensor (computed by tensor_absmax_kernel) sets the scale
  if (tensor_amax) amax_bits = *tensor_amax;
  const RowQuantizer rq(__uint_as_float(amax_bits), BITS);
  if (threadIdx.x == 0) scales[n] = rq.s;

  uint8_t* out_row = packed + (size_t)n * ((size_t)Kpad * BITS / 8);
#pragma unroll
  for (int c = 0; c < CACHE; ++c) {
    const int gi = threadIdx.x + c * blockDim.x;
    if (gi < n_gran) store_granule<BITS>(out_row, gi, v[c], rq);
  }
  for (int gi = threadIdx.x + CACHE * blockDim.x; gi < n_gran; gi += blockDim.x) {
    float t[8];
    load_granule(gi, t);
    store_granule<BITS>(out_row, gi, t, rq);
  }
}

// All four bit-widths of a layer from one read of its rows (the weight bank of a model: the
// per-width kernel above would be launched four times on the same small matrix).  Same
// quantizer and packing routines, so the bytes equal those of four separate calls.
struct BankOut { uint8_t* packed[4]; float* scales[4]; };

template <int CACHE>
__global__ void __launch_bounds__(256, CACHE == 1 ? 4 : 3)
quantize_bank_kernel(const float* __restrict__ W, int K, int Kpad, BankOut out, int32_t* __restrict__ nonfinite_flag,
                     const uint32_t* __restrict__ tensor_amax) {
  const int n = blockIdx.x;
  const float* row = W + (size_t)n * K;
  const int n_gran = Kpad >> 3;
  const bool vec_ok = ((K & 3) == 0) && ((((uintptr_t)row) & 15) == 0);
  float v[CACHE][8];
  uint32_t amax_bits = 0;
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
      for (int j = 0; j < 8; ++j) amax_bits = max(amax_bits, absbits(v[c][j]));
    }
  }
  for (int gi = threadIdx.x + CACHE * blockDim.x; gi < n_gran; gi += blockDim.x) {
    float t[8];
    load_granule(gi, t);
#pragma unroll
    for (int j = 0; j < 8; ++j) amax_bits = max(amax_bits, absbits(t[j]));
  }
  __shared__ uint32_t s_max[8];
  amax_bits = __reduce_max_sync(0xffffffffu, amax_bits);
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax_bits;
  __syncthreads();
  amax_bits = 0;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) amax_bits = max(amax_bits, s_max[w]);
  if (amax_bits >= kInfBits) {
    if (threadIdx.x == 0 && nonfinite_flag) *nonfinite_flag = 1;
    return;
  }
  const uint32_t code_amax = tensor_amax ? *tensor_amax : amax_bits;   // per-tensor scales apply to the integer codes only
  auto emit = [&](auto bits_tag, int slot, uint32_t amax) {
    constexpr int BITS = decltype(bits_tag)::value;
    const RowQuantizer rq(__uint_as_float(amax), BITS);
    if (threadIdx.x == 0) out.scales[slot][n] = rq.s;
    uint8_t* out_row = out.packed[slot] + (size_t)n * ((size_t)Kpad * BITS / 8);
#pragma unroll
    for (int c = 0; c < CACHE; ++c) {
      const int gi = threadIdx.x + c * blockDim.x;
      if (gi < n_gran) store_granule<BITS>(out_row, gi, v[c], rq);
    }
    for (int gi = threadIdx.x + CACHE * blockDim.x; gi < n_gran; gi += blockDim.x) {
      float t[8];
      load_granule(gi, t);
      store_granule<BITS>(out_row, gi, t, rq);
    }
  };
  emit(std::integral_constant<int, 4>(), 0, code_amax);
  emit(std::integral_constant<int, 8>(), 1, code_amax);
  emit(std::integral_constant<int, 16>(), 2, amax_bits);
  emit(std::integral_constant<int, 32>(), 3, amax_bits);
}

// --- streaming kernel for large matrices (the roofline case): persistent blocks, every row
// arrives in shared memory by one bulk copy issued kStreamStages rows ahead, so the memory
// system stays busy while a block reduces, rounds and packs.  A row goes from shared memory
// into registers once (the stage is refilled right after), is reduced with one block-wide
// barrier and leaves as packed words.  Needs K % 32 == 0, 16-byte aligned rows and
// K <= 8192 (4 granules of 8 elements per thread).
constexpr int kStreamThreads = 256;
constexpr int kStreamCache = 4;

// Bounded by SM clocks (about 2 s), like the waits of the tensor-core kernels: the time one poll
// takes is up to the hardware, so a poll count alone would not bound the wait in seconds.
__device__ __forceinline__ bool stream_wait(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  for (uint32_t i = 0; i < (1u << 30); ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
    if ((i & 255u) == 255u && clock64() - t0 > 4000ll * 1000ll * 1000ll) break;
  }
  return false;                          // bounded: a copy that never lands must not hang the GPU
}

template <int BITS>
__global__ void __launch_bounds__(kStreamThreads, 4)
quantize_stream_kernel(const float* __restrict__ W, int N, int K, uint8_t* __restrict__ packed,
                       float* __restrict__ scales, int32_t* __restrict__ nonfinite_flag, int stages) {
  extern __shared__ __align__(128) uint8_t qs[];
  const uint32_t row_bytes_in = (uint32_t)K * 4u;
  uint64_t* bars = reinterpret_cast<uint64_t*>(qs + (size_t)stages * row_bytes_in);
  __shared__ uint32_t s_max[2][8];
  const int tid = threadIdx.x;
  const int n_gran = K >> 3;
  const int n_mine = (N - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  const uint32_t buf0 = (uint32_t)__cvta_generic_to_shared(qs);

  auto issue = [&](int i) {              // row i of this block -> stage i % stages (thread 0)
    const int st = i % stages;
    const float* src = W + (size_t)(blockIdx.x + (size_t)i * gridDim.x) * K;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar0 + 8 * st), "r"(row_bytes_in) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(buf0 + st * row_bytes_in), "l"(reinterpret_cast<uint64_t>(src)), "r"(row_bytes_in), "r"(bar0 + 8 * st)
                 : "memory");
  };
  if (tid == 0) {
    for (int i = 0; i < stages; ++i)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar0 + 8 * i), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int i = 0; i < stages && i < n_mine; ++i) issue(i);
  }
  __syncthreads();

  for (int i = 0; i < n_mine; ++i) {
    const int st = i % stages;
    const int n = blockIdx.x + i * gridDim.x;
    if (!stream_wait(bar0 + 8 * st, (uint32_t)(i / stages) & 1u)) {
      if (nonfinite_flag) *nonfinite_flag = 2;
      return;
    }
    const float* row = reinterpret_cast<const float*>(qs + (size_t)st * row_bytes_in);
    float v[kStreamCache][8];
    uint32_t amax_bits = 0;
#pragma unroll
    for (int c = 0; c < kStreamCache; ++c) {
      const int gi = tid + c * kStreamThreads;
      if (gi < n_gran) {
        const float4 a = *reinterpret_cast<const float4*>(row + 8 * gi);
        const float4 b = *reinterpret_cast<const float4*>(row + 8 * gi + 4);
        v[c][0] = a.x; v[c][1] = a.y; v[c][2] = a.z; v[c][3] = a.w;
        v[c][4] = b.x; v[c][5] = b.y; v[c][6] = b.z; v[c][7] = b.w;
#pragma unroll
        for (int j = 0; j < 8; ++j) amax_bits = max(amax_bits, absbits(v[c][j]));
      }
    }
    amax_bits = __reduce_max_sync(0xffffffffu, amax_bits);
    if ((tid & 31) == 0) s_max[i & 1][tid >> 5] = amax_bits;
    __syncthreads();                     // every thread holds its part of the row in registers
    if (tid == 0 && i + stages < n_mine) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the reads above before the copy's writes
      issue(i + stages);
    }
    amax_bits = 0;
#pragma unroll
    for (int w = 0; w < kStreamThreads / 32; ++w) amax_bits = max(amax_bits, s_max[i & 1][w]);
    if (amax_bits >= kInfBits) {         // uniform over the block: the row is skipped
      if (tid == 0 && nonfinite_flag) *nonfinite_flag = 1;
      continue;
    }
    const RowQuantizer rq(__uint_as_float(amax_bits), BITS);
    if (tid == 0) scales[n] = rq.s;
    uint8_t* out_row = packed + (size_t)n * ((size_t)K * BITS / 8);
#pragma unroll
    for (int c = 0; c < kStreamCache; ++c) {
      const int gi = tid + c * kStreamThreads;
      if (gi < n_gran) store_granule<BITS>(out_row, gi, v[c], rq);
    }
  }
}

// max |w| over a whole tensor, as the integer maximum of the sign-stripped bit patterns (order-free,
// so atomics give a reproducible result).  *out must be zero before the launch.
__global__ void tensor_absmax_kernel(const float* __restrict__ W, size_t n, uint32_t* __restrict__ out) {
  uint32_t m = 0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    m = max(m, absbits(__ldg(W + i)));
  m = __reduce_max_sync(0xffffffffu, m);
  if ((threadIdx.x & 31) == 0 && m) atomicMax(out, m);
}

template <int BITS>
aiq_status_t launch_quantize_bits(const float* W, int N, int K, void* packed, float* scales,
                                  int32_t* nonfinite_flag, uint32_t* tensor_amax, cudaStream_t s) {
  const int Kpad = padded_k(K);
  const int n_gran = Kpad / 8;
  uint8_t* p = static_cast<uint8_t*>(packed);
  LaunchScope scope(AIQ_KERNEL_QUANTIZE, s, 2.0 * N * K,
                    4.0 * N * K + (double)N * row_bytes(K, BITS) + 4.0 * N);
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  const int n_sms = props.n_sms, smem_limit = props.smem_optin;
  if (tensor_amax) {
    AIQ_CUDA_TRY(cudaMemsetAsync(tensor_amax, 0, 4, s));
    const size_t n = (size_t)N * K;
    int blocks = (int)((n + 1023) / 1024);
    if (blocks > 8 * n_sms) blocks = 8 * n_sms;
    tensor_absmax_kernel<<<blocks, 256, 0, s>>>(W, n, tensor_amax);
    AIQ_LAUNCH_CHECK("tensor_absmax");
  }
  const bool stream_ok = !tensor_amax && K % 32 == 0 && K >= 2048 && K <= kStreamThreads * 8 * kStreamCache &&
                         N >= 4 * n_sms && ((uintptr_t)W & 15) == 0;
  if (stream_ok) {
    // As many blocks per SM (up to 4) as leave each a ring of at least two rows: the rounding
    // pass is a chain of dependent instructions, so resident warps matter as much as bytes in
    // flight (ncu at two blocks per SM: 25 % of the warp slots, issue slots half used).
    int blocks_per_sm = 4, stages = 0;
    for (; blocks_per_sm >= 2; --blocks_per_sm) {
      const int per_block = (smem_limit + 1024) / blocks_per_sm - 2048;   // minus the per-block reserve
      stages = per_block / (K * 4);
      if (stages >= 2) break;
    }
    if (stages > 8) stages = 8;
    if (stages >= 2) {
      const int smem = stages * K * 4 + stages * 8;
      AIQ_ENSURE_DYNAMIC_SMEM(quantize_stream_kernel<BITS>, smem_limit - 1024);   // the kernel also has static shared memory
      quantize_stream_kernel<BITS><<<blocks_per_sm * n_sms, kStreamThreads, smem, s>>>(W, N, K, p, scales, nonfinite_flag, stages);
      AIQ_LAUNCH_CHECK("quantize_stream");
      return AIQ_OK;
    }
  }
  int threads = 32;
  while (threads < 256 && threads < n_gran) threads <<= 1;
  if (n_gran <= threads) {
    quantize_rows_kernel<1, BITS><<<N, threads, 0, s>>>(W, K, Kpad, p, scales, nonfinite_flag, tensor_amax);
  } else {
    quantize_rows_kernel<4, BITS><<<N, threads, 0, s>>>(W, K, Kpad, p, scales, nonfinite_flag, tensor_amax);
  }
  AIQ_LAUNCH_CHECK("quantize_rows");
  return AIQ_OK;
}

aiq_status_t launch_quantize(const float* W, int N, int K, int bits, void* packed, float* scales,
                             int32_t* nonfinite_flag, uint32_t* tensor_amax, cudaStream_t s) {
  switch (bits) {
    case 4: return launch_quantize_bits<4>(W, N, K, packed, scales, nonfinite_flag, tensor_amax, s);
    case 8: return launch_quantize_bits<8>(W, N, K, packed, scales, nonfinite_flag, tensor_amax, s);
    case 16: return launch_quantize_bits<16>(W, N, K, packed, scales, nonfinite_flag, nullptr, s);
    default: return launch_quantize_bits<32>(W, N, K, packed, scales, nonfinite_flag, nullptr, s);
  }
}

// The four versions (4, 8, 16, 32 bits) of one layer of a model's weight bank.
aiq_status_t launch_quantize_bank(const float* W, int N, int K, void* const* packed, float* const* scales,
                                  int32_t* nonfinite_flag, uint32_t* tensor_amax, cudaStream_t s) {
  static const int kBits[4] = {4, 8, 16, 32};
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  const int Kpad = padded_k(K), n_gran = Kpad / 8;
  // large matrices take the streaming kernel, one launch per width
  const bool stream_ok = !tensor_amax && K % 32 == 0 && K >= 2048 && N >= 4 * props.n_sms;
  if (stream_ok) {
    for (int b = 0; b < 4; ++b)
      if (aiq_status_t st = launch_quantize(W, N, K, kBits[b], packed[b], scales[b], nonfinite_flag, nullptr, s)) return st;
    return AIQ_OK;
  }
  double out_bytes = 0.0;
  for (int b = 0; b < 4; ++b) out_bytes += (double)N * row_bytes(K, kBits[b]) + 4.0 * N;
  LaunchScope scope(AIQ_KERNEL_QUANTIZE, s, 8.0 * N * K, 4.0 * N * K + out_bytes);
  if (tensor_amax) {
    AIQ_CUDA_TRY(cudaMemsetAsync(tensor_amax, 0, 4, s));
    const size_t n = (size_t)N * K;
    int blocks = (int)((n + 1023) / 1024);
    if (blocks > 8 * props.n_sms) blocks = 8 * props.n_sms;
    tensor_absmax_kernel<<<blocks, 256, 0, s>>>(W, n, tensor_amax);
    AIQ_LAUNCH_CHECK("tensor_absmax");
  }
  BankOut out;
  for (int b = 0; b < 4; ++b) { out.packed[b] = static_cast<uint8_t*>(packed[b]); out.scales[b] = scales[b]; }
  int threads = 32;
  while (threads < 256 && threads < n_gran) threads <<= 1;
  if (n_gran <= threads) quantize_bank_kernel<1><<<N, threads, 0, s>>>(W, K, Kpad, out, nonfinite_flag, tensor_amax);
  else quantize_bank_kernel<4><<<N, threads, 0, s>>>(W, K, Kpad, out, nonfinite_flag, tensor_amax);
  AIQ_LAUNCH_CHECK("quantize_bank");
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
  return aiq::launch_quantize(W, N, K, bits, packed_out, scales_out, nonfinite_flag, nullptr, (cudaStream_t)stream);
}

extern "C" aiq_status_t aiq_quantize_layer_per_tensor(const float* W, int N, int K, int bits, void* packed_out,
                                                      float* scales_out, int32_t* nonfinite_flag, void* scratch,
                                                      void* stream) {
  if (!aiq::bits_ok(bits))
    return aiq::set_error(AIQ_ERR_UNSUPPORTED_BITS, "aiq_quantize_layer_per_tensor: bits=%d", bits);
  if (!W || !packed_out || !scales_out || !scratch)
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_quantize_layer_per_tensor: null pointer");
  if (N <= 0 || K <= 0)
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_quantize_layer_per_tensor: N=%d K=%d", N, K);
  if ((((uintptr_t)packed_out) & 15) || (((uintptr_t)scratch) & 3))
    return aiq::set_error(AIQ_ERR_INVALID_ARG, "aiq_quantize_layer_per_tensor: packed_out must be 16-byte, scratch 4-byte aligned");
  aiq_status_t st = aiq::check_device_sm100();
  if (st != AIQ_OK) return st;
  return aiq::launch_quantize(W, N, K, bits, packed_out, scales_out, nonfinite_flag, static_cast<uint32_t*>(scratch),
                              (cudaStream_t)stream);
}
