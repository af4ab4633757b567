// Small-batch quantized linear layer for 4- and 8-bit weights, M <= 16, on the warp-level
// integer tensor-core path.
//
//   y[m][n] = s_n * sum_k code[n][k] * x[m][k] + bias[n]
//
// At 4 bits the weight stream arrives at ~13 T elements/s when HBM runs at full speed; a
// kernel that converts every code to floating point and multiplies it on the CUDA cores
// cannot keep up.  Here the codes stay integers: packed words go from global memory to shared
// memory (cp.async) to registers and feed mma.sync.m16n8k32 (s8 x s8 -> s32) as the A operand
// (16 output channels x 32 k).  8-bit rows are used as they are; a 4-bit word needs one AND
// and one shift-AND to become two registers of bytes (the +8 of the offset-binary nibbles is
// taken out again exactly, in integers, with the column sums of the activations).
//
// The activations are brought to the integer side once per block: for each batch row and
// K-slice, x = 2^(e-6) * (d1 + d2 / 2^7 + d3 / 2^14) with three int8 digits and a shared
// exponent e (2^e > max |x| of the slice), a 21-bit fixed-point image of x relative to that
// maximum.  Each digit is a column of the B operand, so a batch row costs three of the eight
// columns of an MMA; the three int32 sums are exact and are recombined in float32 as
// s_n * 2^(e-6) * (S1 + S2 / 2^7 + S3 / 2^14).
//
// Work split: a block owns 128 output channels x a K-slice of 512 or 1024; each of its 4
// warps owns 32 channels (two 16-row MMA tiles) and streams them through a private
// shared-memory ring (a stage = 32 rows x 64 bytes; 40 KB per block, so five blocks = 20
// warps share an SM).  Rows 2i and 2i+1 fill one 128-byte bank window, so the fragment
// reads are free of bank conflicts.  The element order inside a fragment follows what the
// unpacking produces (the k index is permuted identically on both operands).  K-slices add
// their partial sums into y with float atomics (y is zeroed first); the order of those few
// additions is not fixed, so the last bit of y may differ from run to run.
#include "common.cuh"

namespace aiq {

namespace {

constexpr int kMmaWarps = 4;
constexpr int kMmaRowsPerWarp = 32;
constexpr int kMmaRowsPerBlock = kMmaWarps * kMmaRowsPerWarp;
constexpr int kStageRowBytes = 64;                 // bytes of one weight row per pipeline stage
constexpr int kStageBytes = kMmaRowsPerWarp * kStageRowBytes;
constexpr int kStages = 3;
constexpr int kMaxM = 16;

__device__ __forceinline__ void mma_s8_16832(int* d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N_>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N_) : "memory"); }

// k offsets (inside the run of consecutive elements a lane owns in one stage) of the eight A
// bytes a lane contributes to MMA j: o[0..3] feed a0 / a1 (k = 4t .. 4t+3 of the fragment),
// o[4..7] feed a2 / a3 (k = 16 + 4t ..).
//   4 bits: a lane owns 32 k (one 16-byte unit); word j gives its even nibbles to a0 and its
//           odd nibbles to a2.
//   8 bits: a lane owns 16 k; words 2j and 2j+1 are a0 and a2.
template <int BITS>
__device__ __forceinline__ void frag_k_offsets(int j, int* o) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o[i] = BITS == 4 ? 8 * j + 2 * i : 8 * j + i;
    o[4 + i] = BITS == 4 ? 8 * j + 2 * i + 1 : 8 * j + 4 + i;
  }
}

__device__ __forceinline__ uint32_t pack_s8(int a, int b, int c, int d) {
  return (uint32_t)(a & 0xFF) | ((uint32_t)(b & 0xFF) << 8) | ((uint32_t)(c & 0xFF) << 16) | ((uint32_t)(d & 0xFF) << 24);
}

constexpr int kGroupK = 512;                       // k that share one activation exponent
constexpr int kGroupFrags = kGroupK / 32;          // k32 fragments per group

// Workspace layout: [group][fragment][column tile][lane] uint2, then per group 16 floats
// (2^(e-6) per batch row) and 48 ints (digit-column sums).
__host__ __device__ inline size_t ws_frag_bytes(int n_groups, int nt) { return (size_t)n_groups * kGroupFrags * nt * 32 * sizeof(uint2); }
constexpr int kMetaBytes = 16 * 4 + 48 * 4;

// Pre-pass: one block per group of 512 k.  Brings the activations to the integer side:
// x = 2^(e-6) * (d1 + d2 / 2^7 + d3 / 2^14), digits written in B-fragment order.
template <int BITS, int NT>
__global__ void __launch_bounds__(256)
qlinear_digits_kernel(const float* __restrict__ x, int K, int M, uint8_t* __restrict__ ws, int n_groups,
                      float* __restrict__ y, int y_elems) {
  // let the main kernel start right away: its first weight loads do not depend on this grid
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < y_elems; i += gridDim.x * blockDim.x) y[i] = 0.f;
  constexpr int KL = BITS == 4 ? 32 : 16;
  constexpr int CHUNK = 4 * KL;
  constexpr int MPC = CHUNK / 32;
  __shared__ int s_xmax[kMaxM];
  __shared__ float s_up[kMaxM];
  __shared__ int s_colsum[48];
  const int grp = blockIdx.x, k0 = grp * kGroupK, lane = threadIdx.x & 31;
  uint2 (*frags)[NT][32] = reinterpret_cast<uint2 (*)[NT][32]>(ws + (size_t)grp * kGroupFrags * NT * 32 * sizeof(uint2));
  uint8_t* meta = ws + ws_frag_bytes(n_groups, NT) + (size_t)grp * kMetaBytes;
  if (threadIdx.x < kMaxM) s_xmax[threadIdx.x] = 0;
  if (threadIdx.x < 48) s_colsum[threadIdx.x] = 0;
  for (int idx = threadIdx.x; idx < kGroupFrags * NT * 32; idx += blockDim.x) {
    const int fl = idx & 31, nt = (idx >> 5) % NT, f = idx / (32 * NT);
    if (nt * 8 + (fl >> 2) >= 3 * M) frags[f][nt][fl] = make_uint2(0u, 0u);      // unused columns
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < M * kGroupK; idx += blockDim.x) {            // one batch row per warp pass
    const int m = idx / kGroupK, k = k0 + (idx - m * kGroupK);
    int bits = k < K ? (__float_as_int(__ldg(x + (size_t)m * K + k)) & 0x7FFFFFFF) : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bits = max(bits, __shfl_xor_sync(0xffffffffu, bits, o));
    if (lane == 0) atomicMax(&s_xmax[m], bits);
  }
  __syncthreads();
  if (threadIdx.x < M) {
    const float xmax = __int_as_float(s_xmax[threadIdx.x]);
    int e = 0;
    frexpf(xmax, &e);                                   // xmax = f * 2^e with f in [0.5, 1)
    s_up[threadIdx.x] = xmax > 0.f ? ldexpf(1.f, 6 - e) : 0.f;
    reinterpret_cast<float*>(meta)[threadIdx.x] = xmax > 0.f ? ldexpf(1.f, e - 6) : 0.f;
  }
  __syncthreads();
  const int n_entries = kGroupFrags * M * 4;            // (fragment, batch row, t)
  for (int idx = threadIdx.x; idx < n_entries; idx += blockDim.x) {
    const int ft = idx & 3, m = (idx >> 2) % M, f = idx / (4 * M);
    int o[8];
    frag_k_offsets<BITS>(f % MPC, o);
    const int kb = k0 + (f / MPC) * CHUNK + ft * KL;
    const float up = s_up[m];
    int d[3][8];
    int sum[3] = {0, 0, 0};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float xv = (kb + o[i] < K) ? __ldg(x + (size_t)m * K + kb + o[i]) * up : 0.f;   // |xv| < 64
      const float d1 = rintf(xv);
      const float r1 = (xv - d1) * 128.f;                // exact: |xv - d1| <= 0.5
      const float d2 = rintf(r1);
      const float d3 = rintf((r1 - d2) * 128.f);
      d[0][i] = (int)d1; d[1][i] = (int)d2; d[2][i] = (int)d3;
      sum[0] += d[0][i]; sum[1] += d[1][i]; sum[2] += d[2][i];
    }
#pragma unroll
    for (int dig = 0; dig < 3; ++dig) {
      const int col = 3 * m + dig;
      frags[f][col >> 3][(col & 7) * 4 + ft] = make_uint2(pack_s8(d[dig][0], d[dig][1], d[dig][2], d[dig][3]),
                                                          pack_s8(d[dig][4], d[dig][5], d[dig][6], d[dig][7]));
      atomicAdd(&s_colsum[col], sum[dig]);
    }
  }
  __syncthreads();
  if (threadIdx.x < 48) reinterpret_cast<int*>(meta + 64)[threadIdx.x] = s_colsum[threadIdx.x];
}

// Main kernel: GROUPS groups of 512 k per block.
template <int BITS, int NT, int GROUPS>
__global__ void __launch_bounds__(kMmaWarps * 32)
qlinear_mma_kernel(const uint8_t* __restrict__ w, const float* __restrict__ scale, const float* __restrict__ bias,
                   const uint8_t* __restrict__ ws, int n_groups, float* __restrict__ y, int N, int K, int M) {
  constexpr int SLICE = GROUPS * kGroupK;
  constexpr int KL = BITS == 4 ? 32 : 16;          // k per lane per stage (one 16-byte unit)
  constexpr int CHUNK = 4 * KL;                    // k per stage: 128 / 64
  constexpr int MPC = CHUNK / 32;                  // MMAs per stage: 4 / 2
  constexpr int NFRAG = SLICE / 32;                // k32 fragments per slice
  constexpr int N_STAGES = SLICE / CHUNK;
  constexpr int STAGES_PER_GROUP = kGroupK / CHUNK;
  constexpr int OFFS = BITS == 4 ? 8 : 0;          // offset the unpacked nibbles carry
  extern __shared__ __align__(128) uint8_t qsm[];
  uint2 (*xs)[NT][32] = reinterpret_cast<uint2 (*)[NT][32]>(qsm);   // B fragments: [fragment][column tile][lane]
  uint8_t* ring = qsm + NFRAG * NT * 32 * sizeof(uint2) + (threadIdx.x >> 5) * kStages * kStageBytes;
  __shared__ float s_down[GROUPS][16];             // 2^(e-6) per group and batch row
  __shared__ int s_colsum[GROUPS][48];             // digit-column sums per group

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int k_slice0 = blockIdx.y * SLICE;
  const size_t row_bytes_ = (size_t)((K + 31) / 32 * 32) * BITS / 8;
  const int n_warp0 = blockIdx.x * kMmaRowsPerBlock + warp * kMmaRowsPerWarp;

  // cp.async sources / destinations of this lane: units lane, lane + 32, ... of a stage
  constexpr int UNITS_PER_LANE = kMmaRowsPerWarp * (kStageRowBytes / 16) / 32;   // 4
  const uint8_t* src[UNITS_PER_LANE];
  uint32_t dst[UNITS_PER_LANE];
#pragma unroll
  for (int i = 0; i < UNITS_PER_LANE; ++i) {
    const int unit = i * 32 + lane, row = unit >> 2, c = unit & 3;
    const int n = min(n_warp0 + row, N - 1);
    src[i] = w + (size_t)n * row_bytes_ + (size_t)k_slice0 * BITS / 8 + c * 16;
    dst[i] = (uint32_t)__cvta_generic_to_shared(ring) + row * kStageRowBytes + (c << 4);
  }
  auto issue_stage = [&](int st) {
    if (st < N_STAGES) {
#pragma unroll
      for (int i = 0; i < UNITS_PER_LANE; ++i)
        cp_async16(dst[i] + (st % kStages) * kStageBytes, src[i] + (size_t)st * kStageRowBytes);
    }
    cp_async_commit();
  };
  issue_stage(0);
  issue_stage(1);

  // Everything below reads what the digit pre-pass wrote (workspace, zeroed y): wait for it.
  // The two weight stages above are already in flight.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // third cp.async group: this slice's B fragments (contiguous in the workspace)
  {
    const uint8_t* fsrc = ws + (size_t)blockIdx.y * GROUPS * kGroupFrags * NT * 32 * sizeof(uint2);
    const uint32_t fdst = (uint32_t)__cvta_generic_to_shared(qsm);
    for (int u = threadIdx.x; u < NFRAG * NT * 32 * (int)sizeof(uint2) / 16; u += kMmaWarps * 32)
      cp_async16(fdst + u * 16, fsrc + (size_t)u * 16);
    cp_async_commit();
    const uint8_t* meta = ws + ws_frag_bytes(n_groups, NT) + (size_t)blockIdx.y * GROUPS * kMetaBytes;
    for (int i = threadIdx.x; i < GROUPS * 64; i += kMmaWarps * 32) {
      const int gi = i / 64, j = i - gi * 64;
      if (j < 16) s_down[gi][j] = reinterpret_cast<const float*>(meta + (size_t)gi * kMetaBytes)[j];
      else s_colsum[gi][j - 16] = reinterpret_cast<const int*>(meta + (size_t)gi * kMetaBytes + 64)[j - 16];
    }
  }


  // ---- unpack + integer MMA -----------------------------------------------------------------
  int acc[2][NT][4];
  float facc[2][NT][4];                              // sum over finished groups, in units of s_n
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int b = 0; b < NT; ++b)
#pragma unroll
      for (int c = 0; c < 4; ++c) { acc[a][b][c] = 0; facc[a][b][c] = 0.f; }

  const uint8_t* my_rows = ring + g * kStageRowBytes + (t << 4);
  for (int st = 0; st < N_STAGES; ++st) {
    issue_stage(st + 2);
    if (st == 0) {
      cp_async_wait<1>();                                          // stages 0, 1 and the B fragments
      __syncthreads();                                             // B fragments and group data: block-wide
    } else {
      cp_async_wait<2>();                                          // stage st has landed (for this lane)
      __syncwarp();                                                // weights: warp-private ring
    }
    const uint8_t* stage = my_rows + (st % kStages) * kStageBytes;
    uint4 q[4];                                                    // rows g, g+8 (tile 0), g+16, g+24 (tile 1)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      q[r] = *reinterpret_cast<const uint4*>(stage + r * 8 * kStageRowBytes);
      if (BITS == 4) {                                             // two's complement -> nibble + 8
        q[r].x ^= 0x88888888u; q[r].y ^= 0x88888888u; q[r].z ^= 0x88888888u; q[r].w ^= 0x88888888u;
      }
    }
#pragma unroll
    for (int j = 0; j < MPC; ++j) {
      uint32_t a[2][4];
#pragma unroll
      for (int tile = 0; tile < 2; ++tile) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const uint4& qq = q[tile * 2 + half];
          if (BITS == 4) {
            const uint32_t word = j == 0 ? qq.x : j == 1 ? qq.y : j == 2 ? qq.z : qq.w;
            a[tile][half] = word & 0x0F0F0F0Fu;                    // even nibbles -> a0 / a1
            a[tile][2 + half] = (word >> 4) & 0x0F0F0F0Fu;         // odd nibbles  -> a2 / a3
          } else {
            a[tile][half] = j == 0 ? qq.x : qq.z;
            a[tile][2 + half] = j == 0 ? qq.y : qq.w;
          }
        }
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const uint2 b = xs[st * MPC + j][nt][lane];
        mma_s8_16832(acc[0][nt], a[0][0], a[0][1], a[0][2], a[0][3], b.x, b.y);
        mma_s8_16832(acc[1][nt], a[1][0], a[1][1], a[1][2], a[1][3], b.x, b.y);
      }
    }
    __syncwarp();                                                  // the slot is refilled two iterations on
    if ((st + 1) % STAGES_PER_GROUP == 0) {
      // end of a group: the exact integer sums leave for float32 with the group's exponent.
      // D fragment: lane (g, t) holds rows g, g+8 and columns 2t, 2t+1 of tile nt; column
      // c = 3 m + digit contributes 2^(e-6) * 2^(-7 digit) * (S - 8 * colsum).
      const int gi = st / STAGES_PER_GROUP;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int col = nt * 8 + 2 * t + e;
          const int m = col / 3, dig = col - 3 * m;
          const float wgt = (m < M ? s_down[gi][m] : 0.f) * (dig == 0 ? 1.f : dig == 1 ? 0.0078125f : 0.00006103515625f);
          const int cs = OFFS * s_colsum[gi][col];
#pragma unroll
          for (int tile = 0; tile < 2; ++tile) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              facc[tile][nt][2 * half + e] = fmaf((float)(acc[tile][nt][2 * half + e] - cs), wgt, facc[tile][nt][2 * half + e]);
              acc[tile][nt][2 * half + e] = 0;
            }
          }
        }
      }
    }
  }
  cp_async_wait<0>();

  // ---- partial sums -> y -------------------------------------------------------------------
#pragma unroll
  for (int tile = 0; tile < 2; ++tile) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int n = n_warp0 + tile * 16 + half * 8 + g;
      if (n >= N) continue;
      const float s = scale[n];
      const float b = (blockIdx.y == 0 && bias) ? bias[n] : 0.f;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int col = nt * 8 + 2 * t + e;
          const int m = col / 3, dig = col - 3 * m;
          if (m >= M) continue;
          atomicAdd(y + (size_t)m * N + n, fmaf(facc[tile][nt][2 * half + e], s, dig == 0 ? b : 0.f));
        }
      }
    }
  }
}

}  // namespace

static int qlinear_nt(int M) {
  const int nt = (3 * M + 7) / 8;                  // 8-column tiles for 3 digit columns per batch row
  return nt <= 1 ? 1 : nt <= 2 ? 2 : nt <= 3 ? 3 : 6;
}

bool qlinear_mma_applicable(int N, int K, int bits, int M) {
  if (bits != 4 && bits != 8) return false;
  if (M < 1 || M > kMaxM) return false;
  if (K % kGroupK != 0) return false;              // whole exponent groups
  return (long long)N * K >= (1 << 20);            // small layers stay on the plain kernel
}

size_t qlinear_mma_workspace_bytes(int K, int M) {
  const int n_groups = K / kGroupK;
  return ws_frag_bytes(n_groups, qlinear_nt(M)) + (size_t)n_groups * kMetaBytes;
}

aiq_status_t launch_qlinear_mma(const LayerJob& job, int N, int K, int M, void* workspace, cudaStream_t s) {
  const int nt_t = qlinear_nt(M);
  const int n_groups = K / kGroupK;
  const int groups = (n_groups % 2 == 0 && nt_t <= 3) ? 2 : 1;   // k per block: 1024 or 512
  const dim3 grid((N + kMmaRowsPerBlock - 1) / kMmaRowsPerBlock, n_groups / groups);
  const uint8_t* w = job.w;
  const float* x = static_cast<const float*>(job.in);
  float* y = static_cast<float*>(job.out);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  LaunchScope scope(AIQ_KERNEL_QLINEAR, s, 2.0 * M * N * K,
                    (double)N * row_bytes(K, job.bits) + 4.0 * N + 4.0 * M * ((double)K + N));
#define AIQ_QMMA(BITS_, NT_, GR_)                                                                           \
  do {                                                                                                      \
    const int smem = GR_ * kGroupFrags * NT_ * 32 * (int)sizeof(uint2) + kMmaWarps * kStages * kStageBytes; \
    AIQ_ENSURE_DYNAMIC_SMEM((qlinear_mma_kernel<BITS_, NT_, GR_>), smem);                                   \
    qlinear_digits_kernel<BITS_, NT_><<<n_groups, 256, 0, s>>>(x, K, M, ws, n_groups, y, M * N);            \
    cudaLaunchConfig_t cfg = {};                                                                            \
    cfg.gridDim = grid; cfg.blockDim = dim3(kMmaWarps * 32); cfg.dynamicSmemBytes = smem; cfg.stream = s;   \
    cudaLaunchAttribute attr[1];                                                                            \
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                        \
    attr[0].val.programmaticStreamSerializationAllowed = 1;                                                 \
    cfg.attrs = attr; cfg.numAttrs = 1;                                                                     \
    const uint8_t* ws_c = ws;                                                                               \
    AIQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, qlinear_mma_kernel<BITS_, NT_, GR_>, w, job.scale, job.bias,      \
                                    ws_c, n_groups, y, N, K, M));                                           \
  } while (0)
#define AIQ_QMMA_BITS(BITS_)                                                                       \
  do {                                                                                             \
    if (nt_t == 1) { if (groups == 2) AIQ_QMMA(BITS_, 1, 2); else AIQ_QMMA(BITS_, 1, 1); }         \
    else if (nt_t == 2) { if (groups == 2) AIQ_QMMA(BITS_, 2, 2); else AIQ_QMMA(BITS_, 2, 1); }    \
    else if (nt_t == 3) { if (groups == 2) AIQ_QMMA(BITS_, 3, 2); else AIQ_QMMA(BITS_, 3, 1); }    \
    else AIQ_QMMA(BITS_, 6, 1);                                                                    \
  } while (0)
  if (job.bits == 4) AIQ_QMMA_BITS(4); else AIQ_QMMA_BITS(8);
#undef AIQ_QMMA_BITS
#undef AIQ_QMMA
  AIQ_LAUNCH_CHECK("qlinear_mma");
  count_launch();                                  // the digit pre-pass
  return AIQ_OK;
}

}  // namespace aiq
