// Dense 3x3 / 1x1 convolution on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
//   out[p][n] = act( s_n * sum_{tap,c} code[n][c][tap] * x[p @ tap][c] + b_n + res[p][n] )
//
// The activations are stored as the sum of two bfloat16 per element (ACT_SPLIT), one pixel
// = [hi(C) | lo(C)], rows padded physically (common.cuh).  The implicit GEMM has
//   M = 128 output pixels  (a tile of 16 padded rows x 8 columns),
//   N = Cout (16 / 32 / 64),
//   K = taps x 2C: the hi and the lo half of a pixel are two K-slices that meet the same
//       weights, so x = hi + lo costs two MMAs and loses nothing in the products
//       (integer codes |q| <= 128 are exact in bfloat16; accumulation is float32 in TMEM).
//
// Data movement per tile: for each horizontal tap t the producer warp issues one TMA load of
// an 18-row x 8-column x 2C box (rows j0-1 .. j0+16, columns c0+t-1 .. c0+t+6; out-of-range
// columns and rows arrive as zeros = the convolution's padding).  The box lands as 18 groups
// of 8 pixel rows in the canonical K-major swizzled layout, so the three vertical taps are
// the same buffer addressed one group further down: 3 loads feed 9 taps.  Weights arrive
// packed (4 or 8 bits) by one bulk copy per CTA and are expanded to bfloat16 in shared
// memory, in the swizzled layout the MMA reads.  One thread issues the MMAs; four warps
// drain the float32 accumulators from tensor memory, apply scale, bias, residual and
// activation, split the result into two bfloat16 and store it.  Two accumulator buffers let
// the epilogue of a tile overlap the MMAs of the next.  Stride-2 layers view the input as
// (column parity, column pair, row parity, row pair), which makes every tap a dense TMA box;
// they use one load and one ring stage per tap.
//
// Every wait is bounded: when a wait gives up the CTA raises an error word in global
// memory, every role falls through, tensor memory is released and the kernel returns.
#include "tc_ptx.cuh"

namespace aiq {

namespace {

// warp 0: TMA producer, warp 1: MMA issuer, then the epilogue warps: 2 per TMEM quarter, 4 where
// N = 64 (those kernels run one CTA per SM, so registers allow it, and their epilogue is the longest)
__host__ __device__ constexpr int tc_epilogue_warps_per_quarter(int n) { return n == 64 ? 4 : 2; }
__host__ __device__ constexpr int tc_threads(int n) { return (2 + 4 * tc_epilogue_warps_per_quarter(n)) * 32; }
constexpr int kRowsPerTile = 16;           // padded rows per tile
constexpr int kColsPerTile = 8;
constexpr int kBoxRows = kRowsPerTile + 2;

struct TcParams {
  int B, H, W;            // input geometry (output = input for stride 1, halved for stride 2)
  int Ho, Wo;
  int ks, stride, act;
  int n_stages;
  int K;                  // Cin * ks * ks (packed row length in elements)
  int ver_pair_rows;      // stride 2: row pairs per version of the input slot = capacity * (H + 2) / 2
  int cs_out;             // multi-piece kernels: channels of an output pixel (N per blockIdx.z)
  int32_t* error_flag;    // device word, set to 1 when a bounded wait expired
};


// 16-byte-unit XOR swizzle of a byte offset inside a tile whose base is aligned to the pattern
__device__ __forceinline__ uint32_t swizzle_off(uint32_t off, uint32_t mask) {
  return off ^ (((off >> 7) & mask) << 4);
}

template <int CS, int N>
struct TcLayout {
  static constexpr int PIX_BYTES = 4 * CS;                       // [hi | lo] bfloat16
  static constexpr int CW_BYTES = PIX_BYTES < 128 ? PIX_BYTES : 128;   // bytes per pixel row of one box
  static constexpr int CHUNKS = PIX_BYTES / CW_BYTES;
  static constexpr int GROUP_BYTES = 8 * CW_BYTES;
  static constexpr int CHUNK_BYTES = kBoxRows * GROUP_BYTES;
  static constexpr int STAGE_BYTES = CHUNKS * CHUNK_BYTES;
  static constexpr uint32_t A_LAYOUT = CW_BYTES == 128 ? 2u : 4u;
  static constexpr int W_ROW_BYTES = 2 * CS;                     // one weight row of one tap
  static constexpr uint32_t W_LAYOUT = W_ROW_BYTES == 128 ? 2u : (W_ROW_BYTES == 64 ? 4u : 6u);
  static constexpr uint32_t W_SWZ_MASK = W_ROW_BYTES == 128 ? 7u : (W_ROW_BYTES == 64 ? 3u : 1u);
  static constexpr int W_TAP_BYTES = N * W_ROW_BYTES;
  static constexpr int TMEM_COLS = 2 * N < 32 ? 32 : 2 * N;      // two accumulator buffers
};

// Offsets of the dynamic shared memory regions (base aligned to 1024 bytes)
template <int CS, int N>
struct TcSmem {
  using L = TcLayout<CS, N>;
  static __host__ __device__ constexpr int ring(int) { return 0; }
  static __host__ __device__ constexpr int weights(int stages) { return stages * L::STAGE_BYTES; }
  static __host__ __device__ constexpr int scale(int stages, int taps) { return weights(stages) + taps * L::W_TAP_BYTES; }
  static __host__ __device__ constexpr int bias(int stages, int taps) { return scale(stages, taps) + N * 4; }
  static __host__ __device__ constexpr int staging(int stages, int taps) { return (bias(stages, taps) + N * 4 + 127) / 128 * 128; }
  static __host__ __device__ constexpr int bars(int stages, int taps) { return staging(stages, taps) + 128 * 4 * N; }
  // barriers: full[stages], empty[stages], acc_full[2], acc_empty[2], wbar; then tmem ptr, abort flag
  static __host__ __device__ constexpr int total(int stages, int taps) { return bars(stages, taps) + (2 * stages + 5) * 8 + 16; }
};

// PIECES: bfloat16 pieces per weight: 1 (4- / 8-bit codes), 2 (half and float32 weights)
template <int CS, int N, int KS, int STRIDE, int PIECES>
__global__ void __launch_bounds__(tc_threads(N), (CS <= 32 && N <= 32) ? 2 : 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap in_map, TcParams p, const LayerJob* __restrict__ jobs) {
  using L = TcLayout<CS, N>;
  using S = TcSmem<CS, N>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // the runtime only promises 16-byte alignment of dynamic shared memory: align by hand
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const LayerJob job = jobs[blockIdx.y];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int taps = KS * KS;
  constexpr int T_FIRST = KS == 3 ? 0 : 1, T_LAST = KS == 3 ? 2 : 1;   // horizontal / vertical tap range
  const int stages = p.n_stages;

  uint8_t* ring = smem;
  uint8_t* wsm = smem + S::weights(stages);
  // 16- and 32-bit weights are not exact in one bfloat16: they are held as hi + lo, two bfloat16
  // pieces (hi = bf16(w), lo = bf16(w - hi): 16 significant bits, exact for a half, within 2^-17
  // of a float32 weight, the precision the activations are stored with), one weight tile per
  // piece and tap, and every MMA is issued once per piece into the same accumulator.  A third
  // piece does not pay: its products are 2^-16 of the sum and the float32 accumulation of the
  // tensor cores drops most of them (measured: all of them when few weights are non-zero).
  constexpr int pieces = PIECES;
  constexpr int wtaps = taps * pieces;           // weight tiles in shared memory
  // The multi-piece kernels hold at most N = 32 output channels' weights: a layer of 2N output
  // channels runs as two slices (blockIdx.z) that write their halves of every output pixel.
  constexpr bool SLICED = PIECES > 1;
  const int n_off = SLICED ? (int)blockIdx.z * N : 0;      // first output channel of this CTA
  const int cs_out = SLICED ? p.cs_out : N;                // channels of an output pixel
  float* s_scale = reinterpret_cast<float*>(smem + S::scale(stages, wtaps));
  float* s_bias = reinterpret_cast<float*>(smem + S::bias(stages, wtaps));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::bars(stages, wtaps));
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8 * stages;
  const uint32_t bar_acc_full = bar_empty + 8 * stages;
  const uint32_t bar_acc_empty = bar_acc_full + 16;
  const uint32_t bar_w = bar_acc_empty + 16;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * stages + 5);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  // Tiles.  Stride 1: 16 consecutive padded rows (image, y') x 8 columns, border rows included
  // (they are written as zeros).  Stride 2: 16 interior output rows x 8 output columns, taken
  // from IPT = 16 / Ho whole images when an image has fewer than 16 rows, or from one of the
  // RBI = Ho / 16 row blocks of an image; the two border rows are zero-filled on the side.
  const int rows_total = p.B * (p.H + 2);               // stride 1: padded rows of the batch
  const int ipt = STRIDE == 2 && p.Ho < kRowsPerTile ? kRowsPerTile / p.Ho : 1;
  const int rows_per_img = STRIDE == 2 ? (p.Ho < kRowsPerTile ? p.Ho : kRowsPerTile) : 0;
  const int rbi = STRIDE == 2 && p.Ho > kRowsPerTile ? p.Ho / kRowsPerTile : 1;
  const int n_rb = STRIDE == 2 ? ((p.B + ipt - 1) / ipt) * rbi : (rows_total + kRowsPerTile - 1) / kRowsPerTile;
  const int n_cb = p.Wo / kColsPerTile;
  const int n_tiles = n_rb * n_cb;

  // ---- set-up -----------------------------------------------------------------------------
  if (tid == 0) {
    for (int i = 0; i < stages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_acc_full + 8 * i, 1);
      mbar_init(bar_acc_empty + 8 * i, 4 * tc_epilogue_warps_per_quarter(N));   // one arrival per epilogue warp
    }
    mbar_init(bar_w, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 1) {
    tmem_alloc(smem_u32(s_tmem), L::TMEM_COLS);
    tmem_relinquish();
  }
  // packed weights: one bulk copy into the (still unused) ring, then expansion to bfloat16
  const int kpad = (p.K + 31) / 32 * 32;
  const uint32_t wrow_bytes = (uint32_t)kpad * job.bits / 8;
  const uint32_t packed_bytes = wrow_bytes * N;
  if (tid == 0) {
    mbar_expect_tx(bar_w, packed_bytes);
    bulk_load(smem_u32(ring), job.w + (size_t)n_off * wrow_bytes, packed_bytes, bar_w);
  }
  for (int i = tid; i < N; i += tc_threads(N)) {
    s_scale[i] = job.scale[n_off + i];
    s_bias[i] = job.bias[n_off + i];
  }
  bool alive = mbar_wait_warp(bar_w, 0, s_abort, p.error_flag);
  if (alive) {
    const int units_per_row = CS / 8;                         // 16-byte units of one weight row
    const int total_units = taps * N * units_per_row;
    for (int u = tid; u < total_units; u += tc_threads(N)) {
      const int c8 = u % units_per_row;
      const int n = (u / units_per_row) % N;
      const int tap = u / (units_per_row * N);
      const uint8_t* row = ring + (size_t)n * wrow_bytes;
      const uint32_t off = swizzle_off((uint32_t)(n * L::W_ROW_BYTES + c8 * 16), L::W_SWZ_MASK);
      if constexpr (PIECES > 1) {
        uint32_t pk[PIECES][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int k = (c8 * 8 + j) * taps + tap;
          float w = job.bits == 16 ? __half2float(reinterpret_cast<const __half*>(row)[k])
                                   : reinterpret_cast<const float*>(row)[k];
#pragma unroll
          for (int pc = 0; pc < PIECES; ++pc) {
            const __nv_bfloat16 h = __float2bfloat16_rn(w);
            w -= __bfloat162float(h);                            // exact: the remainder of the rounding
            const uint32_t hb = (uint32_t)__bfloat16_as_ushort(h);
            if (j & 1) pk[pc][j >> 1] |= hb << 16; else pk[pc][j >> 1] = hb;
          }
        }
#pragma unroll
        for (int pc = 0; pc < PIECES; ++pc)
          *reinterpret_cast<uint4*>(wsm + (size_t)(pc * taps + tap) * L::W_TAP_BYTES + off) =
              make_uint4(pk[pc][0], pk[pc][1], pk[pc][2], pk[pc][3]);
      } else {
        uint32_t packed[4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int k = (c8 * 8 + j) * taps + tap;             // element index in the (c, r, t) ordered row
          int code;
          if (job.bits == 8) {
            code = (int)(int8_t)row[k];
          } else {
            const int byte = row[k >> 1];
            const int nib = (k & 1) ? (byte >> 4) : (byte & 0xF);
            code = (nib ^ 8) - 8;
          }
          const uint32_t h = (uint32_t)__bfloat16_as_ushort(__int2bfloat16_rn(code));
          if (j & 1) packed[j >> 1] |= h << 16; else packed[j >> 1] = h;
        }
        *reinterpret_cast<uint4*>(wsm + (size_t)tap * L::W_TAP_BYTES + off) =
            make_uint4(packed[0], packed[1], packed[2], packed[3]);
      }
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // expanded weights -> visible to the MMA
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  alive = alive && (*s_abort == 0);            // the same answer in every thread

  // ---- roles ------------------------------------------------------------------------------
  if (warp == 0) {
    if (lane == 0 && alive) {
      uint32_t stage = 0, phase = 0;
      uint32_t issued = 0, issued_phase = 0;       // per stage: a load was issued / parity of the last one
      for (int tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x) {
        const int rb = tile / n_cb, cb = tile - rb * n_cb;
        if (STRIDE == 1) {
          for (int t = T_FIRST; t <= T_LAST && alive; ++t) {
            alive = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
            if (!alive) break;
            issued |= 1u << stage;
            issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
            mbar_expect_tx(bar_full + 8 * stage, L::STAGE_BYTES);
#pragma unroll
            for (int ch = 0; ch < L::CHUNKS; ++ch)
              tma_load_4d(smem_u32(ring) + stage * L::STAGE_BYTES + ch * L::CHUNK_BYTES, &in_map,
                          bar_full + 8 * stage, ch * 64, cb * kColsPerTile + t - 1, rb * kRowsPerTile - 1,
                          job.in_version);
            if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
          }
        } else {
          // One stage per tap: the map views the input as (channel, column parity, column pair,
          // row parity, row pair), so tap (r, t) of a stride-2 window is a dense box.  Input
          // padded row 2*oy + r = pair oy + (r >> 1), parity r & 1; input column 2*ox + t - 1 =
          // pair ox + ((t - 1) >> 1), parity (t - 1) & 1 (pair -1 is out of range: zeros).
          const int b0 = (rb / rbi) * ipt, oy0 = (rb % rbi) * kRowsPerTile;
          for (int t = T_FIRST; t <= T_LAST && alive; ++t) {
            for (int r = T_FIRST; r <= T_LAST && alive; ++r) {
              alive = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
              if (!alive) break;
              issued |= 1u << stage;
              issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
              mbar_expect_tx(bar_full + 8 * stage, L::CHUNKS * kRowsPerTile * L::GROUP_BYTES);
              for (int img = 0; img < ipt; ++img) {
                const int pair_row = job.in_version * p.ver_pair_rows + (b0 + img) * ((p.H + 2) >> 1) + oy0 + (r >> 1);
#pragma unroll
                for (int ch = 0; ch < L::CHUNKS; ++ch)
                  tma_load_5d(smem_u32(ring) + stage * L::STAGE_BYTES + ch * L::CHUNK_BYTES +
                                  img * rows_per_img * L::GROUP_BYTES,
                              &in_map, bar_full + 8 * stage, ch * 64, (t - 1) & 1, cb * kColsPerTile + ((t - 1) >> 1),
                              r & 1, pair_row);
              }
              if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
            }
          }
        }
      }
      // copies in flight must land before the CTA exits: wait (bounded) for the last load
      // of every stage.  On the normal path the consumer has seen them all and this returns
      // at once; it matters when another role gave up.
      for (int i = 0; i < stages; ++i)
        if (issued & (1u << i)) {
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_full + 8 * i, (issued_phase >> i) & 1u) && clock64() - t0 < kWaitLimitCycles) {}
        }
    }
  } else if (warp == 1) {
    if (alive) {                                   // all 32 lanes, converged (see umma_bf16)
      // instruction descriptor: D float32, A and B bfloat16, both K-major, M = 128, N
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((128u >> 4) << 24);
      // Shared-memory descriptors differ only in their start address, so the upper words are
      // constants and every MMA costs one add per operand: the tiles are small (8-32 tensor
      // cycles each), issue overhead would otherwise dominate.
      constexpr uint32_t A_HI = (uint32_t)(L::GROUP_BYTES >> 4) | (1u << 14) | (L::A_LAYOUT << 29);
      constexpr uint32_t B_HI = (uint32_t)((8 * L::W_ROW_BYTES) >> 4) | (1u << 14) | (L::W_LAYOUT << 29);
      constexpr uint32_t LBO_FIELD = 1u << 16;
      const uint32_t w_lo0 = (smem_u32(wsm) >> 4) | LBO_FIELD;
      uint32_t stage = 0, phase = 0;
      int it = 0;
      for (int tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x, ++it) {
        const int buf = it & 1;
        alive = mbar_wait_warp(bar_acc_empty + 8 * buf, ((it >> 1) & 1) ^ 1u, s_abort, p.error_flag);
        if (!alive) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * N);
#pragma unroll
        for (int t = T_FIRST; t <= T_LAST; ++t) {
          if (STRIDE == 1) {
            if (!alive) break;
            alive = mbar_wait_warp(bar_full + 8 * stage, phase, s_abort, p.error_flag);
            if (!alive) break;
            tc_fence_after();
          }
          const uint32_t a_lo1 = ((smem_u32(ring) + stage * L::STAGE_BYTES) >> 4) | LBO_FIELD;
#pragma unroll
          for (int r = T_FIRST; r <= T_LAST; ++r) {
            uint32_t a_lo0 = a_lo1;
            if (STRIDE == 2) {                     // every tap has a stage of its own
              if (!alive) break;
              alive = mbar_wait_warp(bar_full + 8 * stage, phase, s_abort, p.error_flag);
              if (!alive) break;
              tc_fence_after();
              a_lo0 = ((smem_u32(ring) + stage * L::STAGE_BYTES) >> 4) | LBO_FIELD;
            }
            const int tap = KS == 3 ? r * 3 + t : 0;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
#pragma unroll
              for (int kk = 0; kk < CS / 16; ++kk) {
                const int byte = (part * CS + kk * 16) * 2;              // offset inside the pixel
                const uint32_t a_off = (byte / L::CW_BYTES) * L::CHUNK_BYTES + (STRIDE == 1 ? r * L::GROUP_BYTES : 0) +
                                       (byte % L::CW_BYTES);
                const uint64_t adesc = ((uint64_t)A_HI << 32) | (uint64_t)(a_lo0 + (a_off >> 4));
                const uint32_t b_lo = w_lo0 + ((tap * L::W_TAP_BYTES + kk * 32) >> 4);
                const uint32_t accumulate = (t == T_FIRST && r == T_FIRST && part == 0 && kk == 0) ? 0u : 1u;
                umma_bf16(d_tmem, adesc, ((uint64_t)B_HI << 32) | (uint64_t)b_lo, idesc, accumulate);
#pragma unroll
                for (int pc = 1; pc < pieces; ++pc)             // the lo piece of 16- / 32-bit weights
                  umma_bf16(d_tmem, adesc,
                            ((uint64_t)B_HI << 32) | (uint64_t)(b_lo + (uint32_t)((pc * taps * L::W_TAP_BYTES) >> 4)),
                            idesc, 1u);
              }
            }
            if (STRIDE == 2) {
              umma_commit(bar_empty + 8 * stage);
              if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
            }
          }
          if (STRIDE == 1) {
            umma_commit(bar_empty + 8 * stage);        // the stage is free once these MMAs retire
            if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
          }
        }
        if (alive) umma_commit(bar_acc_full + 8 * buf);
      }
    }
  } else {
    // Epilogue: TMEM lanes 32q .. 32q+31 (tile rows 4q .. 4q+3, 8 pixels each) belong to the
    // EPW (2, or 4 at N = 64) warps with warp index mod 4 = q; warp h of them takes 1/EPW of the
    // output channels.  The arithmetic of the epilogue (scale, bias, residual, activation, the
    // split into two bfloat16) is a long dependent chain per tile, so it is spread over many
    // warps; with four in all the tensor cores waited for the epilogue more than half of the time.
    // A lane owns one pixel for the arithmetic, but a pixel is only 4N bytes, so per-lane global
    // accesses would touch 32 cache lines per instruction.  Instead the 32 pixels of a quarter
    // are staged in shared memory: the residual rows go into the staging buffer with coalesced
    // 16-byte accesses, the result overwrites them in place, and the finished rows leave with
    // coalesced stores (a row of 8 pixels is 32N contiguous bytes).  Each warp moves 4/EPW of
    // the quarter's four rows; two named-barrier syncs per tile order the warps of a quarter
    // (ids 1 .. 4).  16-byte units are XOR-swizzled so that both access patterns are free of
    // bank conflicts.
    const int q = warp & 3;
    constexpr int EPW = tc_epilogue_warps_per_quarter(N);   // warps that share a quarter
    constexpr int RPW = 4 / EPW;                             // rows of the quarter each of them moves
    const int h = (warp - 2) >> 2;
    const int m = q * 32 + lane;                       // row of the tile: pixel (g, wl)
    const int g = m >> 3;
    constexpr int PIXB = 4 * N;                        // bytes of one output pixel
    constexpr int UNITS = PIXB / 16;                   // 16-byte units per pixel (4, 8, 16)
    constexpr int KEY_SHIFT = PIXB < 128 ? 1 : 0;      // N = 16: two pixels share a 128-byte window
    constexpr int KEY_MASK = (UNITS < 8 ? UNITS : 8) - 1;
    constexpr int CW = N >= 32 ? 16 : 8;               // accumulator columns per chunk
    constexpr int NCH = N / (EPW * CW);                // chunks per warp (1)
    uint8_t* stg = smem + S::staging(stages, wtaps) + q * 32 * PIXB;
    uint8_t* my_row = stg + lane * PIXB;
    const int my_key = (lane >> KEY_SHIFT) & KEY_MASK;
    const uint32_t pair_bar = 1u + (uint32_t)q;
    // Global layout of a row of 8 output pixels: pixel pitch 4 cs_out bytes, [hi(cs_out) | lo(cs_out)].
    // Staging unit u of the row (pixel u / UNITS, unit u % UNITS of [hi(N) | lo(N)]) lands at
    // unit_off(u) bytes from the row's first pixel; without slices that is simply 16 u.
    const size_t pix_pitch = SLICED ? (size_t)4 * cs_out : (size_t)PIXB;
    auto unit_off = [&](int u) -> size_t {
      if (!SLICED) return (size_t)u * 16;
      const int px = u / UNITS, uu = u % UNITS;
      const int half = uu >= UNITS / 2 ? 1 : 0;
      return (size_t)px * pix_pitch + 2 * n_off + (half ? 2 * cs_out : 0) + (uu - half * (UNITS / 2)) * 16;
    };
    // output row (image, padded y) of group gi of a tile, or -1 when the group is past the batch
    auto tile_row = [&](int t, int gi) -> int {
      const int trb = t / n_cb;
      if (STRIDE == 1) {
        const int jr = trb * kRowsPerTile + gi;
        return jr < rows_total ? jr : -1;
      }
      const int rpi = STRIDE == 2 ? rows_per_img : 1;    // (stride 1 never gets here)
      const int tb0 = (trb / rbi) * ipt, toy0 = (trb % rbi) * kRowsPerTile;
      const int img = gi / rpi;
      const int bb = tb0 + img;
      return bb < p.B ? bb * (p.Ho + 2) + toy0 + (gi - img * rpi) + 1 : -1;
    };
    // The residual rows of the next tile are fetched into registers while the current tile is
    // computed and stored, so their memory latency is off the critical path of the epilogue.
    constexpr int RPL = (8 * UNITS + 31) / 32;         // 16-byte units per lane and row
    uint4 rpre[RPW][RPL];
    auto fetch_residual = [&](int t) {
      const int tcb = t % n_cb;
#pragma unroll
      for (int ii = 0; ii < RPW; ++ii) {
        const int jr = tile_row(t, q * 4 + RPW * h + ii);
        const uint8_t* src = static_cast<const uint8_t*>(job.res) +
                             ((size_t)(jr < 0 ? 0 : jr) * p.Wo + tcb * kColsPerTile) * pix_pitch;
#pragma unroll
        for (int k = 0; k < RPL; ++k) {
          const int u = lane + 32 * k;
          rpre[ii][k] = (jr >= 0 && u < 8 * UNITS) ? __ldg(reinterpret_cast<const uint4*>(src + unit_off(u)))
                                                   : make_uint4(0u, 0u, 0u, 0u);
        }
      }
    };
    if (job.res && (int)blockIdx.x < n_tiles && alive) fetch_residual(blockIdx.x);
    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x, ++it) {
      const int buf = it & 1;
      const int rb = tile / n_cb, cb = tile - rb * n_cb;
      const int b0 = STRIDE == 2 ? (rb / rbi) * ipt : 0, oy0 = STRIDE == 2 ? (rb % rbi) * kRowsPerTile : 0;
      auto out_row = [&](int gi) -> int { return tile_row(tile, gi); };
      // (1) residual rows (fetched during the previous tile) -> staging: this warp's two rows
      if (job.res) {
#pragma unroll
        for (int ii = 0; ii < RPW; ++ii) {
          const int i = RPW * h + ii;
#pragma unroll
          for (int k = 0; k < RPL; ++k) {
            const int u = lane + 32 * k;
            if (u < 8 * UNITS) {
              const int pl = i * 8 + u / UNITS, uu = u % UNITS;
              *reinterpret_cast<uint4*>(stg + pl * PIXB + ((uu ^ ((pl >> KEY_SHIFT) & KEY_MASK)) << 4)) = rpre[ii][k];
            }
          }
        }
      }
      mbar_wait_warp(bar_acc_full + 8 * buf, (it >> 1) & 1, s_abort, p.error_flag);   // false => *s_abort is set
      // all warps of the quarter, unconditionally: the partners' residual rows are in place and their
      // stores of the previous tile have left the staging rows
      asm volatile("bar.sync %0, %1;" ::"r"(pair_bar), "n"(32 * EPW) : "memory");
      alive = *s_abort == 0;                      // the same answer in every warp of the quarter
      if (!alive) break;
      if (job.res && tile + (int)gridDim.x < n_tiles) fetch_residual(tile + gridDim.x);
      tc_fence_after();
      bool interior = true;                       // stride 2 tiles hold interior rows only
      if (STRIDE == 1) {
        const int j = rb * kRowsPerTile + g;             // padded row (image, y')
        const int yp = j % (p.H + 2);
        interior = yp >= 1 && yp <= p.H;
      }
      const bool use_res = job.res != nullptr && interior;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * N);
      uint32_t v[NCH][CW];
#pragma unroll
      for (int ch = 0; ch < NCH; ++ch) {
        const int c0 = (EPW * ch + h) * CW;
        if (CW == 16) tmem_ld16(taddr + c0, v[ch]); else tmem_ld8(taddr + c0, v[ch]);
      }
      tmem_ld_wait();
      // the accumulator values are in registers: hand the buffer back before the arithmetic
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
#pragma unroll
      for (int ch = 0; ch < NCH; ++ch) {
        const int c0 = (EPW * ch + h) * CW;
#pragma unroll
        for (int u8 = 0; u8 < CW / 8; ++u8) {
          // the 16-byte units of this pixel that hold columns c0 + 8 u8 .. + 7: one of hi, one of lo
          const int cc = c0 + 8 * u8;
          uint4* ph = reinterpret_cast<uint4*>(my_row + (((cc / 8) ^ my_key) << 4));
          uint4* pl = reinterpret_cast<uint4*>(my_row + ((((N + cc) / 8) ^ my_key) << 4));
          uint32_t rh[4] = {0, 0, 0, 0}, rl[4] = {0, 0, 0, 0};
          if (use_res) {
            const uint4 a = *ph, l = *pl;
            rh[0] = a.x; rh[1] = a.y; rh[2] = a.z; rh[3] = a.w;
            rl[0] = l.x; rl[1] = l.y; rl[2] = l.z; rl[3] = l.w;
          }
          const float4 sc0 = *reinterpret_cast<const float4*>(s_scale + cc), sc1 = *reinterpret_cast<const float4*>(s_scale + cc + 4);
          const float4 bi0 = *reinterpret_cast<const float4*>(s_bias + cc), bi1 = *reinterpret_cast<const float4*>(s_bias + cc + 4);
          const float sc[8] = {sc0.x, sc0.y, sc0.z, sc0.w, sc1.x, sc1.y, sc1.z, sc1.w};
          const float bi[8] = {bi0.x, bi0.y, bi0.z, bi0.w, bi1.x, bi1.y, bi1.z, bi1.w};
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int e = 0; e < 8; e += 2) {
            float u0 = 0.f, u1 = 0.f;
            if (interior) {
              u0 = fmaf(__uint_as_float(v[ch][8 * u8 + e]), sc[e], bi[e]);
              u1 = fmaf(__uint_as_float(v[ch][8 * u8 + e + 1]), sc[e + 1], bi[e + 1]);
              // a bfloat16 is the upper half of a float: residual = hi + lo
              u0 += __uint_as_float(rh[e >> 1] << 16) + __uint_as_float(rl[e >> 1] << 16);
              u1 += __uint_as_float(rh[e >> 1] & 0xFFFF0000u) + __uint_as_float(rl[e >> 1] & 0xFFFF0000u);
              u0 = apply_act(u0, p.act);
              u1 = apply_act(u1, p.act);
            }
            split_pair(u0, u1, hi[e >> 1], lo[e >> 1]);
          }
          *ph = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *pl = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      }
      // every column of the quarter's rows is final once the partner is here too
      asm volatile("bar.sync %0, %1;" ::"r"(pair_bar), "n"(32 * EPW) : "memory");
      // (3) staging -> global, one row of 8 pixels (32N contiguous bytes) at a time
#pragma unroll
      for (int ii = 0; ii < RPW; ++ii) {
        const int i = RPW * h + ii;
        const int jr = out_row(q * 4 + i);
        if (jr >= 0) {
          uint8_t* dst = static_cast<uint8_t*>(job.out) + ((size_t)jr * p.Wo + cb * kColsPerTile) * pix_pitch;
#pragma unroll
          for (int u = lane; u < 8 * UNITS; u += 32) {
            const int pl = i * 8 + u / UNITS, uu = u % UNITS;
            *reinterpret_cast<uint4*>(dst + unit_off(u)) =
                *reinterpret_cast<const uint4*>(stg + pl * PIXB + ((uu ^ ((pl >> KEY_SHIFT) & KEY_MASK)) << 4));
          }
        }
      }
      if (STRIDE == 2) {
        // zero border rows of the output images this tile touches (rows 0 and Ho + 1)
        const bool top = oy0 == 0, bottom = oy0 + rows_per_img == p.Ho;
        for (int img = q + 4 * h; img < ipt; img += 4 * EPW) {
          const int bb = b0 + img;
          if (bb >= p.B) break;
          for (int side = 0; side < 2; ++side) {
            if (side == 0 ? !top : !bottom) continue;
            const int jr = bb * (p.Ho + 2) + (side == 0 ? 0 : p.Ho + 1);
            uint8_t* dst = static_cast<uint8_t*>(job.out) + ((size_t)jr * p.Wo + cb * kColsPerTile) * pix_pitch;
            for (int u = lane; u < 8 * UNITS; u += 32)
              *reinterpret_cast<uint4*>(dst + unit_off(u)) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      __syncwarp();                                   // this warp's staging rows are reused by the next tile
    }
  }

  // ---- teardown -----------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, L::TMEM_COLS);
  }
}

// ---- host side ------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* sym = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(sym);
  return fn;
}

template <int CS, int N, int KS, int STRIDE, int PIECES>
aiq_status_t launch_tc(const ConvGeom& g, const CUtensorMap& map, const LayerJob* jobs_dev, int n_jobs,
                       int batch_capacity, int32_t* error_flag, double weight_bytes, int weight_bits, cudaStream_t s) {
  using L = TcLayout<CS, N>;
  using S = TcSmem<CS, N>;
  const int taps = g.ks * g.ks * PIECES;         // weight tiles held in shared memory
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  const int smem_limit = props.smem_optin, n_sms = props.n_sms;
  // Shared memory decides how many CTAs share an SM.  More resident CTAs hide the latency of
  // a tile's load -> MMA -> epilogue chain better than a deeper ring does, so prefer two
  // CTAs with at least 4 stages, then one with as many stages as fit (at most 6).
  const int sm_budget = smem_limit + 1024;                 // per-SM capacity = opt-in block limit + 1 KB
  constexpr int occ_cap = (CS <= 32 && N <= 32) ? 2 : 1;   // what __launch_bounds__ of the kernel allows
  int stages = 0;
  for (int want = occ_cap; want >= 1 && !stages; --want) {
    const int per_cta = sm_budget / want - 1024;           // every block also reserves 1 KB
    for (int st = 6; st >= (want > 1 ? 4 : (PIECES > 1 ? 2 : 3)); --st)
      if (S::total(st, taps) + 1024 <= per_cta && S::total(st, taps) + 1024 <= smem_limit) { stages = st; break; }
  }
  if (!stages)
    return set_error(AIQ_ERR_SHAPE, "conv_tc: shared memory for %d taps does not fit (%d bytes available)", taps, smem_limit);
  const int smem_bytes = S::total(stages, taps) + 1024;
  const int packed = N * (int)row_bytes(g.K, weight_bits <= 8 ? 8 : weight_bits);
  if (packed > stages * L::STAGE_BYTES)
    return set_error(AIQ_ERR_SHAPE, "conv_tc: packed weights (%d bytes) exceed the staging ring", packed);
  AIQ_ENSURE_DYNAMIC_SMEM((conv_tc_kernel<CS, N, KS, STRIDE, PIECES>), smem_limit);
  TcParams p = {};
  p.B = g.B; p.H = g.H; p.W = g.W; p.Ho = g.Ho; p.Wo = g.Wo; p.ks = g.ks; p.stride = g.stride; p.act = g.act;
  p.n_stages = stages; p.K = g.K; p.error_flag = error_flag;
  p.ver_pair_rows = batch_capacity * (g.H + 2) / 2;
  p.cs_out = g.Cout;
  const int slices = g.Cout / N;                 // 1, or 2 output-channel slices (multi-piece kernels)
  int n_tiles;
  if (STRIDE == 1) {
    n_tiles = ((g.B * (g.H + 2) + kRowsPerTile - 1) / kRowsPerTile) * (g.Wo / kColsPerTile);
  } else {
    const int ipt = g.Ho < kRowsPerTile ? kRowsPerTile / g.Ho : 1;
    const int rbi = g.Ho > kRowsPerTile ? g.Ho / kRowsPerTile : 1;
    n_tiles = ((g.B + ipt - 1) / ipt) * rbi * (g.Wo / kColsPerTile);
  }
  // resident CTAs per SM: shared memory, and at most two where the kernel is compiled for two
  // (10 warps of up to 96 registers each), else one
  int occ = sm_budget / (smem_bytes + 1024);
  occ = occ > occ_cap ? occ_cap : (occ < 1 ? 1 : occ);
  // All CTAs of the launch should be resident at once (a second wave would run nearly alone):
  // split the resident capacity evenly over the jobs, rounding down.
  int ctas = (n_sms * occ) / (n_jobs * slices);
  if (ctas > n_tiles) ctas = n_tiles;
  if (ctas < 1) ctas = 1;
  {
    LaunchScope scope(AIQ_KERNEL_CONV_TC, s,
                      2.0 * g.B * g.Ho * g.Wo * g.Cout * (double)(g.ks * g.ks * g.Cin) * n_jobs,
                      weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W +
                                                     (double)g.B * g.Ho * g.Wo * g.Cout));
    conv_tc_kernel<CS, N, KS, STRIDE, PIECES><<<dim3(ctas, n_jobs, slices), tc_threads(N), smem_bytes, s>>>(map, p, jobs_dev);
  }
  AIQ_LAUNCH_CHECK("conv_tc");
  return AIQ_OK;
}

}  // namespace

}  // namespace aiq

#include "conv_pw_tc.cuh"
#include "qlinear_tc.cuh"

namespace aiq {

bool conv_pw_tc_eligible(const ConvGeom& g) {
  if (g.in_is_nchw || g.act_format != ACT_SPLIT) return false;
  if (g.ks != 1 || g.pad != 0 || g.stride != 1) return false;
  if (g.Cin % 8 != 0 || g.Cin < 16) return false;
  return true;
}

aiq_status_t conv_pw_tc_encode_map(const ConvGeom& g, const void* slot_base, int batch_capacity, int n_versions,
                                   void* map_out) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  // (channel within a half, hi | lo, pixel over all versions)
  const cuuint64_t pixels = (cuuint64_t)n_versions * batch_capacity * (g.H + 2) * g.W;
  cuuint64_t dims[3] = {(cuuint64_t)g.Cs_in, 2, pixels};
  cuuint64_t strides[2] = {2ull * g.Cs_in, 4ull * g.Cs_in};
  cuuint32_t box[3] = {(cuuint32_t)kPwChunk, 1u, 128u};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(static_cast<CUtensorMap*>(map_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(slot_base),
                   dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled (pointwise) failed with code %d", (int)r);
  return AIQ_OK;
}

aiq_status_t conv_pw_tc_encode_out_map(const ConvGeom& g, const void* slot_base, int batch_capacity, int n_versions,
                                       void* map_out) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  // (channel within a half, hi | lo, pixel of a version, version): stores are clipped at the
  // padded channel count and at the capacity of a version
  const cuuint64_t pixels = (cuuint64_t)batch_capacity * (g.Ho + 2) * g.Wo;
  cuuint64_t dims[4] = {(cuuint64_t)g.Cs_out, 2, pixels, (cuuint64_t)n_versions};
  cuuint64_t strides[3] = {2ull * g.Cs_out, 4ull * g.Cs_out, 4ull * g.Cs_out * pixels};
  cuuint32_t box[4] = {(cuuint32_t)kPwChunk, 1u, 128u, 1u};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(static_cast<CUtensorMap*>(map_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(slot_base),
                   dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled (pointwise store) failed with code %d", (int)r);
  return AIQ_OK;
}

aiq_status_t launch_conv_pw_tc(const ConvGeom& g, const void* map, const void* out_map, const LayerJob* jobs_dev, int n_jobs,
                               int batch_capacity, int32_t* error_flag, double weight_bytes, int weight_bits, cudaStream_t s) {
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  const int smem_limit = props.smem_optin, n_sms = props.n_sms;
  AIQ_ENSURE_DYNAMIC_SMEM(conv_pw_tc_kernel, smem_limit);
  PwParams p = {};
  p.P = g.B * (g.H + 2) * g.W; p.H = g.H; p.W = g.W;
  p.Cin = g.Cin; p.Cs_in = g.Cs_in; p.Cout = g.Cout; p.Cs_out = g.Cs_out;
  // Output-channel tiles of 128 or of 64 channels (the store box is 64 channels wide, so a tile
  // is a whole number of boxes; only the last tile may be narrower).  A layer's CTAs are split
  // evenly over its tiles, so its time goes with (tile width) / (CTAs per tile): 144 channels
  // run as 64 + 64 + 16 rather than 128 + 16, 576 as 9 x 64 rather than 4 x 128 + 64.
  p.pieces = weight_bits > 8 ? 2 : 1;
  if (g.Cs_out <= 128 && !(p.pieces == 2 && g.Cs_out > 64)) {
    p.Nt = g.Cs_out;
  } else if (p.pieces == 2) {
    p.Nt = 64;                                   // two weight tiles per stage: narrower tiles keep three stages
  } else {
    auto cost = [&](int nt) {
      const int per_tile = n_sms / (n_jobs * ((g.Cs_out + nt - 1) / nt));
      return (double)nt / (per_tile > 0 ? per_tile : 1);
    };
    p.Nt = cost(64) < cost(128) ? 64 : 128;
  }
  p.n_ntiles = (g.Cs_out + p.Nt - 1) / p.Nt;
  p.act = g.act;
  p.ver_pixels = (long long)batch_capacity * (g.H + 2) * g.W;
  p.error_flag = error_flag;
  int stages = 4;
  while (stages > 2 && pw_smem_bytes(p.Nt, stages, p.pieces) + 1024 > smem_limit) --stages;
  if (pw_smem_bytes(p.Nt, stages, p.pieces) + 1024 > smem_limit)
    return set_error(AIQ_ERR_SHAPE, "conv_pw_tc: %d bytes of shared memory needed", pw_smem_bytes(p.Nt, stages, p.pieces) + 1024);
  p.n_stages = stages;
  const int smem_bytes = pw_smem_bytes(p.Nt, stages, p.pieces) + 1024;
  const int n_tiles = (p.P + 127) / 128;
  int ctas = n_sms / (n_jobs * p.n_ntiles);
  if (ctas > n_tiles) ctas = n_tiles;
  if (ctas < 1) ctas = 1;
  const CUtensorMap& m = *static_cast<const CUtensorMap*>(map);
  const CUtensorMap& mo = *static_cast<const CUtensorMap*>(out_map);
  {
    LaunchScope scope(AIQ_KERNEL_CONV_TC, s, 2.0 * g.B * g.Ho * g.Wo * g.Cout * (double)g.Cin * n_jobs,
                      weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W + (double)g.B * g.Ho * g.Wo * g.Cout));
    conv_pw_tc_kernel<<<dim3(ctas, n_jobs * p.n_ntiles), kPwThreads, smem_bytes, s>>>(m, mo, p, jobs_dev);
  }
  AIQ_LAUNCH_CHECK("conv_pw_tc");
  return AIQ_OK;
}

bool conv_tc_eligible(const ConvGeom& g) {
  if (g.in_is_nchw || g.act_format != ACT_SPLIT) return false;
  if (!((g.ks == 3 && g.pad == 1) || (g.ks == 1 && g.pad == 0))) return false;
  if (g.stride != 1 && g.stride != 2) return false;
  if (g.Cin != 16 && g.Cin != 32 && g.Cin != 64) return false;
  if (g.Cout != 16 && g.Cout != 32 && g.Cout != 64) return false;
  if (g.Wo % kColsPerTile != 0) return false;
  if (g.stride == 2) {
    // whole images (or whole 16-row blocks of an image) must tile the 16 rows of a tile
    if ((g.H & 1) || (g.W & 1)) return false;
    if (!(g.Ho % kRowsPerTile == 0 || (g.Ho < kRowsPerTile && kRowsPerTile % g.Ho == 0))) return false;
  }
  return true;
}

aiq_status_t conv_tc_encode_map(const ConvGeom& g, const void* slot_base, int batch_capacity, int n_versions,
                                void* map_out) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  const cuuint64_t pix_bytes = 4ull * g.Cs_in;
  const cuuint64_t rows = (cuuint64_t)batch_capacity * (g.H + 2);
  const cuuint32_t inner = pix_bytes < 128 ? (cuuint32_t)(2 * g.Cs_in) : 64u;
  const CUtensorMapSwizzle swz = pix_bytes < 128 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
  CUresult r;
  if (g.stride == 1) {
    // (channel, column, padded row of the batch, version)
    cuuint64_t dims[4] = {(cuuint64_t)2 * g.Cs_in, (cuuint64_t)g.W, rows, (cuuint64_t)n_versions};
    cuuint64_t strides[3] = {pix_bytes, pix_bytes * g.W, pix_bytes * g.W * rows};
    cuuint32_t box[4] = {inner, (cuuint32_t)kColsPerTile, (cuuint32_t)kBoxRows, 1u};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    r = enc(static_cast<CUtensorMap*>(map_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(slot_base),
            dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    // (channel, column parity, column pair, row parity, row pair over all versions): a tap of a
    // stride-2 window is then a dense box.  Rows per image and per version are even.
    const int rows_per_img = g.Ho < kRowsPerTile ? g.Ho : kRowsPerTile;
    cuuint64_t dims[5] = {(cuuint64_t)2 * g.Cs_in, 2, (cuuint64_t)g.W / 2, 2, rows * n_versions / 2};
    cuuint64_t strides[4] = {pix_bytes, 2 * pix_bytes, pix_bytes * g.W, 2 * pix_bytes * g.W};
    cuuint32_t box[5] = {inner, 1u, (cuuint32_t)kColsPerTile, 1u, (cuuint32_t)rows_per_img};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    r = enc(static_cast<CUtensorMap*>(map_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(slot_base),
            dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return AIQ_OK;
}

bool conv_tc_bits_ok(const ConvGeom& g, int bits) {
  // two weight tiles per tap of a 32-channel output slice fit shared memory beside the
  // activation ring for every eligible shape
  (void)g;
  return bits == 4 || bits == 8 || bits == 16 || bits == 32;
}

aiq_status_t launch_conv_tc(const ConvGeom& g, const void* map, const LayerJob* jobs_dev, int n_jobs,
                            int batch_capacity, int32_t* error_flag, double weight_bytes, int weight_bits,
                            cudaStream_t s) {
  const CUtensorMap& m = *static_cast<const CUtensorMap*>(map);
#define AIQ_TC_ARGS g, m, jobs_dev, n_jobs, batch_capacity, error_flag, weight_bytes, weight_bits, s
#define AIQ_TC_KS(CS_, N_, P_)                                                                                   \
  do {                                                                                                          \
    if (g.stride == 1) return g.ks == 3 ? launch_tc<CS_, N_, 3, 1, P_>(AIQ_TC_ARGS) : launch_tc<CS_, N_, 1, 1, P_>(AIQ_TC_ARGS); \
    return g.ks == 3 ? launch_tc<CS_, N_, 3, 2, P_>(AIQ_TC_ARGS) : launch_tc<CS_, N_, 1, 2, P_>(AIQ_TC_ARGS);    \
  } while (0)
#define AIQ_TC_CASE(CS_, N_)                                                                    \
  if (g.Cin == CS_ && g.Cout == N_ && pieces == 1) AIQ_TC_KS(CS_, N_, 1);
#define AIQ_TC_CASE_WIDE(CS_, N_)                                                               \
  if (g.Cin == CS_ && (g.Cout == N_ || g.Cout == 2 * N_) && pieces == 2) AIQ_TC_KS(CS_, N_, 2);
  const int pieces = weight_bits <= 8 ? 1 : 2;
  AIQ_TC_CASE(16, 16) AIQ_TC_CASE(16, 32) AIQ_TC_CASE(16, 64)
  AIQ_TC_CASE(32, 16) AIQ_TC_CASE(32, 32) AIQ_TC_CASE(32, 64)
  AIQ_TC_CASE(64, 16) AIQ_TC_CASE(64, 32) AIQ_TC_CASE(64, 64)
  // 16- / 32-bit weights: at most 32 output channels per slice, 64 run as two slices of 32
  AIQ_TC_CASE_WIDE(16, 32) AIQ_TC_CASE_WIDE(32, 32) AIQ_TC_CASE_WIDE(64, 32)
  AIQ_TC_CASE_WIDE(16, 16) AIQ_TC_CASE_WIDE(32, 16) AIQ_TC_CASE_WIDE(64, 16)
#undef AIQ_TC_CASE_WIDE
#undef AIQ_TC_KS
#undef AIQ_TC_CASE
#undef AIQ_TC_ARGS
  return set_error(AIQ_ERR_SHAPE, "conv_tc: no kernel for Cin=%d Cout=%d", g.Cin, g.Cout);
}

// ---- the expiry path of the bounded waits, exercised on purpose ------------------------------
// One thread waits, with the same helper the kernels above use, on a barrier that nothing ever
// arrives at.  The wait gives up after `limit_cycles`, raises the error word and the kernel
// returns normally: nothing traps, faults or hangs.
namespace {
__global__ void expire_wait_kernel(int32_t* error_flag, long long limit_cycles, int32_t* observed) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait_for(smem_u32(&bar), 0, &abort_flag, error_flag, limit_cycles);
    if (observed) *observed = ok ? 0 : 1 + abort_flag;      // 2: gave up and raised the abort flag
  }
}
}  // namespace

aiq_status_t launch_expire_wait(int32_t* error_flag, long long limit_cycles, int32_t* observed, cudaStream_t s) {
  expire_wait_kernel<<<1, 32, 0, s>>>(error_flag, limit_cycles, observed);
  AIQ_LAUNCH_CHECK("expire_wait");
  return AIQ_OK;
}

}  // namespace aiq
