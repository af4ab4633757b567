// Row-streaming 3x3 / 1x1 convolution on the tcgen05 tensor cores for networks whose feature
// maps are narrow (8, 16 or 32 columns) and have 16, 32 or 64 channels (the CIFAR ResNets).
//
//   out[y][x][n] = act( s_n * sum_{r,t,c} code[n][c][r][t] * in[y*S + r - 1][x*S + t - 1][c] + b_n + res[y][x][n] )
//
// With few output channels an MMA of 128 pixels x N = Cout spends its time fetching the 128-row
// pixel operand from shared memory, once per tap: nine fetches per pixel and layer.  Here the
// three vertical taps are folded into the MMA's N dimension instead.  The 128 accumulator lanes
// are (column, image) pairs of ONE image row - a group of 8 or 16 images is interleaved in
// memory for that purpose - so the output rows y-1, y, y+1 that an input row feeds live in the
// same lanes, in neighbouring column ranges of tensor memory.  One MMA per horizontal tap with
// the weights [W(r=2) | W(r=1) | W(r=0)] as an N = 3 Cout operand adds an input row's
// contribution to all three; the tensor cores do the vertical sum, the pixel operand is fetched
// three times instead of nine, and the MMAs are three times as wide.
//
// Activation format ACT_RS: [group][row][column][plane][image][8 bfloat16], G = 8 images per
// group when the width is a multiple of 16, else 16; plane p < C/8 holds the hi halves of
// channels 8p .. 8p+7, plane C/8 + p their lo halves (value = hi + lo, see common.cuh); no
// padding rows or columns are stored.  A TMA box brings one input row of a group into shared
// memory as [plane][column][image][16 bytes] with zero columns on both sides; in the canonical
// K-major layout without swizzle (8 rows x 16 bytes per core matrix, 128 bytes from one group
// of 8 rows to the next) that is directly the A operand of every horizontal tap: tap t starts t
// columns further.  Stride-2 layers view the columns as (parity, pair), so that every tap is
// again a dense run of column pairs.  Output rows are finished one input row later; the epilogue
// warps read them from tensor memory, apply scale, bias, residual and activation, split into
// two bfloat16 and store 16 bytes per lane and plane: the 32 lanes of a warp cover whole
// 128-byte lines, so no staging through shared memory is needed.
//
// Every wait is bounded as in the other tcgen05 kernels.
#include "tc_ptx.cuh"

namespace aiq {

namespace {

// Warps: TMA producer, MMA issuer, then the epilogue warps, four per quarter of the accumulator
// lanes where one CTA has an SM to itself, two per quarter where two CTAs share it (then each
// CTA's issuing warp hides the other's per-row bookkeeping, and each takes half of tensor memory).
constexpr int kRsMaxEpiWarps = 16;
constexpr int kRsMaxThreads = (2 + kRsMaxEpiWarps) * 32;
constexpr int kRsMaxStages = 6;
constexpr int kRsMaxSlots = 16;
constexpr int kRsTileBytes = 2048;                     // 128 operand rows x 16 bytes of one plane
constexpr int kRsMaxRows = 64;                         // input rows of a feature map
constexpr int kRsRowWords = 20;                        // words of one row program (see RowProgram)

// What the MMA warp does for one input row: the runs of accumulator slots it feeds.  All K steps
// but the first add to every output row the input row touches: one MMA per run of consecutive
// slots (`rest`, at most two: the ring of slots may wrap).  The first K step must overwrite the
// rows that receive their first contribution: its runs are cut there as well (`head`, at most
// three).  A run = (instruction descriptor with its N, accumulator column, weight row offset in
// 16-byte units).  The slots do not depend on the item because the ring depth divides the rows
// of an item.
struct RowProgram {
  uint32_t head_idesc[3], head_dcol[3], head_boff[3];
  uint32_t rest_idesc[2], rest_dcol[2], rest_boff[2];
  uint32_t head_acc;        // bit i: run i of head accumulates (else overwrites)
  uint32_t n_runs;          // head runs | rest runs << 4
  uint32_t fresh;           // first output row that must be free before the MMAs | count << 8
  uint32_t done;            // output rows complete after this input row: (row A + 1) | (row B + 1) << 8; 0 = none
  uint32_t pad;
};
static_assert(sizeof(RowProgram) == kRsRowWords * 4, "row program size");

struct RsParams {
  int H, W, Ho, Wo;
  int N;                  // output channels of one slice (blockIdx.z selects the slice)
  int cout_total;         // channels of an output pixel
  int act;
  int gmode;              // images per group: 0: 8 in, 8 out;  1: 16 in, 16 out;  2: 8 in, 16 out (stride 2)
  int n_items;            // output groups of the batch
  int rows_per_version;   // step of the TMA row coordinate from one input version to the next
  int n_stages, n_slots;  // input-row ring depth; output rows in flight per column tile (power of two)
  int K;                  // elements of a packed weight row
  int stage_bytes;        // bytes one input row occupies in shared memory
  int a_tap_off[3];       // byte offset of horizontal tap t inside a stage (column tile 0, plane 0)
  int a_lbo;              // bytes from one plane (8 channels) to the next
  int xt;                 // column tiles (128 lanes each) per row
  int tmem_cols;          // tensor-memory columns this CTA allocates (512, or 256 with two CTAs per SM)
  int pool_bytes;         // shared memory for the fused average pool (0: the jobs of this launch do not pool)
  int batch;              // images of the batch (the last group may hold fewer)
  int32_t* error_flag;
};

__host__ __device__ constexpr int rs_taps(int ks) { return ks == 3 ? 3 : 1; }

// shared memory regions (base aligned to 1024 bytes)
struct RsSmem {
  int ring, weights, scale, bias, rows, pool, bars, total;
};
__host__ __device__ inline RsSmem rs_smem(int stages, int stage_bytes, int weight_bytes, int N, int pool_bytes = 0) {
  RsSmem s;
  s.ring = 0;
  s.weights = stages * stage_bytes;
  s.scale = s.weights + weight_bytes;
  s.bias = s.scale + N * 4;
  s.rows = (s.bias + N * 4 + 127) / 128 * 128;          // per input row: the MMA program (kRsRowWords words)
  s.pool = s.rows + kRsMaxRows * kRsRowWords * 4;       // partial sums of the fused average pool
  s.bars = s.pool + pool_bytes;
  s.total = s.bars + (2 * kRsMaxStages + 2 * kRsMaxSlots + 3) * 8 + 16;
  return s;
}

// Row program of input row y (see RowProgram).  R = accumulator slots per column tile.
template <int KS, int STRIDE>
__device__ __forceinline__ RowProgram rs_row_program(int y, int H, int Ho, int N, int R) {
  constexpr uint32_t IDESC0 = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);   // f32 += bf16 x bf16, M = 128
  const uint32_t n_field = ((uint32_t)N >> 3) << 17;                                     // N field of one output row
  // output rows this input row contributes to: [yo, yo + n_rows), weight blocks [blk, ...); the
  // rows from index `fresh` on receive their first contribution; rows done_a / done_b are complete
  int yo, n_rows, blk, fresh, done_a = -1, done_b = -1;
  if (KS == 1) { yo = y / STRIDE; n_rows = 1; blk = 0; fresh = 0; done_a = yo; }
  else if (STRIDE == 1) {
    yo = y > 0 ? y - 1 : 0;
    const int hi = y + 1 < H ? y + 1 : H - 1;
    n_rows = hi - yo + 1;
    blk = yo - (y - 1);
    fresh = y == 0 ? 0 : (y + 1 < H ? n_rows - 1 : n_rows);
    if (y >= 1) done_a = y - 1;
    if (y == H - 1) done_b = y;
  } else if ((y & 1) == 0) { yo = y >> 1; n_rows = 1; blk = 0; fresh = y == 0 ? 0 : 1; }
  else { yo = y >> 1; blk = 1; n_rows = (yo + 1 < Ho) ? 2 : 1; fresh = 1; done_a = yo; }
  const int s0 = yo & (R - 1);
  const int wrap = R - s0;                       // rows from this index on continue at slot 0
  const int cw = (wrap > 0 && wrap < n_rows) ? wrap : n_rows;
  const int cf = (fresh > 0 && fresh < n_rows) ? fresh : n_rows;
  RowProgram rp = {};
  auto set_run = [&](uint32_t* idesc, uint32_t* dcol, uint32_t* boff, int k, int i, int j) {
    idesc[k] = IDESC0 | (uint32_t)(j - i) * n_field;
    dcol[k] = (uint32_t)(((s0 + i) & (R - 1)) * N);
    boff[k] = (uint32_t)((blk + i) * N);
  };
  int n_rest = 1;
  set_run(rp.rest_idesc, rp.rest_dcol, rp.rest_boff, 0, 0, cw);
  if (cw < n_rows) { set_run(rp.rest_idesc, rp.rest_dcol, rp.rest_boff, 1, cw, n_rows); n_rest = 2; }
  const int c1 = cw < cf ? cw : cf;
  int c2 = cw < cf ? cf : cw;
  if (c2 == c1) c2 = n_rows;
  int n_head = 1;
  set_run(rp.head_idesc, rp.head_dcol, rp.head_boff, 0, 0, c1);
  rp.head_acc = 0 >= fresh ? 0u : 1u;
  if (c1 < n_rows) {
    set_run(rp.head_idesc, rp.head_dcol, rp.head_boff, 1, c1, c2);
    rp.head_acc |= (c1 >= fresh ? 0u : 1u) << 1;
    n_head = 2;
    if (c2 < n_rows) {
      set_run(rp.head_idesc, rp.head_dcol, rp.head_boff, 2, c2, n_rows);
      rp.head_acc |= (c2 >= fresh ? 0u : 1u) << 2;
      n_head = 3;
    }
  }
  rp.n_runs = (uint32_t)n_head | ((uint32_t)n_rest << 4);
  rp.fresh = (uint32_t)(yo + fresh) | ((uint32_t)(n_rows - fresh) << 8);
  rp.done = (uint32_t)(done_a + 1) | ((uint32_t)(done_b + 1) << 8);
  return rp;
}

// Packed weight rows (staged in shared memory at `staged`, `wrow_bytes` apart, N rows) -> bfloat16
// operand tiles at `wsm`: [piece][tap][8-channel chunk][vertical tap block, channel][8 channels].
template <int C, int KS, int STRIDE, int PIECES>
__device__ __forceinline__ void rs_expand_weights(const uint8_t* staged, uint32_t wrow_bytes, int bits, int N, uint8_t* wsm,
                                                  int tid, int n_threads) {
  constexpr int T = rs_taps(KS), NBLK = KS == 3 ? 3 : 1, KCH = C / 8;
  const int NB = NBLK * N;
  const int tile_b = KCH * NB * 16;
  const int w_units = T * KCH * NB;
  for (int u = tid; u < w_units; u += n_threads) {
    const int row = u % NB;
    const int kc = (u / NB) % KCH;
    const int ti = u / (NB * KCH);
    const int blk = row / N, n = row - blk * N;
    // vertical tap of a block: stride 1: the input row feeds output rows y-1, y, y+1 = taps 2, 1, 0;
    // stride 2: even input rows carry tap 1 (block 0), odd rows taps 2 and 0 (blocks 1, 2)
    const int r = KS == 1 ? 0 : (STRIDE == 1 ? 2 - blk : (blk == 0 ? 1 : (blk == 1 ? 2 : 0)));
    const uint8_t* wrow = staged + (size_t)n * wrow_bytes;
    uint32_t pk[PIECES][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int c = kc * 8 + j;
      const int k = KS == 1 ? c : (c * 3 + r) * 3 + ti;
      float w;
      if (bits == 8) w = (float)(int)(int8_t)wrow[k];
      else if (bits == 4) {
        const int byte = wrow[k >> 1];
        w = (float)((((k & 1) ? (byte >> 4) : (byte & 0xF)) ^ 8) - 8);
      } else if (bits == 16) w = __half2float(reinterpret_cast<const __half*>(wrow)[k]);
      else w = reinterpret_cast<const float*>(wrow)[k];
#pragma unroll
      for (int pc = 0; pc < PIECES; ++pc) {
        const __nv_bfloat16 hb = __float2bfloat16_rn(w);   // exact for the integer codes
        w -= __bfloat162float(hb);                          // exact: the remainder of the rounding
        const uint32_t bits16 = (uint32_t)__bfloat16_as_ushort(hb);
        if (j & 1) pk[pc][j >> 1] |= bits16 << 16; else pk[pc][j >> 1] = bits16;
      }
    }
#pragma unroll
    for (int pc = 0; pc < PIECES; ++pc)
      *reinterpret_cast<uint4*>(wsm + (size_t)(pc * T + ti) * tile_b + (size_t)kc * NB * 16 + row * 16) =
          make_uint4(pk[pc][0], pk[pc][1], pk[pc][2], pk[pc][3]);
  }
}

// A row program in registers.
struct RowRegs { uint4 w0, w1, w2, w3, w4; };
__device__ __forceinline__ RowRegs rs_load_row(const RowProgram& rp) {
  RowRegs r;
  r.w0 = *reinterpret_cast<const uint4*>(&rp.head_idesc[0]);   // head_idesc[0..2], head_dcol[0]
  r.w1 = *reinterpret_cast<const uint4*>(&rp.head_dcol[1]);    // head_dcol[1..2], head_boff[0..1]
  r.w2 = *reinterpret_cast<const uint4*>(&rp.head_boff[2]);    // head_boff[2], rest_idesc[0..1], rest_dcol[0]
  r.w3 = *reinterpret_cast<const uint4*>(&rp.rest_dcol[1]);    // rest_dcol[1], rest_boff[0..1], head_acc
  r.w4 = *reinterpret_cast<const uint4*>(&rp.n_runs);          // n_runs, fresh, done, pad
  return r;
}

// All MMAs of one input row into one column tile: d_xt = accumulator base of the tile, a_xt = low
// descriptor word of the tile's pixel operand (tap offset 0), operand steps in 16-byte units.
// Called by a converged warp; an elected lane issues.
template <int C, int T, int PIECES>
__device__ __forceinline__ void rs_issue_row(const RowRegs& rr, uint32_t d_xt, uint32_t a_xt, uint32_t a_tap0, uint32_t a_tap1,
                                             uint32_t a_tap2, uint32_t a_part_step, uint32_t a_kk_step, uint32_t w_lo0,
                                             uint32_t b_tile_step, uint32_t b_kk_step) {
  constexpr uint32_t DESC_HI = (uint32_t)(128 >> 4) | (1u << 14);   // 128 bytes between groups of 8 rows; no swizzle
  const uint32_t h0_idesc = rr.w0.x, h1_idesc = rr.w0.y, h2_idesc = rr.w0.z, h0_dcol = rr.w0.w;
  const uint32_t h1_dcol = rr.w1.x, h2_dcol = rr.w1.y, h0_boff = rr.w1.z, h1_boff = rr.w1.w;
  const uint32_t h2_boff = rr.w2.x, r0_idesc = rr.w2.y, r1_idesc = rr.w2.z, r0_dcol = rr.w2.w;
  const uint32_t r1_dcol = rr.w3.x, r0_boff = rr.w3.y, r1_boff = rr.w3.z, head_acc = rr.w3.w;
  const bool head1 = (rr.w4.x & 15u) > 1u, head2 = (rr.w4.x & 15u) > 2u, rest1 = (rr.w4.x >> 4) > 1u;
  const uint32_t h0_acc = head_acc & 1u, h1_acc = (head_acc >> 1) & 1u, h2_acc = (head_acc >> 2) & 1u;
#pragma unroll
  for (int t = 0; t < T; ++t) {
    const uint32_t a_t = a_xt + ((t == 0 ? a_tap0 : (t == 1 ? a_tap1 : a_tap2)) >> 4);
#pragma unroll
    for (int part = 0; part < 2; ++part) {
#pragma unroll
      for (int kk = 0; kk < C / 16; ++kk) {
        const uint64_t adesc = ((uint64_t)DESC_HI << 32) | (uint64_t)(a_t + part * a_part_step + kk * a_kk_step);
#pragma unroll
        for (int pc = 0; pc < PIECES; ++pc) {
          const uint32_t b_lo = w_lo0 + (uint32_t)(pc * T + t) * b_tile_step + (uint32_t)kk * b_kk_step;
          if (t == 0 && part == 0 && kk == 0 && pc == 0) {
            umma_bf16(d_xt + h0_dcol, adesc, ((uint64_t)DESC_HI << 32) | (uint64_t)(b_lo + h0_boff), h0_idesc, h0_acc);
            if (head1) umma_bf16(d_xt + h1_dcol, adesc, ((uint64_t)DESC_HI << 32) | (uint64_t)(b_lo + h1_boff), h1_idesc, h1_acc);
            if (head2) umma_bf16(d_xt + h2_dcol, adesc, ((uint64_t)DESC_HI << 32) | (uint64_t)(b_lo + h2_boff), h2_idesc, h2_acc);
          } else {
            umma_bf16(d_xt + r0_dcol, adesc, ((uint64_t)DESC_HI << 32) | (uint64_t)(b_lo + r0_boff), r0_idesc, 1u);
            if (rest1) umma_bf16(d_xt + r1_dcol, adesc, ((uint64_t)DESC_HI << 32) | (uint64_t)(b_lo + r1_boff), r1_idesc, 1u);
          }
        }
      }
    }
  }
}

// 16 accumulator values of one lane (a 16-channel chunk of one pixel) -> scale, bias, residual,
// activation, split into hi / lo bfloat16 pairs: hi[0..3] / hi[4..7] are the two hi planes of
// the chunk, lo likewise.  res: the four residual planes (hi, hi, lo, lo) of the same pixel.
__device__ __forceinline__ void rs_finish_unit(const uint32_t* v, const float* scale, const float* bias, const uint4* res,
                                               bool has_res, int act, uint32_t* hi, uint32_t* lo) {
#pragma unroll
  for (int e = 0; e < 16; e += 4) {
    const float4 sc = *reinterpret_cast<const float4*>(scale + e);
    const float4 bi = *reinterpret_cast<const float4*>(bias + e);
    float u0 = fmaf(__uint_as_float(v[e]), sc.x, bi.x);
    float u1 = fmaf(__uint_as_float(v[e + 1]), sc.y, bi.y);
    float u2 = fmaf(__uint_as_float(v[e + 2]), sc.z, bi.z);
    float u3 = fmaf(__uint_as_float(v[e + 3]), sc.w, bi.w);
    if (has_res) {
      // planes 0 / 1 of the chunk hold channels 0-7 / 8-15; a bfloat16 is the upper half of a float
      const uint4 rh4 = res[e >> 3], rl4 = res[2 + (e >> 3)];
      const uint32_t rh0 = (e & 4) ? rh4.z : rh4.x, rh1 = (e & 4) ? rh4.w : rh4.y;
      const uint32_t rl0 = (e & 4) ? rl4.z : rl4.x, rl1 = (e & 4) ? rl4.w : rl4.y;
      u0 += __uint_as_float(rh0 << 16) + __uint_as_float(rl0 << 16);
      u1 += __uint_as_float(rh0 & 0xFFFF0000u) + __uint_as_float(rl0 & 0xFFFF0000u);
      u2 += __uint_as_float(rh1 << 16) + __uint_as_float(rl1 << 16);
      u3 += __uint_as_float(rh1 & 0xFFFF0000u) + __uint_as_float(rl1 & 0xFFFF0000u);
    }
    split_pair(apply_act(u0, act), apply_act(u1, act), hi[e >> 1], lo[e >> 1]);
    split_pair(apply_act(u2, act), apply_act(u3, act), hi[(e >> 1) + 1], lo[(e >> 1) + 1]);
  }
}

template <int C, int KS, int STRIDE, int PIECES>
__global__ void __launch_bounds__(kRsMaxThreads, 1)
conv_rs_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1, RsParams p,
               const LayerJob* __restrict__ jobs) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const LayerJob job = jobs[blockIdx.y];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int T = rs_taps(KS);                     // horizontal taps = weight tiles per piece
  constexpr int NBLK = KS == 3 ? 3 : 1;              // vertical taps stacked along N
  constexpr int KCH = C / 8;                         // 16-byte K chunks of the channels
  const int N = p.N, NB = NBLK * N;
  const int tile_b = KCH * NB * 16;                  // bytes of one weight tile
  const int weight_bytes = PIECES * T * tile_b;
  const int stages = p.n_stages, R = p.n_slots;
  const RsSmem sm = rs_smem(stages, p.stage_bytes, weight_bytes, N, p.pool_bytes);
  uint8_t* ring = smem;
  uint8_t* wsm = smem + sm.weights;
  float* s_scale = reinterpret_cast<float*>(smem + sm.scale);
  float* s_bias = reinterpret_cast<float*>(smem + sm.bias);
  RowProgram* s_rows = reinterpret_cast<RowProgram*>(smem + sm.rows);
  float* s_pool = reinterpret_cast<float*>(smem + sm.pool);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
  const uint32_t bar_in_full = smem_u32(bars);
  const uint32_t bar_in_empty = bar_in_full + 8 * kRsMaxStages;
  const uint32_t bar_out_full = bar_in_empty + 8 * kRsMaxStages;
  const uint32_t bar_out_empty = bar_out_full + 8 * kRsMaxSlots;
  const uint32_t bar_w = bar_out_empty + 8 * kRsMaxSlots;
  const uint32_t bar_pool = bar_w + 8;               // two rendezvous of the epilogue warps per pooled item
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * kRsMaxStages + 2 * kRsMaxSlots + 3);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  const int n_off = (int)blockIdx.z * N;             // first output channel of this slice
  // Epilogue work: per output row and quarter of the lanes, `units` = column tiles x 16-channel
  // chunks.  The WQ warps of a quarter either share the units of every row, or, where a row has
  // fewer units than that, take every (WQ / units)-th row each, so several rows are drained at once.
  const int n_threads = (int)blockDim.x;
  const int WQ = (n_threads / 32 - 2) / 4;           // epilogue warps per quarter: 4 or 2
  const int units = p.xt * (N / 16);
  const int epi_sets = units < WQ ? units : WQ;      // warps of a quarter that read one row

  // ---- set-up -----------------------------------------------------------------------------
  if (tid == 0) {
    for (int i = 0; i < kRsMaxStages; ++i) {
      mbar_init(bar_in_full + 8 * i, 1);
      mbar_init(bar_in_empty + 8 * i, 1);
    }
    for (int i = 0; i < kRsMaxSlots; ++i) {
      mbar_init(bar_out_full + 8 * i, 1);
      mbar_init(bar_out_empty + 8 * i, 4 * epi_sets);      // one arrival per epilogue warp that reads the row
    }
    mbar_init(bar_w, 1);
    mbar_init(bar_pool, 4 * WQ);
    mbar_init(bar_pool + 8, 4 * WQ);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 1) {
    tmem_alloc(smem_u32(s_tmem), (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  // packed weight rows of this slice: one bulk copy into the (still unused) ring, then expansion
  // to bfloat16 in the operand layout [tap][8-channel chunk][vertical tap block, channel][8 channels]
  const int kpad = (p.K + 31) / 32 * 32;
  const uint32_t wrow_bytes = (uint32_t)kpad * job.bits / 8;
  const uint32_t packed_bytes = wrow_bytes * N;
  if (tid == 0) {
    mbar_expect_tx(bar_w, packed_bytes);
    bulk_load(smem_u32(ring), job.w + (size_t)n_off * wrow_bytes, packed_bytes, bar_w);
  }
  for (int i = tid; i < N; i += n_threads) {
    s_scale[i] = job.scale[n_off + i];
    s_bias[i] = job.bias[n_off + i];
  }
  for (int i = tid; i < p.pool_bytes / 4; i += n_threads) s_pool[i] = 0.f;
  // row programs (one thread per input row)
  if (tid < p.H) s_rows[tid] = rs_row_program<KS, STRIDE>(tid, p.H, p.Ho, N, R);
  bool alive = mbar_wait_warp(bar_w, 0, s_abort, p.error_flag);
  if (alive) rs_expand_weights<C, KS, STRIDE, PIECES>(ring, wrow_bytes, job.bits, N, wsm, tid, n_threads);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // expanded weights -> visible to the MMA
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  alive = alive && (*s_abort == 0);

  // rows of the input that carry work: a 1x1 convolution at stride 2 only reads the even ones
  auto row_used = [&](int y) -> bool { return !(KS == 1 && STRIDE == 2 && (y & 1)); };

  // ---- roles ------------------------------------------------------------------------------
  if (warp == 0) {
    if (lane == 0 && alive) {
      uint32_t stage = 0, phase = 0;
      uint32_t issued = 0, issued_phase = 0;
      for (int item = blockIdx.x; item < p.n_items && alive; item += gridDim.x) {
        const int row0 = job.in_version * p.rows_per_version + (p.gmode == 2 ? 2 * item : item) * p.H;
        for (int y = 0; y < p.H && alive; ++y) {
          if (!row_used(y)) continue;
          alive = mbar_wait(bar_in_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
          if (!alive) break;
          issued |= 1u << stage;
          issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
          const uint32_t bar = bar_in_full + 8 * stage;
          const uint32_t dst = smem_u32(ring) + stage * p.stage_bytes;
          mbar_expect_tx(bar, (uint32_t)p.stage_bytes);
          if (STRIDE == 1) {
            tma_load_4d(dst, &map0, bar, 0, KS == 3 ? -1 : 0, 0, row0 + y);
          } else if (p.gmode != 2) {
            tma_load_5d(dst, &map0, bar, 0, KS == 3 ? -1 : 0, 0, 0, row0 + y);
          } else if (KS == 3) {
            // odd columns from pair -1 (tap 0), even columns (tap 1), odd columns from pair 0 (tap 2)
            const uint32_t sub = (uint32_t)p.stage_bytes / 3;
            tma_load_5d(dst, &map1, bar, 0, -1, 0, 0, row0 + y);
            tma_load_5d(dst + sub, &map0, bar, 0, 0, 0, 0, row0 + y);
            tma_load_5d(dst + 2 * sub, &map1, bar, 0, 0, 0, 0, row0 + y);
          } else {
            tma_load_5d(dst, &map0, bar, 0, 0, 0, 0, row0 + y);
          }
          if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
        }
      }
      // copies in flight must land before the CTA exits (matters when another role gave up)
      for (int i = 0; i < stages; ++i)
        if (issued & (1u << i)) {
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_in_full + 8 * i, (issued_phase >> i) & 1u) && clock64() - t0 < kWaitLimitCycles) {}
        }
    }
  } else if (warp == 1) {
    if (alive) {                                     // all 32 lanes, converged; an elected lane issues
      constexpr uint32_t IDESC0 = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);   // f32 += bf16 x bf16, M = 128
      constexpr uint32_t DESC_HI = (uint32_t)(128 >> 4) | (1u << 14);   // 128 bytes between groups of 8 rows; no swizzle
      const uint32_t a_lbo_field = ((uint32_t)p.a_lbo >> 4) << 16;
      const uint32_t w_lo0 = (smem_u32(wsm) >> 4) | (((uint32_t)(NB * 16) >> 4) << 16);
      // operand steps in 16-byte units, so that an MMA costs a few additions
      const uint32_t a_part_step = ((uint32_t)KCH * (uint32_t)p.a_lbo) >> 4;     // hi planes -> lo planes
      const uint32_t a_kk_step = (2u * (uint32_t)p.a_lbo) >> 4;                  // 16 channels further
      const uint32_t b_tile_step = (uint32_t)tile_b >> 4, b_kk_step = 2u * (uint32_t)NB;
      const uint32_t n_field = ((uint32_t)N >> 3) << 17;                         // N field of one output row
      const uint32_t a_tap0 = (uint32_t)p.a_tap_off[0], a_tap1 = (uint32_t)p.a_tap_off[1], a_tap2 = (uint32_t)p.a_tap_off[2];
      uint32_t stage = 0, phase = 0;
      int item_local = 0;
      for (int item = blockIdx.x; item < p.n_items && alive; item += gridDim.x, ++item_local) {
        const int q0 = item_local * p.Ho;
        for (int y = 0; y < p.H && alive; ++y) {
          if (!row_used(y)) continue;
          const RowRegs rr = rs_load_row(s_rows[y]);
          const uint4 w4 = rr.w4;
          const int fresh_row = (int)(w4.y & 255u), n_fresh = (int)(w4.y >> 8);
          for (int i = 0; i < n_fresh && alive; ++i) {
            const int q = q0 + fresh_row + i;
            alive = mbar_wait_warp(bar_out_empty + 8 * (q & (R - 1)), ((q / R) & 1) ^ 1u, s_abort, p.error_flag);
          }
          if (!alive) break;
          alive = mbar_wait_warp(bar_in_full + 8 * stage, phase, s_abort, p.error_flag);
          if (!alive) break;
          tc_fence_after();
          const uint32_t a_stage = smem_u32(ring) + stage * p.stage_bytes;
          for (int xt = 0; xt < p.xt; ++xt)
            rs_issue_row<C, T, PIECES>(rr, tmem_base + (uint32_t)(xt * R * N),
                                       ((a_stage + (uint32_t)xt * kRsTileBytes) >> 4) | a_lbo_field, a_tap0, a_tap1, a_tap2,
                                       a_part_step, a_kk_step, w_lo0, b_tile_step, b_kk_step);
          umma_commit(bar_in_empty + 8 * stage);       // the stage is free once these MMAs retire
          if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
          // output rows that are complete with this input row
          if (w4.z & 255u) umma_commit(bar_out_full + 8 * (((w4.z & 255u) - 1u) & (uint32_t)(R - 1)));
          if (w4.z >> 8) umma_commit(bar_out_full + 8 * (((w4.z >> 8) - 1u) & (uint32_t)(R - 1)));
        }
      }
    }
  } else {
    // Epilogue.  Accumulator lanes 32 qd .. 32 qd + 31 belong to the warps with warp index mod 4 = qd.
    const int qd = warp & 3;
    const int h = (warp - 2) >> 2;                     // index among the warps of the quarter
    const int l = qd * 32 + lane;                      // accumulator lane = operand row of the tile
    int x_local, img;
    if (p.gmode == 0) { x_local = l >> 3; img = l & 7; }
    else if (p.gmode == 1) { x_local = l >> 4; img = l & 15; }
    else { x_local = (l >> 3) & 7; img = ((l >> 6) << 3) | (l & 7); }
    const int X = p.gmode == 0 ? 16 : 8;               // columns per tile
    const int Gout = p.gmode == 0 ? 8 : 16;
    const int planes_out = p.cout_total / 4;
    const size_t plane_bytes = (size_t)Gout * 16;
    const size_t px_bytes = (size_t)planes_out * plane_bytes;
    const int chunks = N / 16;
    const uint8_t* res_base = static_cast<const uint8_t*>(job.res);
    uint8_t* out_base = static_cast<uint8_t*>(job.out);
    const int lo_plane0 = p.cout_total / 8;
    const bool pooling = p.pool_bytes > 0 && job.pool != nullptr;
    const float pool_scale = 1.0f / (float)(p.Ho * p.Wo);
    // this warp's units of a row and its rows of an item
    const int unit0 = units >= WQ ? h : h % units;
    const int unit_step = units >= WQ ? WQ : units;
    const int row_first = units >= WQ ? 0 : h / units;
    const int row_step = units >= WQ ? 1 : WQ / units;
    const int rows_mine = p.Ho / row_step;             // rows of an item this warp drains
    const int n_my_items = ((int)blockIdx.x < p.n_items) ? (p.n_items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int total = n_my_items * rows_mine;
    auto row_offset = [&](int k) -> size_t {           // byte offset of this lane's image in the k-th row of this warp
      const int il = k / rows_mine;
      const int y = row_first + (k - il * rows_mine) * row_step;
      return ((size_t)((int)blockIdx.x + il * (int)gridDim.x) * p.Ho + y) * p.Wo * px_bytes + (size_t)img * 16;
    };
    auto unit_offset = [&](int u, int* c0) -> size_t { // byte offset of (column, first hi plane) of unit u inside a row
      const int xt = u / chunks;
      *c0 = (u - xt * chunks) * 16;
      return (size_t)(xt * X + x_local) * px_bytes + (size_t)((n_off + *c0) >> 3) * plane_bytes;
    };
    // The residual of the first unit of this warp's next row is requested as soon as the current
    // row's arithmetic is done, so its memory latency overlaps the stores and the next wait.
    uint4 rres[4];
    auto load_res = [&](int k, int u, uint4* r) {
      int c0;
      const uint8_t* src = res_base + row_offset(k) + unit_offset(u, &c0);
      r[0] = __ldg(reinterpret_cast<const uint4*>(src));
      r[1] = __ldg(reinterpret_cast<const uint4*>(src + plane_bytes));
      r[2] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)lo_plane0 * plane_bytes));
      r[3] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)(lo_plane0 + 1) * plane_bytes));
    };
    if (res_base && total > 0 && alive) load_res(0, unit0, rres);
    for (int k = 0; k < total && alive; ++k) {
      const int il = k / rows_mine;
      const int y = row_first + (k - il * rows_mine) * row_step;
      const int q = il * p.Ho + y;
      const int slot = q & (R - 1);
      const size_t row_off = row_offset(k);
      alive = mbar_wait_warp(bar_out_full + 8 * slot, (q / R) & 1, s_abort, p.error_flag);
      if (!alive) break;
      tc_fence_after();
      for (int u = unit0; u < units; u += unit_step) {
        int c0;
        const size_t uoff = unit_offset(u, &c0);
        const int xt = u / chunks;
        uint32_t v[16];
        tmem_ld16(tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)((xt * R + slot) * N + c0), v);
        if (res_base && u != unit0) load_res(k, u, rres);
        tmem_ld_wait();
        if (u + unit_step >= units) {
          // the last accumulator columns this warp reads from the slot: hand it back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_out_empty + 8 * slot);
        }
        uint32_t hi[8], lo[8];
        rs_finish_unit(v, s_scale + c0, s_bias + c0, rres, res_base != nullptr, p.act, hi, lo);
        // the residual registers are free again: request the first unit of this warp's next row
        if (res_base && u + unit_step >= units && k + 1 < total) load_res(k + 1, unit0, rres);
        if (pooling) {
          // Fused global average pool: the stored value hi + lo of each of the 16 channels, summed
          // over the columns this warp holds (lanes that differ in the column bits), then added to
          // this warp's partial sums [image][16 channels] in shared memory.  The tensor is not stored.
          float* mine = s_pool + ((size_t)(warp - 2) * Gout + img) * 16;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            float a = __uint_as_float(hi[e] << 16) + __uint_as_float(lo[e] << 16);
            float b = __uint_as_float(hi[e] & 0xFFFF0000u) + __uint_as_float(lo[e] & 0xFFFF0000u);
            for (int o = Gout; o < 32; o <<= 1) {
              a += __shfl_xor_sync(0xffffffffu, a, o);
              b += __shfl_xor_sync(0xffffffffu, b, o);
            }
            // channel of word e of [hi plane 0 | hi plane 1]: words 0-3 = channels 0-7, 4-7 = channels 8-15
            if (lane < Gout) { mine[2 * e] += a; mine[2 * e + 1] += b; }
          }
        } else {
        uint8_t* dst = out_base + row_off + uoff;
        *reinterpret_cast<uint4*>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(dst + plane_bytes) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        *reinterpret_cast<uint4*>(dst + (size_t)lo_plane0 * plane_bytes) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        *reinterpret_cast<uint4*>(dst + (size_t)(lo_plane0 + 1) * plane_bytes) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        }
      }
      if (pooling && (k + 1) % rows_mine == 0) {
        // last row of an item for this warp: once all epilogue warps are here, the partial sums of the
        // warps that hold a channel's chunk are added in a fixed order and the means leave for global memory
        const int n_epi = n_threads - 64;
        const uint32_t pool_parity = (uint32_t)(il & 1);
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_pool);
        alive = mbar_wait_warp(bar_pool, pool_parity, s_abort, p.error_flag);
        if (!alive) break;
        const int item = (int)blockIdx.x + il * (int)gridDim.x;
        for (int i = tid - 64; i < Gout * N; i += n_epi) {
          const int im = i / N, c = i - im * N;
          float sum = 0.f;
          for (int e = 0; e < 4 * WQ; ++e) {
            const int eh = e >> 2;                                    // index of warp e among the warps of its quarter
            const int eu = units >= WQ ? eh : eh % units;             // its unit
            if ((eu % chunks) * 16 == (c & ~15)) sum += s_pool[((size_t)e * Gout + im) * 16 + (c & 15)];
          }
          const int b = item * Gout + im;
          if (b < p.batch) job.pool[(size_t)b * p.cout_total + n_off + c] = sum * pool_scale;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_pool + 8);
        alive = mbar_wait_warp(bar_pool + 8, pool_parity, s_abort, p.error_flag);
        if (!alive) break;
        for (int i = lane; i < Gout * 16; i += 32) s_pool[(size_t)(warp - 2) * Gout * 16 + i] = 0.f;
        __syncwarp();
      }
    }
  }

  // ---- teardown -----------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

// ---------------------------------------------------------------------------------------------
// A whole basic block in one kernel:  out = relu( conv2( relu(conv1(x)) ) + x ),  both convolutions
// 3x3 at stride 1 with C -> C channels (C = 16 or 32, 8 images per group, 4- / 8-bit weights).
// The intermediate tensor never leaves the SM: the first epilogue writes each finished row of it
// into a shared-memory ring in the layout the TMA gives input rows (zero columns on both sides
// included), where the second convolution's MMAs read it; the shortcut x[y] is read from the input
// ring, which keeps a row until the output row at the same height is finished.  Per block the
// kernel reads x once and writes out once: 2 tensors instead of 5.
//
// Warps: 0 TMA producer, 1 MMA issuer of conv1, 2 MMA issuer of conv2 (each hides the other's
// per-row bookkeeping), 3-10 first epilogue (accumulators -> shared memory), 11-18 second
// epilogue (accumulators + shortcut -> global memory).  Tensor memory: columns 0-255 hold the
// ring of conv1 rows, 256-511 the ring of conv2 rows.
// ---------------------------------------------------------------------------------------------
constexpr int kRbThreads = 19 * 32;
constexpr int kRbSlots = 8;
constexpr int kRbMaxIn = 6, kRbMaxMid = 4;

struct RbParams {
  int H, W;
  int n_items;
  int rows_per_version;
  int in_stages, mid_stages;
  int K;                  // elements of a packed weight row (9 C)
  int stage_bytes, a_lbo, xt;
  int32_t* error_flag;
};

struct RbSmem { int in_ring, mid_ring, w1, w2, coef, rows, bars, total; };
__host__ __device__ inline RbSmem rb_smem(int in_stages, int mid_stages, int stage_bytes, int C) {
  RbSmem s;
  const int wbytes = 3 * (C / 8) * 3 * C * 16;
  s.in_ring = 0;
  s.mid_ring = in_stages * stage_bytes;
  s.w1 = s.mid_ring + mid_stages * stage_bytes;
  s.w2 = s.w1 + wbytes;
  s.coef = s.w2 + wbytes;                                // scale1, bias1, scale2, bias2
  s.rows = (s.coef + 4 * C * 4 + 127) / 128 * 128;
  s.bars = s.rows + kRsMaxRows * kRsRowWords * 4;
  s.total = s.bars + (2 * kRbMaxIn + 2 * kRbMaxMid + 4 * kRbSlots + 1) * 8 + 16;
  return s;
}

template <int C>
__global__ void __launch_bounds__(kRbThreads, 1)
conv_rs_block_kernel(const __grid_constant__ CUtensorMap in_map, RbParams p, const LayerJob* __restrict__ jobs) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const LayerJob job = jobs[blockIdx.y];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int N = C, NB = 3 * C, KCH = C / 8, R = kRbSlots;
  constexpr int tile_b = KCH * NB * 16;
  const int S_in = p.in_stages, S_mid = p.mid_stages;
  const RbSmem sm = rb_smem(S_in, S_mid, p.stage_bytes, C);
  uint8_t* in_ring = smem;
  uint8_t* mid_ring = smem + sm.mid_ring;
  uint8_t* w1 = smem + sm.w1;
  uint8_t* w2 = smem + sm.w2;
  float* s_coef = reinterpret_cast<float*>(smem + sm.coef);
  RowProgram* s_rows = reinterpret_cast<RowProgram*>(smem + sm.rows);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
  const uint32_t bar_in_full = smem_u32(bars);
  const uint32_t bar_in_free = bar_in_full + 8 * kRbMaxIn;
  const uint32_t bar_mid_full = bar_in_free + 8 * kRbMaxIn;
  const uint32_t bar_mid_free = bar_mid_full + 8 * kRbMaxMid;
  const uint32_t bar_a1_full = bar_mid_free + 8 * kRbMaxMid;
  const uint32_t bar_a1_empty = bar_a1_full + 8 * R;
  const uint32_t bar_a2_full = bar_a1_empty + 8 * R;
  const uint32_t bar_a2_empty = bar_a2_full + 8 * R;
  const uint32_t bar_w = bar_a2_empty + 8 * R;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * kRbMaxIn + 2 * kRbMaxMid + 4 * R + 1);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  if (tid == 0) {
    for (int i = 0; i < kRbMaxIn; ++i) {
      mbar_init(bar_in_full + 8 * i, 1);
      mbar_init(bar_in_free + 8 * i, 1 + 4);           // conv1's MMAs retired + the four shortcut readers of the row
    }
    for (int i = 0; i < kRbMaxMid; ++i) {
      mbar_init(bar_mid_full + 8 * i, 4);              // the four warps of the first epilogue that take the row
      mbar_init(bar_mid_free + 8 * i, 1);
    }
    for (int i = 0; i < R; ++i) {
      mbar_init(bar_a1_full + 8 * i, 1);
      mbar_init(bar_a1_empty + 8 * i, 4);
      mbar_init(bar_a2_full + 8 * i, 1);
      mbar_init(bar_a2_empty + 8 * i, 4);
    }
    mbar_init(bar_w, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 1) {
    tmem_alloc(smem_u32(s_tmem), 512);
    tmem_relinquish();
  }
  // packed weights of both convolutions -> the (still unused) input ring, then expansion
  const int kpad = (p.K + 31) / 32 * 32;
  const uint32_t wrow1 = (uint32_t)kpad * job.bits_pre / 8, wrow2 = (uint32_t)kpad * job.bits / 8;
  const uint32_t packed1 = wrow1 * N, packed2 = wrow2 * N;
  if (tid == 0) {
    mbar_expect_tx(bar_w, packed1 + packed2);
    bulk_load(smem_u32(in_ring), job.w_pre, packed1, bar_w);
    bulk_load(smem_u32(in_ring) + packed1, job.w, packed2, bar_w);
  }
  for (int i = tid; i < N; i += kRbThreads) {
    s_coef[i] = job.scale_pre[i];
    s_coef[N + i] = job.bias_pre[i];
    s_coef[2 * N + i] = job.scale[i];
    s_coef[3 * N + i] = job.bias[i];
  }
  if (tid < p.H) s_rows[tid] = rs_row_program<3, 1>(tid, p.H, p.H, N, R);
  // the zero columns on both sides of every row of the intermediate ring are written once, here
  for (int i = tid; i < S_mid * p.stage_bytes / 16; i += kRbThreads)
    reinterpret_cast<uint4*>(mid_ring)[i] = make_uint4(0u, 0u, 0u, 0u);
  bool alive = mbar_wait_warp(bar_w, 0, s_abort, p.error_flag);
  if (alive) {
    rs_expand_weights<C, 3, 1, 1>(in_ring, wrow1, job.bits_pre, N, w1, tid, kRbThreads);
    rs_expand_weights<C, 3, 1, 1>(in_ring + packed1, wrow2, job.bits, N, w2, tid, kRbThreads);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  alive = alive && (*s_abort == 0);

  const int n_my_items = ((int)blockIdx.x < p.n_items) ? (p.n_items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  const int total = n_my_items * p.H;                  // rows this CTA streams, numbered g = item_local * H + y
  // operand constants of the MMA issuers
  const uint32_t a_lbo_field = ((uint32_t)p.a_lbo >> 4) << 16;
  const uint32_t a_part_step = ((uint32_t)KCH * (uint32_t)p.a_lbo) >> 4, a_kk_step = (2u * (uint32_t)p.a_lbo) >> 4;
  const uint32_t b_tile_step = (uint32_t)tile_b >> 4, b_kk_step = 2u * (uint32_t)NB;
  const uint32_t b_lbo_field = ((uint32_t)(NB * 16) >> 4) << 16;
  const uint32_t tap1 = 128u, tap2 = 256u;             // one column = 8 images x 16 bytes

  if (warp == 0) {
    if (lane == 0 && alive) {
      uint32_t issued = 0, issued_phase = 0;
      for (int g = 0; g < total && alive; ++g) {
        const int il = g / p.H, y = g - il * p.H;
        const uint32_t stage = (uint32_t)(g % S_in), phase = (uint32_t)((g / S_in) & 1);
        alive = mbar_wait(bar_in_free + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
        if (!alive) break;
        issued |= 1u << stage;
        issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
        mbar_expect_tx(bar_in_full + 8 * stage, (uint32_t)p.stage_bytes);
        const int item = (int)blockIdx.x + il * (int)gridDim.x;
        tma_load_4d(smem_u32(in_ring) + stage * p.stage_bytes, &in_map, bar_in_full + 8 * stage, 0, -1, 0,
                    job.in_version * p.rows_per_version + item * p.H + y);
      }
      for (int i = 0; i < S_in; ++i)
        if (issued & (1u << i)) {
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_in_full + 8 * i, (issued_phase >> i) & 1u) && clock64() - t0 < kWaitLimitCycles) {}
        }
    }
  } else if (warp == 1 || warp == 2) {
    // conv1 streams the input ring into accumulator ring 1; conv2 streams the intermediate ring into
    // accumulator ring 2.  Same row programs: both are 3x3, stride 1, on H rows.
    const bool second = warp == 2;
    const uint32_t bar_src_full = second ? bar_mid_full : bar_in_full;
    const uint32_t bar_src_free = second ? bar_mid_free : bar_in_free;
    const uint32_t bar_acc_full = second ? bar_a2_full : bar_a1_full;
    const uint32_t bar_acc_empty = second ? bar_a2_empty : bar_a1_empty;
    const int S = second ? S_mid : S_in;
    const uint32_t src_ring = smem_u32(second ? mid_ring : in_ring);
    const uint32_t w_lo0 = (smem_u32(second ? w2 : w1) >> 4) | b_lbo_field;
    const uint32_t d_base = tmem_base + (second ? 256u : 0u);
    for (int g = 0; g < total && alive; ++g) {
      const int il = g / p.H, y = g - il * p.H;
      const RowRegs rr = rs_load_row(s_rows[y]);
      const int fresh_row = (int)(rr.w4.y & 255u), n_fresh = (int)(rr.w4.y >> 8);
      for (int i = 0; i < n_fresh && alive; ++i) {
        const int q = il * p.H + fresh_row + i;
        alive = mbar_wait_warp(bar_acc_empty + 8 * (q & (R - 1)), ((q / R) & 1) ^ 1u, s_abort, p.error_flag);
      }
      if (!alive) break;
      const uint32_t stage = (uint32_t)(g % S), phase = (uint32_t)((g / S) & 1);
      alive = mbar_wait_warp(bar_src_full + 8 * stage, phase, s_abort, p.error_flag);
      if (!alive) break;
      tc_fence_after();
      const uint32_t a_stage = src_ring + stage * p.stage_bytes;
      for (int xt = 0; xt < p.xt; ++xt)
        rs_issue_row<C, 3, 1>(rr, d_base + (uint32_t)(xt * R * N), ((a_stage + (uint32_t)xt * kRsTileBytes) >> 4) | a_lbo_field,
                              0u, tap1, tap2, a_part_step, a_kk_step, w_lo0, b_tile_step, b_kk_step);
      umma_commit(bar_src_free + 8 * stage);
      // rows complete with this one (H is a multiple of the ring depth, so the slot is the row's low bits)
      if (rr.w4.z & 255u) umma_commit(bar_acc_full + 8 * (((rr.w4.z & 255u) - 1u) & (uint32_t)(R - 1)));
      if (rr.w4.z >> 8) umma_commit(bar_acc_full + 8 * (((rr.w4.z >> 8) - 1u) & (uint32_t)(R - 1)));
    }
  } else {
    // Each quarter of the accumulator lanes has two warps per epilogue; they take alternate rows, and
    // a warp finishes both 16-channel units of its row, so two rows per epilogue are in flight.
    const bool second = warp >= 11;
    const int qd = warp & 3;
    const int h = ((second ? warp - 11 : warp - 3) >> 2);       // 0 or 1: the parity of the rows this warp takes
    const int l = qd * 32 + lane;
    const int x_local = l >> 3, img = l & 7;
    constexpr int chunks = N / 16;                               // units of a row: (column tile, chunk), two in all
    constexpr int lo_plane0 = C / 8;
    const uint32_t bar_acc_full = second ? bar_a2_full : bar_a1_full;
    const uint32_t bar_acc_empty = second ? bar_a2_empty : bar_a1_empty;
    const float* scale = s_coef + (second ? 2 * N : 0);
    const float* bias = s_coef + (second ? 3 * N : N);
    const size_t plane_bytes = 128, px_bytes = (size_t)(C / 4) * 128;
    uint8_t* out_base = static_cast<uint8_t*>(job.out);
    // per unit: accumulator column and offset of this lane's cell inside a ring stage (first hi plane of the chunk)
    uint32_t t_col[2], cell[2];
    int ux[2], uph[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int xt = u / chunks, c0 = (u - xt * chunks) * 16;
      ux[u] = xt * 16 + x_local;
      uph[u] = c0 >> 3;
      t_col[u] = (second ? 256u : 0u) + (uint32_t)(xt * R * N + c0);
      cell[u] = (uint32_t)uph[u] * (uint32_t)p.a_lbo + (uint32_t)(ux[u] + 1) * 128u + (uint32_t)img * 16u;
    }
    for (int g = h; g < total && alive; g += 2) {
      const int il = g / p.H, y = g - il * p.H;
      const int slot = g & (R - 1);
      uint32_t v0[16], v1[16];
      uint32_t hi[8], lo[8];
      alive = mbar_wait_warp(bar_acc_full + 8 * slot, (g / R) & 1, s_abort, p.error_flag);
      if (!alive) break;
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)(slot * N);
      tmem_ld16(t_row + t_col[0], v0);
      tmem_ld16(t_row + t_col[1], v1);
      if (!second) {
        const uint32_t ms = (uint32_t)(g % S_mid), mphase = (uint32_t)((g / S_mid) & 1);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acc_empty + 8 * slot);
        // the stage of the intermediate ring must have been read by conv2's MMAs of its last occupant
        alive = mbar_wait_warp(bar_mid_free + 8 * ms, mphase ^ 1u, s_abort, p.error_flag);
        if (!alive) break;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int c0 = (u % chunks) * 16;
          rs_finish_unit(u == 0 ? v0 : v1, scale + c0, bias + c0, nullptr, false, AIQ_ACT_RELU, hi, lo);
          uint8_t* dst = mid_ring + ms * p.stage_bytes + cell[u];
          *reinterpret_cast<uint4*>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(dst + p.a_lbo) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
          *reinterpret_cast<uint4*>(dst + lo_plane0 * p.a_lbo) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          *reinterpret_cast<uint4*>(dst + (lo_plane0 + 1) * p.a_lbo) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_mid_full + 8 * ms);
      } else {
        const uint32_t is = (uint32_t)(g % S_in), iphase = (uint32_t)((g / S_in) & 1);
        // shortcut: the block input at the same row, still in the input ring (its copy completed long
        // ago; observing the barrier makes the data visible to this thread)
        alive = mbar_wait_warp(bar_in_full + 8 * is, iphase, s_abort, p.error_flag);
        uint4 r0[4], r1[4];
        {
          const uint8_t* src = in_ring + is * p.stage_bytes;
          r0[0] = *reinterpret_cast<const uint4*>(src + cell[0]);
          r0[1] = *reinterpret_cast<const uint4*>(src + cell[0] + p.a_lbo);
          r0[2] = *reinterpret_cast<const uint4*>(src + cell[0] + lo_plane0 * p.a_lbo);
          r0[3] = *reinterpret_cast<const uint4*>(src + cell[0] + (lo_plane0 + 1) * p.a_lbo);
          r1[0] = *reinterpret_cast<const uint4*>(src + cell[1]);
          r1[1] = *reinterpret_cast<const uint4*>(src + cell[1] + p.a_lbo);
          r1[2] = *reinterpret_cast<const uint4*>(src + cell[1] + lo_plane0 * p.a_lbo);
          r1[3] = *reinterpret_cast<const uint4*>(src + cell[1] + (lo_plane0 + 1) * p.a_lbo);
        }
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acc_empty + 8 * slot);
        if (!alive) break;
        const int item = (int)blockIdx.x + il * (int)gridDim.x;
        uint8_t* row_dst = out_base + ((size_t)item * p.H + y) * p.W * px_bytes + (size_t)img * 16;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int c0 = (u % chunks) * 16;
          rs_finish_unit(u == 0 ? v0 : v1, scale + c0, bias + c0, u == 0 ? r0 : r1, true, AIQ_ACT_RELU, hi, lo);
          uint8_t* dst = row_dst + (size_t)ux[u] * px_bytes + (size_t)uph[u] * plane_bytes;
          *reinterpret_cast<uint4*>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(dst + plane_bytes) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
          *reinterpret_cast<uint4*>(dst + (size_t)lo_plane0 * plane_bytes) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          *reinterpret_cast<uint4*>(dst + (size_t)(lo_plane0 + 1) * plane_bytes) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        }
        // the shortcut words have been used, so their loads have returned: only now may the TMA refill the stage
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_in_free + 8 * is);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn rs_encode_fn() {
  static std::atomic<EncodeTiledFn> fn{nullptr};
  if (EncodeTiledFn f = fn.load(std::memory_order_acquire)) return f;
  void* sym = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess)
    return nullptr;
  fn.store(reinterpret_cast<EncodeTiledFn>(sym), std::memory_order_release);
  return reinterpret_cast<EncodeTiledFn>(sym);
}

// geometry shared by the map encoder and the launcher
struct RsShape {
  int Gin, Gout, gmode, planes, xt, stage_bytes, a_lbo, a_tap_off[3];
};

bool rs_shape(const ConvGeom& g, RsShape* s) {
  if (g.in_is_nchw || g.act_format != ACT_RS) return false;
  if (!((g.ks == 3 && g.pad == 1) || (g.ks == 1 && g.pad == 0))) return false;
  if (g.stride != 1 && g.stride != 2) return false;
  if (g.Cin != 16 && g.Cin != 32 && g.Cin != 64) return false;
  if (g.Cout != 16 && g.Cout != 32 && g.Cout != 64) return false;
  if (g.W % 8 != 0 || g.Wo % 8 != 0 || g.W > 64 || g.H < 2 || g.H > kRsMaxRows || g.Ho % 4 != 0) return false;
  if (g.stride == 2 && ((g.H & 1) || (g.W & 1))) return false;
  s->Gin = rs_group_images(g.W);
  s->Gout = rs_group_images(g.Wo);
  s->planes = g.Cin / 4;
  if (s->Gin == 8 && s->Gout == 8) s->gmode = 0;
  else if (s->Gin == 16 && s->Gout == 16) s->gmode = 1;
  else if (s->Gin == 8 && s->Gout == 16 && g.stride == 2 && g.W == 16) s->gmode = 2;
  else return false;
  if (s->gmode == 1 && g.stride != 1) return false;
  const int X = s->gmode == 0 ? 16 : 8;
  s->xt = g.Wo / X;
  const int gb = s->Gin * 16;                        // bytes of one (column, plane) cell
  s->a_tap_off[0] = s->a_tap_off[1] = s->a_tap_off[2] = 0;
  if (g.stride == 1) {
    const int cols = g.ks == 3 ? g.W + 2 : g.W;
    s->a_lbo = cols * gb;
    s->stage_bytes = s->planes * s->a_lbo;
    if (g.ks == 3) for (int t = 0; t < 3; ++t) s->a_tap_off[t] = t * gb;
  } else if (s->gmode == 0) {
    if (g.ks == 3) {
      const int pairs = g.W / 2 + 1;                 // pair -1 .. W/2 - 1
      s->a_lbo = 2 * pairs * gb;                     // [plane][parity][pair]
      s->stage_bytes = s->planes * s->a_lbo;
      s->a_tap_off[0] = pairs * gb;                  // odd columns, from pair -1
      s->a_tap_off[1] = gb;                          // even columns, from pair 0
      s->a_tap_off[2] = pairs * gb + gb;             // odd columns, from pair 0
    } else {
      s->a_lbo = (g.W / 2) * gb;
      s->stage_bytes = s->planes * s->a_lbo;
    }
  } else {
    // 8 -> 16 images per group: per load [plane][half of the output group][8 column pairs][128 bytes]
    s->a_lbo = 2048;
    const int sub = s->planes * 2048;
    s->stage_bytes = (g.ks == 3 ? 3 : 1) * sub;
    if (g.ks == 3) for (int t = 0; t < 3; ++t) s->a_tap_off[t] = t * sub;
  }
  return true;
}

int rs_weight_slices(const ConvGeom& g, int weight_bits) { return (weight_bits > 8 && g.Cout == 64) ? 2 : 1; }

int rs_weight_bytes(const ConvGeom& g, int weight_bits) {
  const int pieces = weight_bits > 8 ? 2 : 1;
  const int n = g.Cout / rs_weight_slices(g, weight_bits);
  return pieces * rs_taps(g.ks) * (g.Cin / 8) * (g.ks == 3 ? 3 : 1) * n * 16;
}

// Launch configuration of one layer and weight class.
struct RsConfig { int slices, N, occ, stages, slots, threads, tmem_cols, pool_bytes, smem_bytes; bool ok; };

RsConfig rs_config(const ConvGeom& g, const RsShape& sh, int weight_bits, int smem_optin, bool pool) {
  RsConfig c = {};
  c.slices = rs_weight_slices(g, weight_bits);
  c.N = g.Cout / c.slices;
  const int wbytes = rs_weight_bytes(g, weight_bits);
  const int packed = c.N * (int)row_bytes(g.K, weight_bits <= 8 ? 8 : weight_bits);
  // Two CTAs per SM where two rings of at least three input rows and two copies of the weights fit
  // (the 16- and 32-channel layers), else one CTA with as deep a ring as fits.
  const int per_cta = (smem_optin + 1024) / 2 - 1024;   // an SM holds the opt-in limit + 1 KB; each CTA reserves 1 KB
  auto fits = [&](int st, int limit, int pool_bytes) {
    return rs_smem(st, sh.stage_bytes, wbytes, c.N, pool_bytes).total + 1024 <= limit && packed <= st * sh.stage_bytes;
  };
  for (int occ = 2; occ >= 1 && !c.stages; --occ) {
    const int threads = (2 + (occ == 2 ? 8 : kRsMaxEpiWarps)) * 32;
    const int pool_bytes = pool ? (threads / 32 - 2) * sh.Gout * 16 * 4 : 0;
    // output rows in flight: a power of two that divides the rows of an item (the slot of a row then
    // does not depend on the item) and fits the CTA's share of tensor memory
    const int tmem_cols = 512 / occ;
    int slots = kRsMaxSlots;
    while (slots > 4 && (sh.xt * slots * c.N > tmem_cols || g.Ho % slots != 0)) slots >>= 1;
    if (sh.xt * slots * c.N > tmem_cols || g.Ho % slots != 0) continue;
    for (int st = kRsMaxStages; st >= (occ == 2 ? 3 : 2); --st)
      if (fits(st, occ == 2 ? per_cta : smem_optin, pool_bytes)) {
        c.occ = occ; c.stages = st; c.slots = slots; c.threads = threads; c.tmem_cols = tmem_cols; c.pool_bytes = pool_bytes;
        c.smem_bytes = rs_smem(st, sh.stage_bytes, wbytes, c.N, pool_bytes).total + 1024;
        break;
      }
  }
  c.ok = c.stages > 0;
  return c;
}

template <int C, int KS, int STRIDE, int PIECES>
aiq_status_t launch_rs(const ConvGeom& g, const RsShape& sh, const CUtensorMap* maps, const LayerJob* jobs_dev, int n_jobs,
                       int batch_capacity, int32_t* error_flag, double weight_bytes, int weight_bits, bool pool_jobs,
                       cudaStream_t s) {
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  const RsConfig c = rs_config(g, sh, weight_bits, props.smem_optin, pool_jobs);
  if (!c.ok) return set_error(AIQ_ERR_SHAPE, "conv_rs: shared or tensor memory does not fit (%d bytes per input row)", sh.stage_bytes);
  RsParams p = {};
  p.H = g.H; p.W = g.W; p.Ho = g.Ho; p.Wo = g.Wo; p.N = c.N; p.cout_total = g.Cout; p.act = g.act;
  p.gmode = sh.gmode;
  p.n_items = rs_padded_batch(g.B) / sh.Gout;
  p.rows_per_version = rs_padded_batch(batch_capacity) / sh.Gin * g.H;
  p.n_stages = c.stages; p.n_slots = c.slots; p.tmem_cols = c.tmem_cols;
  p.K = g.K; p.stage_bytes = sh.stage_bytes; p.a_lbo = sh.a_lbo; p.xt = sh.xt;
  for (int t = 0; t < 3; ++t) p.a_tap_off[t] = sh.a_tap_off[t];
  p.error_flag = error_flag;
  p.batch = g.B;
  p.pool_bytes = c.pool_bytes;
  AIQ_ENSURE_DYNAMIC_SMEM((conv_rs_kernel<C, KS, STRIDE, PIECES>), props.smem_optin);
  int ctas = c.occ * props.n_sms / (n_jobs * c.slices);
  if (ctas > p.n_items) ctas = p.n_items;
  if (ctas < 1) ctas = 1;
  {
    LaunchScope scope(AIQ_KERNEL_CONV_TC, s,
                      2.0 * g.B * g.Ho * g.Wo * g.Cout * (double)(g.ks * g.ks * g.Cin) * n_jobs,
                      weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W +
                                                     (pool_jobs ? 0.0 : (double)g.B * g.Ho * g.Wo * g.Cout)));
    conv_rs_kernel<C, KS, STRIDE, PIECES><<<dim3(ctas, n_jobs, c.slices), c.threads, c.smem_bytes, s>>>(maps[0], maps[1], p, jobs_dev);
  }
  AIQ_LAUNCH_CHECK("conv_rs");
  return AIQ_OK;
}

bool rb_shape_ok(const ConvGeom& g) {
  if (g.in_is_nchw || g.act_format != ACT_RS) return false;
  if (g.ks != 3 || g.pad != 1 || g.stride != 1 || g.Cin != g.Cout) return false;
  if (!((g.Cin == 16 && g.W == 32) || (g.Cin == 32 && g.W == 16))) return false;   // two epilogue units per row
  return g.H % kRbSlots == 0 && g.H <= kRsMaxRows && g.Ho == g.H && g.Wo == g.W;
}

template <int C>
aiq_status_t launch_rb(const ConvGeom& g, const CUtensorMap* map, const LayerJob* jobs_dev, int n_jobs, int batch_capacity,
                       int32_t* error_flag, double weight_bytes, cudaStream_t s) {
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  RbParams p = {};
  p.H = g.H; p.W = g.W;
  p.n_items = rs_padded_batch(g.B) / 8;
  p.rows_per_version = rs_padded_batch(batch_capacity) / 8 * g.H;
  p.K = g.K;
  p.a_lbo = (g.W + 2) * 128;
  p.stage_bytes = (C / 4) * p.a_lbo;
  p.xt = g.W / 16;
  p.error_flag = error_flag;
  int in_stages = kRbMaxIn, mid_stages = kRbMaxMid;
  while (rb_smem(in_stages, mid_stages, p.stage_bytes, C).total + 1024 > props.smem_optin && (in_stages > 4 || mid_stages > 3)) {
    if (in_stages > 4 && in_stages - mid_stages >= 2) --in_stages; else if (mid_stages > 3) --mid_stages; else --in_stages;
  }
  const int smem_bytes = rb_smem(in_stages, mid_stages, p.stage_bytes, C).total + 1024;
  const int packed = 2 * C * (int)row_bytes(g.K, 8);
  if (smem_bytes > props.smem_optin || packed > in_stages * p.stage_bytes)
    return set_error(AIQ_ERR_SHAPE, "conv_rs_block: %d bytes of shared memory needed", smem_bytes);
  p.in_stages = in_stages; p.mid_stages = mid_stages;
  AIQ_ENSURE_DYNAMIC_SMEM(conv_rs_block_kernel<C>, props.smem_optin);
  int ctas = props.n_sms / n_jobs;
  if (ctas > p.n_items) ctas = p.n_items;
  if (ctas < 1) ctas = 1;
  {
    const double px = (double)g.B * g.H * g.W * C;
    LaunchScope scope(AIQ_KERNEL_CONV_TC, s, 2.0 * 2.0 * px * (9.0 * C) * n_jobs, weight_bytes + 4.0 * n_jobs * 2.0 * px);
    conv_rs_block_kernel<C><<<dim3(ctas, n_jobs), kRbThreads, smem_bytes, s>>>(map[0], p, jobs_dev);
  }
  AIQ_LAUNCH_CHECK("conv_rs_block");
  return AIQ_OK;
}

}  // namespace

bool conv_rs_eligible(const ConvGeom& g) {
  RsShape s;
  if (!rs_shape(g, &s)) return false;
  DeviceProps props;
  int smem_limit = 227 * 1024;
  if (current_device_props(&props) == AIQ_OK) smem_limit = props.smem_optin;
  for (int bits : {8, 16, 32})
    if (!rs_config(g, s, bits, smem_limit, false).ok) return false;
  return true;
}

// The average pool can ride in the epilogue when every warp of the epilogue finishes one unit of a row.
bool conv_rs_pool_fusable(const ConvGeom& g) {
  RsShape s;
  if (!rs_shape(g, &s) || s.gmode == 2) return false;
  DeviceProps props;
  if (current_device_props(&props) != AIQ_OK) return false;
  for (int bits : {8, 16, 32}) {
    const RsConfig c = rs_config(g, s, bits, props.smem_optin, true);
    if (!c.ok || s.xt * (c.N / 16) > (c.threads / 32 - 2) / 4) return false;
  }
  return true;
}

aiq_status_t conv_rs_encode_maps(const ConvGeom& g, const void* slot_base, int batch_capacity, int n_versions,
                                 void* maps_out /* 2 x 128 bytes */) {
  EncodeTiledFn enc = rs_encode_fn();
  if (!enc) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  RsShape s;
  if (!rs_shape(g, &s)) return set_error(AIQ_ERR_SHAPE, "conv_rs: layer shape is not supported");
  CUtensorMap* maps = static_cast<CUtensorMap*>(maps_out);
  const cuuint64_t gb = (cuuint64_t)s.Gin * 16;                         // bytes of a (column, plane) cell
  const cuuint64_t col_bytes = (cuuint64_t)s.planes * gb;               // one column of a group
  const cuuint64_t row_bytes_ = (cuuint64_t)g.W * col_bytes;            // one row of a group
  const cuuint64_t rows = (cuuint64_t)n_versions * (rs_padded_batch(batch_capacity) / s.Gin) * g.H;
  void* base = const_cast<void*>(slot_base);
  CUresult r = CUDA_SUCCESS;
  const cuuint32_t one[5] = {1, 1, 1, 1, 1};
  if (g.stride == 1) {
    // (image x 8 channels, column, plane, row over all groups and versions)
    cuuint64_t dims[4] = {(cuuint64_t)s.Gin * 8, (cuuint64_t)g.W, (cuuint64_t)s.planes, rows};
    cuuint64_t strides[3] = {col_bytes, gb, row_bytes_};
    cuuint32_t box[4] = {(cuuint32_t)s.Gin * 8, (cuuint32_t)(g.ks == 3 ? g.W + 2 : g.W), (cuuint32_t)s.planes, 1u};
    r = enc(&maps[0], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, one, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    maps[1] = maps[0];
  } else if (s.gmode == 0) {
    // (image x 8 channels, column pair, column parity, plane, row)
    cuuint64_t dims[5] = {(cuuint64_t)s.Gin * 8, (cuuint64_t)g.W / 2, 2, (cuuint64_t)s.planes, rows};
    cuuint64_t strides[4] = {2 * col_bytes, col_bytes, gb, row_bytes_};
    cuuint32_t box[5] = {(cuuint32_t)s.Gin * 8, (cuuint32_t)(g.ks == 3 ? g.W / 2 + 1 : g.W / 2), g.ks == 3 ? 2u : 1u,
                         (cuuint32_t)s.planes, 1u};
    r = enc(&maps[0], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, one, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    maps[1] = maps[0];
  } else {
    // two input groups of 8 images feed one output group of 16: (image x 8 channels, column pair,
    // group of the pair, plane, row), one map over the even columns and one over the odd ones
    const cuuint64_t group_bytes = (cuuint64_t)g.H * row_bytes_;
    cuuint64_t dims[5] = {64, (cuuint64_t)g.W / 2, 2, (cuuint64_t)s.planes, rows};
    cuuint64_t strides[4] = {2 * col_bytes, group_bytes, gb, row_bytes_};
    cuuint32_t box[5] = {64u, 8u, 2u, (cuuint32_t)s.planes, 1u};
    for (int par = 0; par < 2 && r == CUDA_SUCCESS; ++par)
      r = enc(&maps[par], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, static_cast<uint8_t*>(base) + par * col_bytes, dims, strides, box,
              one, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled (row-streaming convolution) failed with code %d", (int)r);
  return AIQ_OK;
}

aiq_status_t launch_conv_rs(const ConvGeom& g, const void* maps, const LayerJob* jobs_dev, int n_jobs, int batch_capacity,
                            int32_t* error_flag, double weight_bytes, int weight_bits, bool pool_jobs, cudaStream_t s) {
  RsShape sh;
  if (!rs_shape(g, &sh)) return set_error(AIQ_ERR_SHAPE, "conv_rs: layer shape is not supported");
  const CUtensorMap* m = static_cast<const CUtensorMap*>(maps);
#define AIQ_RS_ARGS g, sh, m, jobs_dev, n_jobs, batch_capacity, error_flag, weight_bytes, weight_bits, pool_jobs, s
#define AIQ_RS_KS(C_, P_)                                                                              \
  do {                                                                                                \
    if (g.ks == 3) return g.stride == 1 ? launch_rs<C_, 3, 1, P_>(AIQ_RS_ARGS) : launch_rs<C_, 3, 2, P_>(AIQ_RS_ARGS); \
    return g.stride == 1 ? launch_rs<C_, 1, 1, P_>(AIQ_RS_ARGS) : launch_rs<C_, 1, 2, P_>(AIQ_RS_ARGS); \
  } while (0)
#define AIQ_RS_C(C_)                                  \
  if (g.Cin == C_) {                                  \
    if (weight_bits <= 8) AIQ_RS_KS(C_, 1);           \
    AIQ_RS_KS(C_, 2);                                 \
  }
  AIQ_RS_C(16) AIQ_RS_C(32) AIQ_RS_C(64)
#undef AIQ_RS_C
#undef AIQ_RS_KS
#undef AIQ_RS_ARGS
  return set_error(AIQ_ERR_SHAPE, "conv_rs: no kernel for Cin=%d", g.Cin);
}

bool conv_rs_block_eligible(const ConvGeom& g) { return rb_shape_ok(g); }

aiq_status_t launch_conv_rs_block(const ConvGeom& g, const void* maps, const LayerJob* jobs_dev, int n_jobs, int batch_capacity,
                                  int32_t* error_flag, double weight_bytes, cudaStream_t s) {
  if (!rb_shape_ok(g)) return set_error(AIQ_ERR_SHAPE, "conv_rs_block: layer shape is not supported");
  const CUtensorMap* m = static_cast<const CUtensorMap*>(maps);
  if (g.Cin == 16) return launch_rb<16>(g, m, jobs_dev, n_jobs, batch_capacity, error_flag, weight_bytes, s);
  return launch_rb<32>(g, m, jobs_dev, n_jobs, batch_capacity, error_flag, weight_bytes, s);
}

}  // namespace aiq
