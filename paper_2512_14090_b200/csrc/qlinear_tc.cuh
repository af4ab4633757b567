// Quantized linear layer at batch sizes where it is a dense contraction (M >= 9), on the
// tcgen05 tensor cores.  Included by conv_tc.cu (shares its PTX wrappers); not a stand-alone
// translation unit.
//
//   y[m][n] = s_n * sum_k code[n][k] * x[m][k] + bias[n]           (4- and 8-bit weights)
//
// The weight matrix is the M operand of the MMA (128 output channels per CTA) and the batch
// is its N operand (up to 256 batch rows per CTA), so the packed weights - the bytes that
// bound the layer at small batch - are read from memory exactly once:
//   D[128 n][Mt m] += A[128 n][64 k] * B[Mt m][64 k]^T     per chunk of 64 k,
// A = integer codes expanded to bfloat16 in shared memory (exact), B = the activations as
// the sum of two bfloat16 (hi + lo, 16+ significant bits), one MMA group for each half.
// A pre-pass writes the two bfloat16 planes of x into the caller's workspace (and zeroes y
// when K is split over several CTAs); the main kernel starts under programmatic dependent
// launch, so its weight prefetch overlaps the pre-pass.
//   warp 0      TMA producer of the B tiles (hi and lo planes, Mt rows x 64 k, 128-byte swizzle)
//   warp 1      MMA issuer (converged warp, elected lane)
//   warps 2-5   epilogue: TMEM -> scale, bias -> y (a lane owns an output channel, so a
//               warp-wide store covers 32 consecutive floats of a row of y).  Before that, warp 2
//               is the TMA producer of the packed weights: 128 rows x 128 bytes at a time (2 or
//               4 chunks of k), so that every row is read from memory in whole 128-byte lines,
//               running as far ahead of the MMAs as its own ring allows (the weight stream is
//               what bounds the layer at small batch)
//   warps 6-21  weight expanders: packed tile in shared memory -> bfloat16 A tile (the integer ->
//               bfloat16 expansion is a dependent chain per thread; sixteen warps hide it)
// A CTA owns one (128-channel block, K split, 256-row batch block) and runs once.
#pragma once

namespace aiq {
namespace {

constexpr int kQtExpWarps = 16;                      // weight expander warps
constexpr int kQtThreads = (6 + kQtExpWarps) * 32;
constexpr int kQtChunk = 64;                         // k per stage
constexpr int kQtATile = 128 * kQtChunk * 2;         // 16 KB: 128 channels x 64 bfloat16
constexpr int kQtWTile = 128 * 128;                  // 16 KB: 128 channels x 128 packed bytes
constexpr int kQtMaxWStages = 8;

struct QtParams {
  int N, K, M, bits;
  int Mt;                   // batch rows per CTA tile (multiple of 16, <= 256)
  int m_block;              // batch rows per blockIdx.z: 256, or 128 with two weight pieces (shared memory)
  int n_chunks;             // ceil(K / 64)
  int chunks_per_split;
  int splits;
  int n_stages;             // A tiles (expanded weights) in flight
  int b_stages;             // activation tile pairs in flight (a ring of its own: these are the
                            // TMA loads with a long round trip, and at small batch they are small)
  int w_stages;             // packed weight tiles in flight
  int pieces;               // bfloat16 pieces per weight: 1 (4- / 8-bit codes), 2 (16- / 32-bit weights as hi + lo)
  int stack;                // 1: hi and lo rows of B form one N = 2 Mt operand (Mt <= 128)
  int tmem_cols;
  int32_t* error_flag;      // optional
};

constexpr int kQtMaxBStages = 24;
__host__ __device__ inline int qt_b_stage_bytes(int Mt) { return 2 * Mt * kQtChunk * 2; }   // hi tile + lo tile
__host__ __device__ inline int qt_smem_bytes(int Mt, int stages, int b_stages, int w_stages, int pieces = 1) {
  return stages * pieces * kQtATile + b_stages * qt_b_stage_bytes(Mt) + w_stages * kQtWTile +
         (2 * stages + 2 * b_stages + 2 * w_stages + 1) * 8 + 16;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

// x [M][K] float32 -> planes hi [M][K], lo [M][K] bfloat16 (x = hi + lo up to 2^-17 relative);
// optionally y = 0 (the split-K partial sums are added atomically)
__global__ void __launch_bounds__(256)
qlinear_split_x_kernel(const float* __restrict__ x, long long n_elems, __nv_bfloat16* __restrict__ planes,
                       float* __restrict__ y, long long y_elems) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long step = (long long)gridDim.x * blockDim.x;
  for (long long i = tid; i < y_elems; i += step) y[i] = 0.f;
  // n_elems is a multiple of 8 (K % 8 == 0)
  for (long long i = tid * 4; i < n_elems; i += step * 4) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(x + i));
    uint32_t h0, l0, h1, l1;
    split_pair(v.x, v.y, h0, l0);
    split_pair(v.z, v.w, h1, l1);
    *reinterpret_cast<uint2*>(planes + i) = make_uint2(h0, h1);
    *reinterpret_cast<uint2*>(planes + n_elems + i) = make_uint2(l0, l1);
  }
}

__global__ void __launch_bounds__(kQtThreads, 1)
qlinear_tc_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map, QtParams p,
                  const float* __restrict__ scale, const float* __restrict__ bias, float* __restrict__ y) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n0 = blockIdx.x * 128, split = blockIdx.y, m0 = blockIdx.z * p.m_block;
  const int stages = p.n_stages, b_stages = p.b_stages, Mt = p.Mt, w_stages = p.w_stages;
  const int b_stage_bytes = qt_b_stage_bytes(Mt);
  const int c_begin = split * p.chunks_per_split;
  const int c_end = min(p.n_chunks, c_begin + p.chunks_per_split);

  // k chunks per packed tile: 128 bytes of a row are 256 (4 bits), 128 (8 bits) or 64 (16 bits) elements;
  // at 32 bits a chunk of 64 k spans tpc = 2 packed tiles
  const int cpw = p.bits == 4 ? 4 : (p.bits == 8 ? 2 : 1);
  const int tpc = p.bits == 32 ? 2 : 1;
  const int a_stage_bytes = p.pieces * kQtATile;            // hi tile (+ lo tile of 16- / 32-bit weights)
  // shared memory: A ring | B ring | packed weight ring | barriers (every tile 1024-aligned)
  uint8_t* bring = smem + stages * a_stage_bytes;
  uint8_t* wring = bring + b_stages * b_stage_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(wring + w_stages * kQtWTile);
  const uint32_t bar_a_full = smem_u32(bars);               // expanders finished an A tile
  const uint32_t bar_a_empty = bar_a_full + 8 * stages;     // the MMAs that read an A tile have retired
  const uint32_t bar_b_full = bar_a_empty + 8 * stages;     // TMA bytes of an activation tile pair have landed
  const uint32_t bar_b_empty = bar_b_full + 8 * b_stages;   // the MMAs that read it have retired
  const uint32_t bar_w_full = bar_b_empty + 8 * b_stages;   // a packed weight tile has landed
  const uint32_t bar_w_empty = bar_w_full + 8 * w_stages;   // the expanders are done with a packed tile
  const uint32_t bar_acc_full = bar_w_empty + 8 * w_stages;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * stages + 2 * b_stages + 2 * w_stages + 1);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) {
      mbar_init(bar_a_full + 8 * i, kQtExpWarps);   // one arrival per expander warp
      mbar_init(bar_a_empty + 8 * i, 1);
    }
    for (int i = 0; i < b_stages; ++i) {
      mbar_init(bar_b_full + 8 * i, 1);
      mbar_init(bar_b_empty + 8 * i, 1);
    }
    for (int i = 0; i < w_stages; ++i) {
      mbar_init(bar_w_full + 8 * i, 1);
      mbar_init(bar_w_empty + 8 * i, kQtExpWarps);  // one arrival per expander warp
    }
    mbar_init(bar_acc_full, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 1) {
    tmem_alloc(smem_u32(s_tmem), (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  bool alive = true;

  if (warp == 0) {
    // ---- TMA producer of the activation tiles (the planes are written by the pre-pass) -----------
    if (lane == 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      uint32_t stage = 0, phase = 0, issued = 0, issued_phase = 0;
      for (int c = c_begin; c < c_end && alive; ++c) {
        alive = mbar_wait(bar_b_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
        if (!alive) break;
        issued |= 1u << stage;
        issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
        const uint32_t tile_bytes = (uint32_t)Mt * kQtChunk * 2;
        mbar_expect_tx(bar_b_full + 8 * stage, 2 * tile_bytes);
        const uint32_t dst = smem_u32(bring) + stage * b_stage_bytes;
        tma_load_3d(dst, &x_map, bar_b_full + 8 * stage, c * kQtChunk, m0, 0);                // hi
        tma_load_3d(dst + tile_bytes, &x_map, bar_b_full + 8 * stage, c * kQtChunk, m0, 1);   // lo
        if (++stage == (uint32_t)b_stages) { stage = 0; phase ^= 1u; }
      }
      for (int i = 0; i < b_stages; ++i)           // copies in flight must land before the CTA exits
        if (issued & (1u << i)) {
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_b_full + 8 * i, (issued_phase >> i) & 1u) && clock64() - t0 < kWaitLimitCycles) {}
        }
    }
  } else if (warp >= 6) {
    // ---- weight expanders: packed tile -> bfloat16 A tile (128 rows x 64 k, 128-byte swizzle) ------
    // The packed tile holds 128 bytes of each of the 128 rows, 16-byte units XOR-swizzled by
    // the row (the tensor map's 128-byte swizzle), so the 4- or 8-byte reads of a warp spread
    // over all banks.  A thread expands 2 units of 8 codes per chunk.
    constexpr int ET = kQtExpWarps * 32;                        // expander threads
    const int et = tid - 6 * 32;                                // 0 .. ET-1
    constexpr int UPR = kQtChunk / 8;                           // 8 units of 8 k per row and chunk
    constexpr int UPT = 128 * UPR / ET;                         // units per thread
    const int unit_bytes = p.bits;                              // 8 codes: 4 or 8 bytes
    uint32_t stage = 0, phase = 0, wst = 0, wphase = 0;
    if (p.pieces == 2) {
      // 16- / 32-bit weights: w = hi + lo with hi = bf16(w), lo = bf16(w - hi) (exact for a half, within 2^-17
      // of a float32 weight); one A tile per piece, the MMAs of a chunk are issued once per piece.
      for (int c = c_begin; c < c_end && alive; ++c) {
        uint32_t tile_stage[2] = {wst, 0};
        for (int t = 0; t < tpc && alive; ++t) {
          tile_stage[t] = wst;
          alive = mbar_wait_warp(bar_w_full + 8 * wst, wphase, s_abort, p.error_flag);
          if (++wst == (uint32_t)w_stages) { wst = 0; wphase ^= 1u; }
        }
        if (!alive) break;
        float w[UPT][8];
#pragma unroll
        for (int i = 0; i < UPT; ++i) {
          const int u = et + i * ET;
          const int nl = u / UPR, cu = u - nl * UPR;
          if (p.bits == 16) {
            const uint4 r = *reinterpret_cast<const uint4*>(wring + tile_stage[0] * kQtWTile + swizzle_off((uint32_t)(nl * 128 + cu * 16), 7u));
            const __half2* h2 = reinterpret_cast<const __half2*>(&r);
#pragma unroll
            for (int j = 0; j < 4; ++j) { const float2 f = __half22float2(h2[j]); w[i][2 * j] = f.x; w[i][2 * j + 1] = f.y; }
          } else {
            const uint8_t* wt = wring + tile_stage[cu >> 2] * kQtWTile;
            const float4 r0 = *reinterpret_cast<const float4*>(wt + swizzle_off((uint32_t)(nl * 128 + (cu & 3) * 32), 7u));
            const float4 r1 = *reinterpret_cast<const float4*>(wt + swizzle_off((uint32_t)(nl * 128 + (cu & 3) * 32 + 16), 7u));
            w[i][0] = r0.x; w[i][1] = r0.y; w[i][2] = r0.z; w[i][3] = r0.w; w[i][4] = r1.x; w[i][5] = r1.y; w[i][6] = r1.z; w[i][7] = r1.w;
          }
        }
        alive = mbar_wait_warp(bar_a_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
        if (!alive) break;
        uint8_t* atile = smem + stage * a_stage_bytes;
#pragma unroll
        for (int i = 0; i < UPT; ++i) {
          const int u = et + i * ET;
          const int nl = u / UPR, cu = u - nl * UPR;
          uint32_t hi4[4], lo4[4];
#pragma unroll
          for (int j = 0; j < 8; j += 2) split_pair(w[i][j], w[i][j + 1], hi4[j >> 1], lo4[j >> 1]);
          const uint32_t off = swizzle_off((uint32_t)(nl * 128 + cu * 16), 7u);
          *reinterpret_cast<uint4*>(atile + off) = make_uint4(hi4[0], hi4[1], hi4[2], hi4[3]);
          *reinterpret_cast<uint4*>(atile + kQtATile + off) = make_uint4(lo4[0], lo4[1], lo4[2], lo4[3]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        // The packed tiles are released only now, after their words have been used: every lane's loads
        // have then returned.  (Released right after the loads were issued, a refill by the TMA reached
        // shared memory before the last loads of a warp had read it: wrong weights in 2-4 adjacent rows,
        // a few times per million outputs.)
        if (lane == 0) {
          for (int t = 0; t < tpc; ++t) mbar_arrive(bar_w_empty + 8 * tile_stage[t]);
          mbar_arrive(bar_a_full + 8 * stage);
        }
        if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
      }
    } else
    for (int c = c_begin; c < c_end && alive; ++c) {
      const int sub = (c - c_begin) % cpw;                      // chunk inside the packed tile
      if (sub == 0) {
        alive = mbar_wait_warp(bar_w_full + 8 * wst, wphase, s_abort, p.error_flag);
        if (!alive) break;
      }
      const uint8_t* wt = wring + wst * kQtWTile;
      uint2 raw[UPT];
#pragma unroll
      for (int i = 0; i < UPT; ++i) {
        const int u = et + i * ET;
        const int nl = u / UPR, cu = u - nl * UPR;
        const uint32_t off = swizzle_off((uint32_t)(nl * 128 + (sub * UPR + cu) * unit_bytes), 7u);
        if (p.bits == 8) raw[i] = *reinterpret_cast<const uint2*>(wt + off);
        else raw[i] = make_uint2(*reinterpret_cast<const uint32_t*>(wt + off), 0u);
      }
      // the packed tile is released further down, once its words have been used (see the two-piece path)
      const bool last_of_tile = sub == cpw - 1 || c + 1 == c_end;
      const uint32_t release_stage = wst;
      if (last_of_tile && ++wst == (uint32_t)w_stages) { wst = 0; wphase ^= 1u; }
      alive = mbar_wait_warp(bar_a_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
      if (!alive) break;
      uint8_t* atile = smem + stage * a_stage_bytes;
#pragma unroll
      for (int i = 0; i < UPT; ++i) {
        const int u = et + i * ET;
        const int nl = u / UPR, cu = u - nl * UPR;
        uint32_t out[4];
        expand8_bf16(raw[i], p.bits, out);
        *reinterpret_cast<uint4*>(atile + swizzle_off((uint32_t)(nl * 128 + cu * 16), 7u)) =
            make_uint4(out[0], out[1], out[2], out[3]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA
      __syncwarp();
      if (lane == 0) {
        if (last_of_tile) mbar_arrive(bar_w_empty + 8 * release_stage);
        mbar_arrive(bar_a_full + 8 * stage);
      }
      if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
    }
  } else if (warp == 1) {
    // ---- MMA issuer: all 32 lanes converged, one elected lane issues (see umma_bf16) ------------
    // Up to Mt = 128 the hi and the lo tile (adjacent in shared memory) are one B operand of
    // 2 Mt rows: half as many MMAs, the two partial products land in separate accumulator
    // columns and are added in the epilogue.  Small MMAs cost more to issue than to execute.
    const int mma_n = p.stack ? 2 * Mt : Mt;
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(mma_n >> 3) << 17) | ((128u >> 4) << 24);
    constexpr uint32_t DESC_HI = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);   // SBO 1024, version 1, 128-byte swizzle
    constexpr uint32_t LBO_FIELD = 1u << 16;
    const uint32_t tile_units = (uint32_t)(Mt * kQtChunk * 2) >> 4;
    uint32_t stage = 0, phase = 0, bstage = 0, bphase = 0, accumulate = 0;
    for (int c = c_begin; c < c_end && alive; ++c) {
      alive = mbar_wait_warp(bar_a_full + 8 * stage, phase, s_abort, p.error_flag) &&
              mbar_wait_warp(bar_b_full + 8 * bstage, bphase, s_abort, p.error_flag);
      if (!alive) break;
      tc_fence_after();
      const uint32_t a_lo = ((smem_u32(smem) + stage * a_stage_bytes) >> 4) | LBO_FIELD;
      const uint32_t b_lo = ((smem_u32(bring) + bstage * b_stage_bytes) >> 4) | LBO_FIELD;
      const int parts = p.stack ? 1 : 2;
      for (int piece = 0; piece < p.pieces; ++piece) {
        for (int part = 0; part < parts; ++part) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const uint64_t adesc = ((uint64_t)DESC_HI << 32) | (uint64_t)(a_lo + ((piece * kQtATile + kk * 32) >> 4));
            const uint64_t bdesc = ((uint64_t)DESC_HI << 32) | (uint64_t)(b_lo + part * tile_units + ((kk * 32) >> 4));
            umma_bf16(tmem_base, adesc, bdesc, idesc, accumulate);
            accumulate = 1;
          }
        }
      }
      umma_commit(bar_a_empty + 8 * stage);
      umma_commit(bar_b_empty + 8 * bstage);
      if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
      if (++bstage == (uint32_t)b_stages) { bstage = 0; bphase ^= 1u; }
    }
    if (alive) umma_commit(bar_acc_full);
  } else {
    // ---- epilogue: warp q owns TMEM lanes 32q .. 32q+31 = output channels n0 + 32q + lane ---------
    const int q = warp & 3;
    const int n = n0 + q * 32 + lane;
    if (warp == 2) {
      // packed weight tiles: independent of the pre-pass, requested as early as the ring allows
      if (lane == 0) {
        uint32_t wst = 0, wphase = 0, w_issued = 0, w_issued_phase = 0;
        bool ok = true;
        for (int c = c_begin; c < c_end && ok; c += cpw) {   // bytes [c * 64 * bits / 8, + 128 tpc) of 128 rows
          for (int t = 0; t < tpc && ok; ++t) {
            ok = mbar_wait(bar_w_empty + 8 * wst, wphase ^ 1u, s_abort, p.error_flag);
            if (!ok) break;
            w_issued |= 1u << wst;
            w_issued_phase = (w_issued_phase & ~(1u << wst)) | (wphase << wst);
            mbar_expect_tx(bar_w_full + 8 * wst, kQtWTile);
            tma_load_2d(smem_u32(wring) + wst * kQtWTile, &w_map, bar_w_full + 8 * wst, c * kQtChunk * p.bits / 8 + t * 128, n0);
            if (++wst == (uint32_t)w_stages) { wst = 0; wphase ^= 1u; }
          }
        }
        if (!ok)                                   // copies in flight must land before the CTA exits
          for (int i = 0; i < w_stages; ++i)
            if (w_issued & (1u << i)) {
              const long long t0 = clock64();
              while (!mbar_try_wait(bar_w_full + 8 * i, (w_issued_phase >> i) & 1u) && clock64() - t0 < kWaitLimitCycles) {}
            }
      }
      __syncwarp();
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");       // y is zeroed by the pre-pass
    const bool n_ok = n < p.N;
    const float s = n_ok ? scale[n] : 0.f;
    const float b = (n_ok && bias && split == 0) ? bias[n] : 0.f;
    alive = mbar_wait_warp(bar_acc_full, 0, s_abort, p.error_flag);
    if (alive && c_begin < c_end) {
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      for (int c0 = 0; c0 < Mt; c0 += 16) {
        if (m0 + c0 >= p.M) break;
        uint32_t v[16], v2[16];
        tmem_ld16(taddr + c0, v);
        if (p.stack) tmem_ld16(taddr + Mt + c0, v2);       // the lo half's partial products
        tmem_ld_wait();
        if (n_ok) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            if (m < p.M) {
              const float acc = p.stack ? __uint_as_float(v[j]) + __uint_as_float(v2[j]) : __uint_as_float(v[j]);
              const float val = fmaf(acc, s, b);
              float* dst = y + (size_t)m * p.N + n;
              if (p.splits > 1) atomicAdd(dst, val); else *dst = val;
            }
          }
        }
      }
    }
  }

  // ---- teardown -------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

}  // namespace

bool qlinear_tc_applicable(int N, int K, int bits, int M) {
  if (!bits_ok(bits)) return false;
  if (M < 9) return false;                         // smaller batches: the warp-level kernels
  if (K % 8 != 0 || K < 64 || N < 32) return false;
  return true;
}

size_t qlinear_tc_workspace_bytes(int K, int M) { return (size_t)2 * M * K * sizeof(__nv_bfloat16); }

aiq_status_t launch_qlinear_tc(const LayerJob& job, int N, int K, int M, void* workspace, int32_t* error_flag,
                               cudaStream_t s) {
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  const int smem_limit = props.smem_optin, n_sms = props.n_sms;
  AIQ_ENSURE_DYNAMIC_SMEM(qlinear_tc_kernel, smem_limit);
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  QtParams p = {};
  p.N = N; p.K = K; p.M = M; p.bits = job.bits; p.error_flag = error_flag;
  p.pieces = job.bits > 8 ? 2 : 1;
  p.m_block = p.pieces == 2 ? 128 : 256;           // two A tiles per stage leave room for activation tiles of 128 rows
  p.Mt = M >= p.m_block ? p.m_block : (M + 15) / 16 * 16;
  const int m_blocks = (M + p.m_block - 1) / p.m_block, row_blocks = (N + 127) / 128;
  p.n_chunks = (K + kQtChunk - 1) / kQtChunk;
  int splits = n_sms / (row_blocks * m_blocks);
  if (splits < 1) splits = 1;
  if (splits > p.n_chunks) splits = p.n_chunks;
  p.chunks_per_split = (p.n_chunks + splits - 1) / splits;
  p.splits = (p.n_chunks + p.chunks_per_split - 1) / p.chunks_per_split;
  // Shared memory: at least 2 A tiles, 2 activation tile pairs and 3 packed weight tiles.  Then
  // up to 4 A tiles (they are produced on chip, a short ring suffices), as many activation
  // stages as fit up to 24 (their TMA round trip is what a shallow ring would expose), and
  // whatever is left goes to packed weight tiles in flight.
  auto fits = [&](int a, int b, int w) { return qt_smem_bytes(p.Mt, a, b, w, p.pieces) + 1024 <= smem_limit; };
  if (!fits(2, 2, 3))
    return set_error(AIQ_ERR_SHAPE, "qlinear_tc: %d bytes of shared memory needed", qt_smem_bytes(p.Mt, 2, 2, 3, p.pieces) + 1024);
  int stages = 2, b_stages = 2, w_stages = 3;
  while (stages < 4 && fits(stages + 1, b_stages, w_stages)) ++stages;
  while (w_stages < 4 && fits(stages, b_stages, w_stages + 1)) ++w_stages;
  while (b_stages < kQtMaxBStages && b_stages < p.chunks_per_split && fits(stages, b_stages + 1, w_stages)) ++b_stages;
  while (w_stages < kQtMaxWStages && fits(stages, b_stages, w_stages + 1)) ++w_stages;
  p.n_stages = stages;
  p.b_stages = b_stages;
  p.w_stages = w_stages;
  p.stack = p.Mt <= 128 ? 1 : 0;
  p.tmem_cols = 32;
  while (p.tmem_cols < (p.stack ? 2 * p.Mt : p.Mt)) p.tmem_cols <<= 1;

  // activation planes in the workspace: (k, batch row, hi | lo)
  __nv_bfloat16* planes = static_cast<__nv_bfloat16*>(workspace);
  CUtensorMap x_map;
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)M, 2};
  cuuint64_t strides[2] = {2ull * K, 2ull * K * M};
  cuuint32_t box[3] = {(cuuint32_t)kQtChunk, (cuuint32_t)p.Mt, 1u};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(&x_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, planes, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled (linear layer) failed with code %d", (int)r);

  // packed weights: (byte of a row, row); rows past N and bytes past the row arrive as zeros
  CUtensorMap w_map;
  {
    const cuuint64_t wrow = (cuuint64_t)row_bytes(K, job.bits);
    cuuint64_t wdims[2] = {wrow, (cuuint64_t)N};
    cuuint64_t wstrides[1] = {wrow};
    cuuint32_t wbox[2] = {128u, 128u};
    cuuint32_t westr[2] = {1, 1};
    r = enc(&w_map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(job.w), wdims, wstrides, wbox, westr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return set_error(AIQ_ERR_CUDA, "cuTensorMapEncodeTiled (packed weights) failed with code %d", (int)r);
  }

  const float* x = static_cast<const float*>(job.in);
  float* y = static_cast<float*>(job.out);
  LaunchScope scope(AIQ_KERNEL_QLINEAR, s, 2.0 * M * N * K,
                    (double)N * row_bytes(K, job.bits) + 4.0 * N + 4.0 * M * ((double)K + N));
  const long long n_elems = (long long)M * K;
  int pre_blocks = (int)((n_elems / 4 + 255) / 256);
  if (pre_blocks > 4 * n_sms) pre_blocks = 4 * n_sms;
  if (pre_blocks < 1) pre_blocks = 1;
  qlinear_split_x_kernel<<<pre_blocks, 256, 0, s>>>(x, n_elems, planes, y, p.splits > 1 ? (long long)M * N : 0ll);
  AIQ_LAUNCH_CHECK("qlinear_split_x");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(row_blocks, p.splits, m_blocks);
  cfg.blockDim = dim3(kQtThreads);
  cfg.dynamicSmemBytes = qt_smem_bytes(p.Mt, stages, b_stages, w_stages, p.pieces) + 1024;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  AIQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, qlinear_tc_kernel, x_map, w_map, p, job.scale, job.bias, y));
  AIQ_LAUNCH_CHECK("qlinear_tc");
  return AIQ_OK;
}

}  // namespace aiq
