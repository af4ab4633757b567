// Pointwise (1x1, stride 1) convolution with many channels on the tcgen05 tensor cores.
// Included by conv_tc.cu (shares its PTX wrappers); not a stand-alone translation unit.
//
// A 1x1 convolution over split activations is a plain GEMM over all (padded) pixels:
//   D[128 pixels][Nt channels] += A[128][64 k] * B[Nt][64 k]^T   per chunk of 64 input channels,
// once for the hi half and once for the lo half of the pixels (same B).  MobileNetV2's
// expand / project / head layers have 16 .. 960 input and 16 .. 1280 output channels, so
// neither operand fits in shared memory: both stream through a ring, one stage per chunk.
//   warp 0      TMA producer: A tiles (hi and lo, 128 pixels x 64 channels each, 128-byte swizzle;
//               channels past C arrive as zeros)
//   warp 1      MMA issuer
//   warps 2-5   epilogue (TMEM -> scale, bias, residual, activation -> split bfloat16 -> global)
//   warps 6-9   weight expanders: packed 4 / 8-bit rows from global memory (L2) -> bfloat16 ->
//               swizzled B tile in shared memory, made visible to the MMA with a proxy fence
// A CTA owns one (job, tile of Nt output channels) and walks over pixel tiles.
#pragma once

namespace aiq {
namespace {

constexpr int kPwThreads = 448;                      // producer, MMA, 4 epilogue, 4 expander, 4 more epilogue warps
constexpr int kPwChunk = 64;                         // input channels per stage
constexpr int kPwATile = 128 * kPwChunk * 2;         // 16 KB: 128 pixels x 64 bfloat16

struct PwParams {
  int P;                    // padded pixels of the batch: B * (H + 2) * W
  int H, W;                 // spatial size (rows 0 and H + 1 of every image are border rows)
  int Cin, Cs_in, Cout, Cs_out;
  int Nt;                   // output channels per CTA (multiple of 16, <= 128)
  int n_ntiles;
  int act, n_stages;
  int pieces;               // bfloat16 pieces per weight: 1 (4- / 8-bit codes), 2 (16- / 32-bit weights as hi + lo)
  long long ver_pixels;     // pixels per version of the input slot (capacity * (H + 2) * W)
  int32_t* error_flag;
};

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// shared memory: [stage: A_hi | A_lo | B (one tile per weight piece)] x n_stages, scale, bias, barriers, tmem ptr, abort flag
__host__ __device__ inline int pw_stage_bytes(int Nt, int pieces) { return 2 * kPwATile + pieces * Nt * kPwChunk * 2; }
// output staging: per 64-channel group of the N tile one hi and one lo box of 128 pixels x 128 bytes
__host__ __device__ inline int pw_out_groups(int Nt) { return (Nt + 63) / 64; }
__host__ __device__ inline int pw_staging_bytes(int Nt) { return pw_out_groups(Nt) * 2 * kPwATile; }
__host__ __device__ inline int pw_smem_bytes(int Nt, int stages, int pieces) {
  return stages * pw_stage_bytes(Nt, pieces) + pw_staging_bytes(Nt) + 2 * 128 * 4 + (3 * stages + 4) * 8 + 16;
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}

__global__ void __launch_bounds__(kPwThreads, 1)
conv_pw_tc_kernel(const __grid_constant__ CUtensorMap in_map, const __grid_constant__ CUtensorMap out_map, PwParams p,
                  const LayerJob* __restrict__ jobs) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int job_idx = blockIdx.y / p.n_ntiles, ntile = blockIdx.y - job_idx * p.n_ntiles;
  const LayerJob job = jobs[job_idx];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int stages = p.n_stages, Nt = p.Nt, n0 = ntile * Nt;
  const int stage_bytes = pw_stage_bytes(Nt, p.pieces);

  uint8_t* staging = smem + stages * stage_bytes;            // 1024-aligned: every stage is a multiple of 2 KB
  float* s_scale = reinterpret_cast<float*>(staging + pw_staging_bytes(Nt));
  float* s_bias = s_scale + 128;
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_bias + 128);
  const uint32_t bar_a_full = smem_u32(bars);               // TMA bytes of a stage have landed
  const uint32_t bar_b_full = bar_a_full + 8 * stages;      // expanders finished the B tile of a stage
  const uint32_t bar_empty = bar_b_full + 8 * stages;       // the MMAs that read a stage have retired
  const uint32_t bar_acc_full = bar_empty + 8 * stages;
  const uint32_t bar_acc_empty = bar_acc_full + 16;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 3 * stages + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int n_tiles = (p.P + 127) / 128;
  const int n_chunks = (p.Cs_in + kPwChunk - 1) / kPwChunk;

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) {
      mbar_init(bar_a_full + 8 * i, 1);
      mbar_init(bar_b_full + 8 * i, 4);          // one arrival per expander warp
      mbar_init(bar_empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_acc_full + 8 * i, 1);
      mbar_init(bar_acc_empty + 8 * i, 8);       // one arrival per epilogue warp
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < 128; i += kPwThreads) {
    const int n = n0 + i;
    s_scale[i] = (i < Nt && n < p.Cout) ? job.scale[n] : 0.f;   // padded channels come out as zeros
    s_bias[i] = (i < Nt && n < p.Cout) ? job.bias[n] : 0.f;
  }
  __syncthreads();
  if (warp == 1) {
    tmem_alloc(smem_u32(s_tmem), 256);           // two accumulator buffers of up to 128 columns
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  bool alive = true;

  if (warp == 0) {
    // ---- TMA producer -----------------------------------------------------------------------
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued = 0, issued_phase = 0;
      for (int tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x) {
        for (int c = 0; c < n_chunks && alive; ++c) {
          alive = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
          if (!alive) break;
          issued |= 1u << stage;
          issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
          mbar_expect_tx(bar_a_full + 8 * stage, 2 * kPwATile);
          const uint32_t dst = smem_u32(smem) + stage * stage_bytes;
          const int pix = (int)(job.in_version * p.ver_pixels) + tile * 128;
          tma_load_3d(dst, &in_map, bar_a_full + 8 * stage, c * kPwChunk, 0, pix);             // hi
          tma_load_3d(dst + kPwATile, &in_map, bar_a_full + 8 * stage, c * kPwChunk, 1, pix);  // lo
          if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
        }
      }
      for (int i = 0; i < stages; ++i)             // copies in flight must land before the CTA exits
        if (issued & (1u << i)) {
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_a_full + 8 * i, (issued_phase >> i) & 1u) && clock64() - t0 < kWaitLimitCycles) {}
        }
    }
  } else if (warp >= 6 && warp < 10) {
    // ---- weight expanders: packed codes -> bfloat16 B tile (Nt rows x 64 channels, 128-byte swizzle)
    // The packed words of a chunk are the same for every pixel tile and come from L2; they are
    // fetched one chunk ahead into registers so that their latency hides behind the expansion of
    // the current chunk and the wait for a free stage.
    const int et = tid - 6 * 32;                                // 0 .. 127
    const int kpad = (p.Cin + 31) / 32 * 32;
    const size_t wrow = (size_t)kpad * job.bits / 8;
    constexpr int UPR = kPwChunk / 8;                           // 8 units of 8 channels per row and chunk
    constexpr int UPT = 128 * UPR / 128;                        // units per thread at Nt = 128: 8
    const int n_units = Nt * UPR;
    auto fetch = [&](int c, uint2* raw) {
#pragma unroll
      for (int i = 0; i < UPT; ++i) {
        const int u = et + i * 128;
        const int nl = u / UPR, cu = u - nl * UPR;
        const int n = n0 + nl, ch = c * kPwChunk + cu * 8;
        raw[i] = make_uint2(0u, 0u);
        if (u < n_units && n < p.Cout && ch < p.Cin) {          // Cin is a multiple of 8 here
          const uint8_t* src = job.w + (size_t)n * wrow;
          if (job.bits == 8) raw[i] = __ldg(reinterpret_cast<const uint2*>(src + ch));
          else raw[i].x = __ldg(reinterpret_cast<const uint32_t*>(src + ch / 2));
        }
      }
    };
    uint2 cur[UPT], nxt[UPT];
    uint32_t stage = 0, phase = 0;
    if (p.pieces == 2) {
      // 16- / 32-bit weights: w = hi + lo, hi = bf16(w), lo = bf16(w - hi) (exact for a half, within 2^-17 of
      // a float32 weight): two B tiles per stage, the MMAs are issued once per piece.  The words come from
      // L2 when they are needed (no register prefetch: a unit is 16 or 32 bytes here).
      for (int tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x) {
        for (int c = 0; c < n_chunks && alive; ++c) {
          alive = mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
          if (!alive) break;
          uint8_t* btile = smem + stage * stage_bytes + 2 * kPwATile;
          for (int u = et; u < n_units; u += 128) {
            const int nl = u / UPR, cu = u - nl * UPR;
            const int n = n0 + nl, ch = c * kPwChunk + cu * 8;
            float w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = 0.f;
            if (n < p.Cout && ch < p.Cin) {
              const uint8_t* src = job.w + (size_t)n * wrow;
              if (job.bits == 16) {
                const uint4 r = __ldg(reinterpret_cast<const uint4*>(src + (size_t)ch * 2));
                const __half2* h2 = reinterpret_cast<const __half2*>(&r);
#pragma unroll
                for (int j = 0; j < 4; ++j) { const float2 f = __half22float2(h2[j]); w[2 * j] = f.x; w[2 * j + 1] = f.y; }
              } else {
                const float4 r0 = __ldg(reinterpret_cast<const float4*>(src + (size_t)ch * 4));
                const float4 r1 = __ldg(reinterpret_cast<const float4*>(src + (size_t)ch * 4) + 1);
                w[0] = r0.x; w[1] = r0.y; w[2] = r0.z; w[3] = r0.w; w[4] = r1.x; w[5] = r1.y; w[6] = r1.z; w[7] = r1.w;
              }
            }
            uint32_t hi4[4], lo4[4];
#pragma unroll
            for (int j = 0; j < 8; j += 2) split_pair(w[j], w[j + 1], hi4[j >> 1], lo4[j >> 1]);
            const uint32_t off = swizzle_off((uint32_t)(nl * 128 + cu * 16), 7u);
            *reinterpret_cast<uint4*>(btile + off) = make_uint4(hi4[0], hi4[1], hi4[2], hi4[3]);
            *reinterpret_cast<uint4*>(btile + Nt * 128 + off) = make_uint4(lo4[0], lo4[1], lo4[2], lo4[3]);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_b_full + 8 * stage);
          if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
        }
      }
    } else {
    fetch(0, cur);
    for (int tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x) {
      for (int c = 0; c < n_chunks && alive; ++c) {
        fetch(c + 1 < n_chunks ? c + 1 : 0, nxt);               // next chunk (of this or the next tile)
        alive = mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1u, s_abort, p.error_flag);
        if (!alive) break;
        uint8_t* btile = smem + stage * stage_bytes + 2 * kPwATile;
#pragma unroll
        for (int i = 0; i < UPT; ++i) {
          const int u = et + i * 128;
          if (u >= n_units) break;
          const int nl = u / UPR, cu = u - nl * UPR;
          uint32_t out[4];
          expand8_bf16(cur[i], job.bits, out);   // a unit that was not fetched holds zero words = zero codes
          *reinterpret_cast<uint4*>(btile + swizzle_off((uint32_t)(nl * 128 + cu * 16), 7u)) =
              make_uint4(out[0], out[1], out[2], out[3]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_b_full + 8 * stage);
        if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
#pragma unroll
        for (int i = 0; i < UPT; ++i) cur[i] = nxt[i];
      }
    }
    }
  }
  else if (warp == 1) {
    // ---- MMA issuer: all 32 lanes converged, one elected lane issues (see umma_bf16) ----------
    {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(Nt >> 3) << 17) | ((128u >> 4) << 24);
      constexpr uint32_t DESC_HI = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);   // SBO 1024, version 1, 128-byte swizzle
      constexpr uint32_t LBO_FIELD = 1u << 16;
      uint32_t stage = 0, phase = 0;
      int it = 0;
      for (int tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x, ++it) {
        const int buf = it & 1;
        alive = mbar_wait_warp(bar_acc_empty + 8 * buf, ((it >> 1) & 1) ^ 1u, s_abort, p.error_flag);
        if (!alive) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 128);
        uint32_t accumulate = 0;
        for (int c = 0; c < n_chunks && alive; ++c) {
          alive = mbar_wait_warp(bar_a_full + 8 * stage, phase, s_abort, p.error_flag) &&
                  mbar_wait_warp(bar_b_full + 8 * stage, phase, s_abort, p.error_flag);
          if (!alive) break;
          tc_fence_after();
          const uint32_t a_lo = ((smem_u32(smem) + stage * stage_bytes) >> 4) | LBO_FIELD;
          const uint32_t b_lo = a_lo + ((2 * kPwATile) >> 4);
          const int kmax = min(4, (p.Cs_in - c * kPwChunk) / 16);      // 16-channel steps that hold data
#pragma unroll
          for (int part = 0; part < 2; ++part) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              if (kk < kmax) {
                const uint64_t adesc = ((uint64_t)DESC_HI << 32) | (uint64_t)(a_lo + ((part * kPwATile + kk * 32) >> 4));
                const uint64_t bdesc = ((uint64_t)DESC_HI << 32) | (uint64_t)(b_lo + ((kk * 32) >> 4));
                umma_bf16(d_tmem, adesc, bdesc, idesc, accumulate);
                accumulate = 1;
                if (p.pieces == 2)                  // the lo piece of 16- / 32-bit weights
                  umma_bf16(d_tmem, adesc, ((uint64_t)DESC_HI << 32) | (uint64_t)(b_lo + ((Nt * 128 + kk * 32) >> 4)), idesc, 1u);
              }
            }
          }
          umma_commit(bar_empty + 8 * stage);
          if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
        }
        if (alive) umma_commit(bar_acc_full + 8 * buf);
      }
    }
  } else {
    // ---- epilogue: warps 2 .. 5 and 10 .. 13.  TMEM lanes 32q .. 32q+31 = pixels 32q .. 32q+31 of
    // the tile belong to the two warps with warp index mod 4 = q; they take alternate groups of
    // 16 output channels (for layers that widen the channels the epilogue is most of the work).
    const int q = warp & 3;
    const int h = warp >= 10 ? 1 : 0;
    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x, ++it) {
      const int buf = it & 1;
      alive = mbar_wait_warp(bar_acc_full + 8 * buf, (it >> 1) & 1, s_abort, p.error_flag);   // false => *s_abort is set
      // the previous tile's stores must have finished reading the staging tiles
      if (warp == 2 && lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      asm volatile("bar.sync 1, 256;" ::: "memory");     // every epilogue thread, unconditionally
      alive = *s_abort == 0;                             // the same answer in all eight warps
      if (!alive) break;
      tc_fence_after();
      const int m = q * 32 + lane;                       // pixel row of the tile
      const int pix = tile * 128 + m;
      const int yp = (pix / p.W) % (p.H + 2);
      const bool interior = pix < p.P && yp >= 1 && yp <= p.H;
      const __nv_bfloat16* res = (job.res && interior)
          ? static_cast<const __nv_bfloat16*>(job.res) + (size_t)pix * (2 * p.Cs_out) : nullptr;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 128);
      for (int c0 = 16 * h; c0 < Nt; c0 += 32) {
        uint32_t v[16];
        tmem_ld16(taddr + c0, v);
        tmem_ld_wait();
        const int n = n0 + c0;
        uint32_t rh[8] = {0, 0, 0, 0, 0, 0, 0, 0}, rl[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (res && n < p.Cs_out) {
          const uint4 a0 = __ldg(reinterpret_cast<const uint4*>(res + n)), a1 = __ldg(reinterpret_cast<const uint4*>(res + n) + 1);
          const uint4 l0v = __ldg(reinterpret_cast<const uint4*>(res + p.Cs_out + n)), l1v = __ldg(reinterpret_cast<const uint4*>(res + p.Cs_out + n) + 1);
          rh[0] = a0.x; rh[1] = a0.y; rh[2] = a0.z; rh[3] = a0.w; rh[4] = a1.x; rh[5] = a1.y; rh[6] = a1.z; rh[7] = a1.w;
          rl[0] = l0v.x; rl[1] = l0v.y; rl[2] = l0v.z; rl[3] = l0v.w; rl[4] = l1v.x; rl[5] = l1v.y; rl[6] = l1v.z; rl[7] = l1v.w;
        }
        uint32_t hi[8], lo[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          float u0 = 0.f, u1 = 0.f;
          if (interior) {
            u0 = fmaf(__uint_as_float(v[e]), s_scale[c0 + e], s_bias[c0 + e]);
            u1 = fmaf(__uint_as_float(v[e + 1]), s_scale[c0 + e + 1], s_bias[c0 + e + 1]);
            u0 += __uint_as_float(rh[e >> 1] << 16) + __uint_as_float(rl[e >> 1] << 16);
            u1 += __uint_as_float(rh[e >> 1] & 0xFFFF0000u) + __uint_as_float(rl[e >> 1] & 0xFFFF0000u);
            u0 = apply_act(u0, p.act);
            u1 = apply_act(u1, p.act);
          }
          split_pair(u0, u1, hi[e >> 1], lo[e >> 1]);
        }
        // staging tile (group, part): 128 rows x 128 bytes, 16-byte units XOR-swizzled by the row
        // exactly as the 128-byte-swizzle tensor map expects
        uint8_t* tile_hi = staging + (c0 >> 6) * 2 * kPwATile;
        uint8_t* tile_lo = tile_hi + kPwATile;
        const int u0i = (c0 & 63) >> 3;                  // first of the two units of these 16 channels
        const uint32_t row = (uint32_t)m * 128u;
        *reinterpret_cast<uint4*>(tile_hi + row + (((u0i) ^ (m & 7)) << 4)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(tile_hi + row + (((u0i + 1) ^ (m & 7)) << 4)) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        *reinterpret_cast<uint4*>(tile_lo + row + (((u0i) ^ (m & 7)) << 4)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        *reinterpret_cast<uint4*>(tile_lo + row + (((u0i + 1) ^ (m & 7)) << 4)) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
      }
      // the accumulator is drained: hand it back, then publish the staging tiles and store them
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (warp == 2 && lane == 0) {
        for (int gi = 0; gi < pw_out_groups(Nt); ++gi) {
          if (n0 + gi * 64 >= p.Cs_out) break;
          // channels past Cs_out and pixels past the slot's capacity are clipped by the tensor map
          tma_store_4d(&out_map, smem_u32(staging) + gi * 2 * kPwATile, n0 + gi * 64, 0, tile * 128, job.out_version);
          tma_store_4d(&out_map, smem_u32(staging) + gi * 2 * kPwATile + kPwATile, n0 + gi * 64, 1, tile * 128, job.out_version);
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    }
    // all stores must have left shared memory (and be complete) before the CTA retires
    if (warp == 2 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  // ---- teardown -------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 256);
  }
}

}  // namespace
}  // namespace aiq
