// A whole MobileNetV2 inverted-residual block in one kernel:
//
//   hidden = act_e( s_e * (W_e  x)      + b_e )      1x1, Cin -> Ch            (tcgen05)
//   mid    = act_d( s_d * (W_d * hidden) + b_d )     depthwise 3x3, stride 1|2 (CUDA cores)
//   out    = act_p( s_p * (W_p  mid)    + b_p + x )  1x1, Ch -> Cout, optional shortcut (tcgen05)
//
// The hidden tensor has six times the channels of the block's input and output; layer by layer it
// is written and read twice.  Here it only exists in shared memory, 32 or 64 channels at a time.
//
// A CTA owns a band of output rows of one image (at most 128 output pixels, full width) and
// the input rows under it (one more above and below).  The input pixels of a band are one
// contiguous run of the [image][row + border rows][column][hi | lo] tensor; they are copied once
// into shared memory in the canonical K-major layout without swizzle ([8-channel plane][pixel]
// [16 bytes], 128 bytes from one group of 8 pixels to the next), which is the A operand of the
// expansion for every tile of 128 pixels.  The weights of the two 1x1 layers are kept by the
// model as ready bfloat16 operand images, one per chunk of hidden channels (built once from
// the packed codes, exact: integer codes), the depthwise weights as float32 rows; a chunk's
// images arrive by bulk copies while the chunk before is being computed.
//
// Roles: 16 worker warps and one issuing warp, which meet only through mbarriers (the workers
// among themselves through a named barrier).  Per chunk of hidden channels the workers
//   A. read the expansion accumulators, apply scale, bias and activation and park the chunk as
//      float32 in shared memory ([4-channel plane][row][W + 2 columns][16 bytes]: a zero column on
//      both sides, written once; rows outside the image are the depthwise layer's zero padding and
//      are stored as zeros),
//   D. run the depthwise 3x3 from the parked chunk (a lane per output pixel, four channels per
//      lane, the nine weights of the plane in registers; nine unconditional 16-byte loads), apply
//      scale, bias, activation and write the result as hi / lo bfloat16 planes: the A operand of
//      the projection;
// the issuing warp
//   - starts the bulk copy of the next expansion image as soon as the chunk's expansion MMAs are done,
//   - issues the expansion MMAs of the NEXT chunk (hi and lo halves of the pixels, all tiles of the
//     band into separate accumulator columns) once every worker has read the accumulators: they run
//     behind D,
//   - issues the projection MMAs of the chunk once every worker has written its part of the operand;
//     they add to the block's output accumulator (128 pixels x Cout) in tensor memory and run behind
//     A of the next chunk; then it fetches the next projection image.
// After the last chunk the workers give the accumulator scale, bias and the shortcut and store it.
// One warp polls an mbarrier on behalf of the workers (seventeen polling warps were measured to slow
// the MMAs they wait for); whether to go on after a wait is decided by one thread before the named
// barrier and read by all after it, so all workers leave at the same barrier.  Every wait is bounded
// as in the other tcgen05 kernels.
#include "tc_ptx.cuh"

#include <algorithm>

namespace aiq {

namespace {

constexpr int kMbWorkers = 16;                      // warps that run the accumulator, depthwise and output passes
constexpr int kMbThreads = (kMbWorkers + 1) * 32;   // + one warp that issues the MMAs and the bulk copies
constexpr int kMbLeader = kMbWorkers * 32;          // its first thread

struct MbParams {
  int H, W, Ho, Wo, stride;
  int Cin, Cs_in, Ch, Cout, Cs_out;
  int Rb;                   // output rows of a band
  int bands;                // bands per image
  int T1;                   // tiles of 128 hidden pixels a band can need
  int NH;                   // hidden channels per chunk: 32 or 64
  int n_chunks;
  int tmem_cols;
  int hid_px;               // pixels of a hidden plane: rows of a band x (W + 2): a zero column on both sides
  int act_e, act_d, act_p;
  int32_t* error_flag;
};

// shared memory regions (base aligned to 128 bytes)
struct MbSmem {
  int a_in, a_lbo;          // input operand: 2 * Cs_in / 8 planes, a_lbo bytes apart
  int b1;                   // expansion operand image of the chunk (mb_etile_bytes)
  int hid, hid_plane;       // hidden chunk, float32: NH / 4 planes of hid_px pixels (rows of W + 2 columns)
  int a2;                   // depthwise output, hi then lo planes of 128 pixels
  int b2;                   // projection operand image of the chunk (mb_ptile_bytes)
  int coef;                 // two buffers (chunk parity) of floats: s_e, b_e [NH]; w_d [9][NH]; s_d, b_d [NH]
  int proj;                 // floats: s_p, b_p [Cs_out]
  int bars, total;
};
__host__ __device__ inline MbSmem mb_smem(int Cs_in, int Cs_out, int T1, int NH, int hid_px) {
  MbSmem s;
  const int px = T1 * 128;
  s.a_in = 0;
  s.a_lbo = px * 16;
  int off = (Cs_in / 4) * s.a_lbo;
  off = (off + 127) / 128 * 128;
  s.b1 = off;  off += (int)mb_etile_bytes(Cs_in, NH);
  s.hid = off; s.hid_plane = hid_px * 16; off += (NH / 4) * s.hid_plane;
  s.a2 = off;  off += (NH / 4) * 2048;
  s.b2 = off;  off += (int)mb_ptile_bytes(Cs_out, NH);
  s.coef = off; off += 2 * 13 * NH * 4;
  s.proj = off; off += 2 * Cs_out * 4;
  s.bars = (off + 15) / 16 * 16;
  s.total = s.bars + 8 * 8 + 16;
  return s;
}

__device__ __forceinline__ float4 act4(float4 v, int act) {
  return make_float4(apply_act(v.x, act), apply_act(v.y, act), apply_act(v.z, act), apply_act(v.w, act));
}

// acc += a * b on two float32 lanes with one instruction (same rounding as two fmaf)
__device__ __forceinline__ void ffma2(float& acc0, float& acc1, float a0, float a1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb, rc;\n\t"
      "mov.b64 ra, {%2, %3};\n\t"
      "mov.b64 rb, {%4, %5};\n\t"
      "mov.b64 rc, {%0, %1};\n\t"
      "fma.rn.f32x2 rc, ra, rb, rc;\n\t"
      "mov.b64 {%0, %1}, rc;\n\t}"
      : "+f"(acc0), "+f"(acc1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

__device__ __forceinline__ void mb_cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

__global__ void __launch_bounds__(kMbThreads, 1)
mb_block_kernel(MbParams p, const LayerJob* __restrict__ jobs) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  const LayerJob job = jobs[blockIdx.y];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NH = p.NH;
  const MbSmem sm = mb_smem(p.Cs_in, p.Cs_out, p.T1, NH, p.hid_px);
  uint8_t* a_in = smem + sm.a_in;
  uint8_t* b1 = smem + sm.b1;
  uint8_t* hid = smem + sm.hid;
  uint8_t* a2 = smem + sm.a2;
  uint8_t* b2 = smem + sm.b2;
  float* coef = reinterpret_cast<float*>(smem + sm.coef);  // [2][13][NH]: by chunk parity
  float* s_p = reinterpret_cast<float*>(smem + sm.proj);
  float* b_p = s_p + p.Cs_out;
  // mbarriers: expansion MMAs done, projection MMAs done, expansion image landed, projection image
  // landed, coefficients of an even / odd chunk landed, every worker warp has read the expansion
  // accumulators, every worker warp has written its part of the projection operand
  const uint32_t bar1 = smem_u32(smem + sm.bars), bar2 = bar1 + 8, bar_w1 = bar1 + 16, bar_w2 = bar1 + 24, bar_cf = bar1 + 32;
  const uint32_t bar_hid = bar1 + 48, bar_a2 = bar1 + 56;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + sm.bars + 64);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  // ---- this CTA's band ------------------------------------------------------------------------
  const int img = blockIdx.x / p.bands, band = blockIdx.x - img * p.bands;
  const int y0 = band * p.Rb;
  const int rb = min(p.Rb, p.Ho - y0);
  const int Po = rb * p.Wo;                          // output pixels of the band (<= 128)
  const int y_first = y0 * p.stride - 1;             // image row of the band's first hidden row
  const int rows_in = (rb - 1) * p.stride + 3;
  const int Ph = rows_in * p.W;                      // hidden pixels of the band
  const int t1 = (Ph + 127) >> 7;
  const int Wp = p.W + 2;                            // hidden rows carry a zero column on both sides
  // Per lane, fixed over the chunks: where this lane's accumulator row of tile t goes in a hidden plane
  // (-1: past the band; bit 30: the row lies outside the image and is stored as zeros), and where the
  // 3x3 window of its it-th output pixel starts (-1: no such pixel)
  int hoff[5], dbase[4];
#pragma unroll
  for (int t = 0; t < 5; ++t) {
    const int ph = t * 128 + (warp & 3) * 32 + lane;
    const int rr = ph / p.W, xx = ph - rr * p.W;
    const int y_in = y_first + rr;
    hoff[t] = ph < Ph ? (((rr * Wp + xx + 1) * 16) | ((y_in < 0 || y_in >= p.H) ? (1 << 30) : 0)) : -1;
  }
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int o = it * 32 + lane;
    const int yo = o / p.Wo, xo = o - yo * p.Wo;
    dbase[it] = o < Po ? ((yo * p.stride) * Wp + xo * p.stride) * 16 : -1;
  }

  if (tid == 0) {
    for (int i = 0; i < 6; ++i) mbar_init(bar1 + 8 * i, 1);
    mbar_init(bar_hid, kMbWorkers);
    mbar_init(bar_a2, kMbWorkers);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMbWorkers) {
    tmem_alloc(smem_u32(s_tmem), (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  // input pixels of the band -> canonical planes, asynchronously (the border rows above / below an
  // image are stored in the tensor, so the run [pix0, pix0 + Ph) always exists)
  {
    const int U = p.Cs_in / 4;                       // 16-byte units of a pixel: hi planes, then lo planes
    const size_t pix0 = ((size_t)img * (p.H + 2) + (size_t)(y_first + 1)) * p.W;
    const uint4* src = reinterpret_cast<const uint4*>(job.in) + pix0 * U;
    const int n_units = Ph * U;
    const uint32_t dst0 = smem_u32(a_in);
    for (int idx = tid; idx < n_units; idx += kMbThreads) {
      const int px = idx / U, u = idx - px * U;
      mb_cp_async16(dst0 + (uint32_t)u * (uint32_t)sm.a_lbo + (uint32_t)px * 16u, src + idx);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  // ---- operand images of a chunk: bulk copies issued by thread 0 ---------------------------------
  const int etile_bytes = (int)mb_etile_bytes(p.Cs_in, NH), ptile_bytes = (int)mb_ptile_bytes(p.Cs_out, NH);
  const int b1_lbo = NH * 16, b2_lbo = p.Cs_out * 16;   // plane strides of the weight images
  int n_w1 = 0, n_w2 = 0, n_cf0 = 0, n_cf1 = 0;      // copies issued per barrier (thread 0)
  auto load_expand = [&](int cc) {                   // expansion image of chunk cc -> b1
    mbar_expect_tx(bar_w1, (uint32_t)etile_bytes);
    bulk_load(smem_u32(b1), job.w_pre + (size_t)cc * etile_bytes, (uint32_t)etile_bytes, bar_w1);
    ++n_w1;
  };
  auto load_project = [&](int cc) {                  // projection image of chunk cc -> b2
    mbar_expect_tx(bar_w2, (uint32_t)ptile_bytes);
    bulk_load(smem_u32(b2), job.w + (size_t)cc * ptile_bytes, (uint32_t)ptile_bytes, bar_w2);
    ++n_w2;
  };
  auto load_coef = [&](int cc) {                     // s_e, b_e and the depthwise rows of chunk cc -> coef[cc & 1]
    const uint32_t bar = bar_cf + 8 * (cc & 1);
    const uint32_t dst = smem_u32(coef + (cc & 1) * 13 * NH);
    mbar_expect_tx(bar, (uint32_t)(13 * NH * 4));
    bulk_load(dst, job.scale_pre + (size_t)cc * 2 * NH, (uint32_t)(2 * NH * 4), bar);
    bulk_load(dst + 2 * NH * 4, job.scale_mid + (size_t)cc * 11 * NH, (uint32_t)(11 * NH * 4), bar);
    if (cc & 1) ++n_cf1; else ++n_cf0;
  };

  constexpr uint32_t DESC_HI = (uint32_t)(128 >> 4) | (1u << 14);       // 128 bytes between groups of 8 rows; no swizzle
  constexpr uint32_t IDESC0 = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);   // f32 += bf16 x bf16, M = 128
  const uint32_t d1_col = (uint32_t)p.Cs_out;        // expansion accumulators behind the output accumulator
  const int n_halves = p.Cs_out > 256 ? 2 : 1;
  const int n_half = p.Cs_out / n_halves;
  // expansion MMAs of chunk cc: all tiles of the band, hi and lo halves of the pixels (called by the issuing warp)
  auto issue_expand = [&](int cc, uint32_t tmem_base) {
    const int nh = min(NH, p.Ch - cc * NH);
    if (!mbar_wait_warp(bar_w1, (uint32_t)(cc & 1), s_abort, p.error_flag)) return;   // the chunk's image has landed
    const uint32_t idesc = IDESC0 | ((uint32_t)(nh >> 3) << 17);
    // low descriptor words (address and plane stride in 16-byte units) advance by constant steps
    const uint32_t a_base = (smem_u32(a_in) >> 4) | (((uint32_t)sm.a_lbo >> 4) << 16);
    const uint32_t b_base = (smem_u32(b1) >> 4) | (((uint32_t)b1_lbo >> 4) << 16);
    const uint32_t a_kk = (uint32_t)(2 * sm.a_lbo) >> 4, a_part = (uint32_t)((p.Cs_in / 8) * sm.a_lbo) >> 4, b_kk = (uint32_t)(2 * b1_lbo) >> 4;
    const int ksteps = p.Cs_in / 16;
    for (int t = 0; t < t1; ++t) {
      const uint32_t d = tmem_base + d1_col + (uint32_t)(t * NH);
      for (int part = 0; part < 2; ++part) {
        uint32_t a_lo = a_base + (uint32_t)t * 128u + (uint32_t)part * a_part, b_lo = b_base;
        for (int kk = 0; kk < ksteps; ++kk, a_lo += a_kk, b_lo += b_kk)
          umma_bf16(d, ((uint64_t)DESC_HI << 32) | a_lo, ((uint64_t)DESC_HI << 32) | b_lo, idesc, (part | kk) ? 1u : 0u);
      }
    }
    umma_commit(bar1);
  };

  // ---- prologue ---------------------------------------------------------------------------------
  for (int n = tid; n < p.Cs_out; n += kMbThreads) {   // projection scale / bias (channels past Cout come out as zeros)
    s_p[n] = n < p.Cout ? job.scale[n] : 0.f;
    b_p[n] = n < p.Cout ? job.bias[n] : 0.f;
  }
  // the zero columns left and right of every hidden row: written once, no pass touches them again
  for (int i = tid; i < (NH >> 2) * rows_in * 2; i += kMbThreads) {
    const int pl = i / (rows_in * 2), r = (i >> 1) % rows_in, side = i & 1;
    *reinterpret_cast<float4*>(hid + (size_t)pl * sm.hid_plane + (size_t)(r * Wp + side * (Wp - 1)) * 16) = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();                                   // barriers initialised, band in place, tensor memory allocated
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  if (tid == kMbLeader) {
    load_expand(0);
    load_coef(0);
    load_project(0);
    if (p.n_chunks > 1) load_coef(1);
  }
  if (warp == kMbWorkers) issue_expand(0, tmem_base);
  bool alive = true;
  // named barrier of the 16 worker warps; the issuing warp runs beside them and meets them only through mbarriers
  // Whether to go on is decided by one thread before the barrier and read by all after it (two slots, used in
  // turn), so that every worker warp leaves the loop at the same barrier.
  volatile int* s_go = s_abort + 1;
  int sync_k = 0;
  auto workers_sync = [&]() -> bool {
    if (tid == 0) s_go[sync_k & 1] = *s_abort == 0;
    asm volatile("bar.sync 1, %0;" ::"n"(kMbWorkers * 32) : "memory");
    const bool go = s_go[sync_k & 1] != 0;
    ++sync_k;
    return go;
  };

  if (warp < kMbWorkers) {
    // =================== worker warps: accumulators -> hidden chunk -> depthwise -> projection operand ===========
    for (int c = 0; c < p.n_chunks; ++c) {
      const int nh = min(NH, p.Ch - c * NH);         // a multiple of 16
      // the chunk's expansion MMAs and coefficients: one warp polls, the others wait at the named barrier (which
      // also ends the depthwise pass of the chunk before: the hidden tile may be overwritten)
      if (warp == 0) {
        mbar_wait_warp(bar1, (uint32_t)(c & 1), s_abort, p.error_flag);
        mbar_wait_warp(bar_cf + 8 * (c & 1), (uint32_t)((c >> 1) & 1), s_abort, p.error_flag);
      }
      if (!workers_sync()) { alive = false; break; }
      tc_fence_after();
      // ---- A. expansion accumulators of chunk c -> hidden chunk (float32) ------------------------
      const int q = warp & 3, h = warp >> 2;
      const int groups = nh >> 4;
      const float* se = coef + (c & 1) * 13 * NH;
      const float* be = se + NH;
      if (warp < kMbWorkers) {
#pragma unroll
        for (int t = 0; t < 5; ++t) {
          if (t >= t1) break;
          for (int cg = 0; cg < groups; ++cg) {
            if (((t * groups + cg) & 3) != h) continue;      // the four warps of a lane quarter take turns
            uint32_t v[16];
            tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + d1_col + (uint32_t)(t * NH + cg * 16), v);
            tmem_ld_wait();
            if (hoff[t] < 0) continue;
            const bool outside = (hoff[t] >> 30) & 1;
            uint8_t* dst = hid + (size_t)(cg * 4) * sm.hid_plane + (hoff[t] & 0xFFFFFF);
#pragma unroll
            for (int e = 0; e < 16; e += 4) {
              const float4 sc = *reinterpret_cast<const float4*>(se + cg * 16 + e);
              const float4 bi = *reinterpret_cast<const float4*>(be + cg * 16 + e);
              float4 o = make_float4(bi.x, bi.y, bi.z, bi.w);
              ffma2(o.x, o.y, __uint_as_float(v[e]), __uint_as_float(v[e + 1]), sc.x, sc.y);
              ffma2(o.z, o.w, __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]), sc.z, sc.w);
              o = act4(o, p.act_e);
              if (outside) o = make_float4(0.f, 0.f, 0.f, 0.f);
              *reinterpret_cast<float4*>(dst + (size_t)(e >> 2) * sm.hid_plane) = o;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_hid);           // this warp has read its accumulators
      // the projection of chunk c - 1 must have read a2 before the depthwise pass overwrites it
      if (warp == 0 && c > 0) mbar_wait_warp(bar2, (uint32_t)((c - 1) & 1), s_abort, p.error_flag);
      if (!workers_sync()) { alive = false; break; }   // the hidden chunk is complete
      // ---- D. depthwise 3x3 on the hidden chunk -> A operand of the projection ---------------------
      for (int pl = warp < kMbWorkers ? warp : (nh >> 2); pl < (nh >> 2); pl += kMbWorkers) {
        float4 wv[9];
        const float* w_d = coef + (c & 1) * 13 * NH + 2 * NH;       // [9][NH], then s_d [NH], b_d [NH]
#pragma unroll
        for (int t = 0; t < 9; ++t) wv[t] = *reinterpret_cast<const float4*>(w_d + t * NH + pl * 4);
        const float4 sc = *reinterpret_cast<const float4*>(w_d + 9 * NH + pl * 4);
        const float4 bi = *reinterpret_cast<const float4*>(w_d + 10 * NH + pl * 4);
        const uint8_t* hp = hid + (size_t)pl * sm.hid_plane;
        uint8_t* dst_hi = a2 + (size_t)(pl >> 1) * 2048 + (pl & 1) * 8;
        uint8_t* dst_lo = dst_hi + (size_t)(NH >> 3) * 2048;
#pragma unroll
        for (int it = 0; it < 4; ++it) {
          if (dbase[it] < 0) continue;
          const uint8_t* r0 = hp + dbase[it];
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int dy = 0; dy < 3; ++dy) {
#pragma unroll
            for (int dx = 0; dx < 3; ++dx) {
              const float4 hv = *reinterpret_cast<const float4*>(r0 + (size_t)(dy * Wp + dx) * 16);
              const float4 w = wv[dy * 3 + dx];
              ffma2(acc.x, acc.y, hv.x, hv.y, w.x, w.y);
              ffma2(acc.z, acc.w, hv.z, hv.w, w.z, w.w);
            }
          }
          float4 u = bi;
          ffma2(u.x, u.y, acc.x, acc.y, sc.x, sc.y);
          ffma2(u.z, u.w, acc.z, acc.w, sc.z, sc.w);
          u = act4(u, p.act_d);
          uint2 hi, lo;
          split_pair(u.x, u.y, hi.x, lo.x);
          split_pair(u.z, u.w, hi.y, lo.y);
          const int o = it * 32 + lane;
          *reinterpret_cast<uint2*>(dst_hi + o * 16) = hi;
          *reinterpret_cast<uint2*>(dst_lo + o * 16) = lo;
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_a2);            // this warp's part of the projection operand is written
    }
    // the last projection
    if (alive) {
      if (warp == 0) mbar_wait_warp(bar2, (uint32_t)((p.n_chunks - 1) & 1), s_abort, p.error_flag);
      alive = workers_sync();
    }
  } else {
    // =================== issuing warp: bulk copies and MMAs ===================================================
    for (int c = 0; c < p.n_chunks && alive; ++c) {
      const int nh = min(NH, p.Ch - c * NH);
      // chunk c's expansion MMAs are done: b1 is free for the next image
      alive = mbar_wait_warp(bar1, (uint32_t)(c & 1), s_abort, p.error_flag);
      if (!alive) break;
      if (lane == 0 && c + 1 < p.n_chunks) load_expand(c + 1);
      // every worker has read the accumulators of chunk c: the expansion MMAs of the next chunk may overwrite them
      alive = mbar_wait_warp(bar_hid, (uint32_t)(c & 1), s_abort, p.error_flag);
      if (!alive) break;
      if (c + 1 < p.n_chunks) {
        tc_fence_after();
        issue_expand(c + 1, tmem_base);
      }
      // the depthwise pass of chunk c is complete: its coefficient buffer is free, the projection can run
      alive = mbar_wait_warp(bar_a2, (uint32_t)(c & 1), s_abort, p.error_flag);
      if (!alive) break;
      if (lane == 0 && c + 2 < p.n_chunks) load_coef(c + 2);
      alive = mbar_wait_warp(bar_w2, (uint32_t)(c & 1), s_abort, p.error_flag);
      if (!alive) break;
      tc_fence_after();
      {
      const uint32_t idesc = IDESC0 | ((uint32_t)(n_half >> 3) << 17);
      const uint32_t a_base = (smem_u32(a2) >> 4) | ((2048u >> 4) << 16);
      const uint32_t b_base = (smem_u32(b2) >> 4) | (((uint32_t)b2_lbo >> 4) << 16);
      const uint32_t b_kk = (uint32_t)(2 * b2_lbo) >> 4, b_half = (uint32_t)(n_half * 16) >> 4;
      for (int part = 0; part < 2; ++part) {
        uint32_t a_lo = a_base + (uint32_t)(part * (NH >> 3)) * 128u, b_lo = b_base;
        for (int kk = 0; kk < (nh >> 4); ++kk, a_lo += 256u, b_lo += b_kk)
          for (int hf = 0; hf < n_halves; ++hf)
            umma_bf16(tmem_base + (uint32_t)(hf * n_half), ((uint64_t)DESC_HI << 32) | a_lo,
                      ((uint64_t)DESC_HI << 32) | (b_lo + (uint32_t)hf * b_half), idesc, (c | part | kk) ? 1u : 0u);
      }
      }
      umma_commit(bar2);
      // the next projection image may land once these MMAs have read b2
      if (c + 1 < p.n_chunks) {
        alive = mbar_wait_warp(bar2, (uint32_t)(c & 1), s_abort, p.error_flag);
        if (!alive) break;
        if (lane == 0) load_project(c + 1);
      }
    }
  }

  // ---- output: accumulator -> scale, bias, shortcut, activation -> hi / lo pixels ------------------
  alive = __syncthreads_and(alive);                  // every thread: the two roles meet again here
  if (alive) {
    tc_fence_after();
    const int q = warp & 3, h = warp >> 2;
    const int o = q * 32 + lane;
    const bool valid = o < Po;
    const int yo = y0 + o / p.Wo, xo = o % p.Wo;
    const size_t opix = ((size_t)img * (p.Ho + 2) + (size_t)(yo + 1)) * p.Wo + xo;   // shortcut: same geometry
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(job.out) + opix * (size_t)(2 * p.Cs_out);
    const __nv_bfloat16* res = job.res ? static_cast<const __nv_bfloat16*>(job.res) + opix * (size_t)(2 * p.Cs_out) : nullptr;
    for (int cg = warp < kMbWorkers ? h : (p.Cs_out >> 4); cg < (p.Cs_out >> 4); cg += kMbWorkers / 4) {
      uint32_t v[16];
      tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(cg * 16), v);
      tmem_ld_wait();
      if (!valid) continue;
      const int n = cg * 16;
      uint32_t rh[8] = {0, 0, 0, 0, 0, 0, 0, 0}, rl[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      if (res) {
        const uint4 a0 = __ldg(reinterpret_cast<const uint4*>(res + n)), a1 = __ldg(reinterpret_cast<const uint4*>(res + n) + 1);
        const uint4 l0 = __ldg(reinterpret_cast<const uint4*>(res + p.Cs_out + n)), l1 = __ldg(reinterpret_cast<const uint4*>(res + p.Cs_out + n) + 1);
        rh[0] = a0.x; rh[1] = a0.y; rh[2] = a0.z; rh[3] = a0.w; rh[4] = a1.x; rh[5] = a1.y; rh[6] = a1.z; rh[7] = a1.w;
        rl[0] = l0.x; rl[1] = l0.y; rl[2] = l0.z; rl[3] = l0.w; rl[4] = l1.x; rl[5] = l1.y; rl[6] = l1.z; rl[7] = l1.w;
      }
      uint32_t hi[8], lo[8];
#pragma unroll
      for (int e = 0; e < 16; e += 2) {
        float u0 = fmaf(__uint_as_float(v[e]), s_p[n + e], b_p[n + e]);
        float u1 = fmaf(__uint_as_float(v[e + 1]), s_p[n + e + 1], b_p[n + e + 1]);
        u0 += __uint_as_float(rh[e >> 1] << 16) + __uint_as_float(rl[e >> 1] << 16);
        u1 += __uint_as_float(rh[e >> 1] & 0xFFFF0000u) + __uint_as_float(rl[e >> 1] & 0xFFFF0000u);
        split_pair(apply_act(u0, p.act_p), apply_act(u1, p.act_p), hi[e >> 1], lo[e >> 1]);
      }
      *reinterpret_cast<uint4*>(out + n) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *(reinterpret_cast<uint4*>(out + n) + 1) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
      *reinterpret_cast<uint4*>(out + p.Cs_out + n) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      *(reinterpret_cast<uint4*>(out + p.Cs_out + n) + 1) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
    }
    // the border rows of the output image are part of the tensor: the first and the last band write them
    const int row_units = p.Wo * p.Cs_out / 4;       // 16-byte units of one row
    if (band == 0) {
      uint4* z = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(job.out) + (size_t)img * (p.Ho + 2) * p.Wo * (2 * p.Cs_out));
      for (int i = tid; i < row_units; i += kMbThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (band == p.bands - 1) {
      uint4* z = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(job.out) +
                                          ((size_t)img * (p.Ho + 2) + (size_t)(p.Ho + 1)) * p.Wo * (2 * p.Cs_out));
      for (int i = tid; i < row_units; i += kMbThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
    }
  }

  // ---- teardown -------------------------------------------------------------------------------
  if (!alive && tid == kMbLeader) {                          // copies in flight must land before the CTA exits
    const uint32_t bars[4] = {bar_w1, bar_w2, bar_cf, bar_cf + 8};
    const int issued[4] = {n_w1, n_w2, n_cf0, n_cf1};
    for (int i = 0; i < 4; ++i) {
      if (!issued[i]) continue;
      const long long t0 = clock64();
      while (!mbar_try_wait(bars[i], (uint32_t)((issued[i] - 1) & 1)) && clock64() - t0 < kWaitLimitCycles) {}
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMbWorkers) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

// Operand images of a block's layers, built once per weight version (see the file header):
//   role 0, expansion  (N = Ch rows of K = Cin codes): per chunk [Cs_in / 8 planes][NH rows][8 bfloat16];
//           coefficients per chunk: s_e [NH], b_e [NH]
//   role 1, projection (N = Cout rows of K = Ch codes): per chunk [NH / 8 planes][Cs_out rows][8 bfloat16]
//   role 2, depthwise  (N = Ch rows of 9 elements): coefficients per chunk: w [9][NH], s_d [NH], b_d [NH]
// Rows, planes and channels past the layer's extent are zero.
__global__ void mb_build_tiles_kernel(int role, const uint8_t* __restrict__ packed, const float* __restrict__ scale,
                                      const float* __restrict__ bias, int bits, int N, int K, int NH, int cs,
                                      uint8_t* __restrict__ tile, float* __restrict__ coef) {
  const int wrow = (K + 31) / 32 * 32 * bits / 8;
  const int Ch = role == 1 ? K : N;                  // hidden channels
  const int n_chunks = (Ch + NH - 1) / NH;
  const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gsize = gridDim.x * blockDim.x;
  if (role == 0 || role == 1) {
    const int planes = role == 0 ? cs / 8 : NH / 8;
    const int rows = role == 0 ? NH : cs;
    const int units = n_chunks * planes * rows;
    for (int u = gtid; u < units; u += gsize) {
      const int r = u % rows, j = (u / rows) % planes, c = u / (rows * planes);
      const int n = role == 0 ? c * NH + r : r;      // weight row
      const int k = role == 0 ? j * 8 : c * NH + j * 8;
      const bool real = n < N && k < K;
      uint2 raw = make_uint2(0u, 0u);
      if (real) {
        const uint8_t* row = packed + (size_t)n * wrow;
        if (bits == 8) raw = *reinterpret_cast<const uint2*>(row + k);
        else raw.x = *reinterpret_cast<const uint32_t*>(row + (k >> 1));
      }
      uint32_t o[4];
      expand8_bf16(raw, bits, o);
      reinterpret_cast<uint4*>(tile)[u] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
  if (role == 0) {
    for (int i = gtid; i < n_chunks * 2 * NH; i += gsize) {
      const int n = (i / (2 * NH)) * NH + i % NH;
      const bool is_bias = (i / NH) & 1;
      coef[i] = n < N ? (is_bias ? bias[n] : scale[n]) : 0.f;
    }
  } else if (role == 2) {
    for (int i = gtid; i < n_chunks * 11 * NH; i += gsize) {
      const int c = i / (11 * NH), t = (i / NH) % 11, n = c * NH + i % NH;
      float v = 0.f;
      if (n < N) v = t < 9 ? load_element(packed + (size_t)n * wrow, t, bits) : (t == 9 ? scale[n] : bias[n]);
      coef[i] = v;
    }
  }
}

struct MbConfig { int Rb, bands, T1, NH, occ, tmem_cols, smem_bytes; bool ok; };

MbConfig mb_config(const ConvGeom& ge, const ConvGeom& gd, const ConvGeom& gp, int smem_optin) {
  MbConfig c = {};
  const int cs_in = padded_channels(ge.Cin), cs_out = padded_channels(gp.Cout);
  // bands of up to 128 output pixels; shorter bands where the input rows of a full one do not fit
  for (int rb = std::min(std::max(128 / gp.Wo, 1), gp.Ho); rb >= 1 && !c.ok; rb >>= 1) {
    const int rows_in = (rb - 1) * gd.stride + 3;
    const int T1 = (rows_in * gd.W + 127) / 128;
    // one CTA (16 warps) per SM; 64-channel chunks where they fit
    const int order[2][2] = {{64, 1}, {32, 1}};
    for (int i = 0; i < 2 && !c.ok; ++i) {
      const int nh = order[i][0], occ = order[i][1];
      int cols = 32;
      while (cols < cs_out + T1 * nh) cols <<= 1;
      const int bytes = mb_smem(cs_in, cs_out, T1, nh, rows_in * (gd.W + 2)).total + 128;
      if (cols > 512 || bytes > smem_optin) continue;
      c.Rb = rb; c.bands = (gp.Ho + rb - 1) / rb; c.T1 = T1;
      c.NH = nh; c.occ = occ; c.tmem_cols = cols; c.smem_bytes = bytes; c.ok = true;
    }
  }
  return c;
}

bool mb_shape_ok(const ConvGeom& ge, const ConvGeom& gd, const ConvGeom& gp) {
  if (ge.act_format != ACT_SPLIT || ge.in_is_nchw) return false;
  if (ge.ks != 1 || ge.stride != 1 || ge.pad != 0 || gp.ks != 1 || gp.stride != 1 || gp.pad != 0) return false;
  if (gd.ks != 3 || gd.pad != 1 || (gd.stride != 1 && gd.stride != 2)) return false;
  if (ge.Cout != gd.Cin || gd.Cin != gd.Cout || gd.Cout != gp.Cin) return false;
  if (ge.H != gd.H || ge.W != gd.W || gd.Ho != gp.H || gd.Wo != gp.W) return false;
  if (ge.Cin % 8 != 0 || ge.Cout % 16 != 0) return false;
  const int cs_out = padded_channels(gp.Cout);
  if (cs_out > 512 || (cs_out > 256 && (cs_out / 2) % 16 != 0)) return false;
  if (gp.Wo > 128 || gp.Wo < 1) return false;
  return true;
}

}  // namespace

int mb_block_chunk_channels(const ConvGeom& ge, const ConvGeom& gd, const ConvGeom& gp) {
  if (!mb_shape_ok(ge, gd, gp)) return 0;
  DeviceProps props;
  if (current_device_props(&props) != AIQ_OK) return 0;
  const MbConfig c = mb_config(ge, gd, gp, props.smem_optin);
  return c.ok ? c.NH : 0;
}

// Where the fused kernel was measured faster than the three layer kernels (B200, both MobileNetV2 variants, batches
// 32 and 256): blocks on maps at most 8 columns wide and stride-2 blocks on maps up to 56 wide, once the batch
// gives at least 128 CTAs; elsewhere (wide maps: many waves of short CTAs; few CTAs: the chunks of a CTA run one
// after the other) the layer kernels win.
bool mb_block_pays(const ConvGeom& gd, const ConvGeom& gp) {
  DeviceProps props;
  if (current_device_props(&props) != AIQ_OK) return false;
  const int rb = std::min(std::max(128 / gp.Wo, 1), gp.Ho);        // band height of mb_config's first choice
  const long long ctas = (long long)gp.B * ((gp.Ho + rb - 1) / rb);
  if (ctas < 128) return false;
  return gd.W <= 8 || (gd.stride == 2 && gd.W <= 56);
}

aiq_status_t launch_mb_build_tiles(int role, const uint8_t* packed, const float* scale, const float* bias, int bits, int N,
                                   int K, int nh, int cs, void* tile_out, float* coef_out, cudaStream_t s) {
  if ((role == 0 || role == 1) && bits != 4 && bits != 8)
    return set_error(AIQ_ERR_UNSUPPORTED_BITS, "mb_build_tiles: the 1x1 layers of a fused block take 4- or 8-bit codes");
  mb_build_tiles_kernel<<<64, 256, 0, s>>>(role, packed, scale, bias, bits, N, K, nh, cs, static_cast<uint8_t*>(tile_out), coef_out);
  AIQ_LAUNCH_CHECK("mb_build_tiles");
  return AIQ_OK;
}

// jobs: one per version of the projection layer; `in` = the block's input (also the shortcut when `res` is set);
// w_pre / scale_pre = operand images / coefficients of the expansion, scale_mid = coefficients of the depthwise
// layer, w = operand images of the projection (launch_mb_build_tiles), scale / bias = those of the projection.
aiq_status_t launch_mb_block(const ConvGeom& ge, const ConvGeom& gd, const ConvGeom& gp, int nh, const LayerJob* jobs_dev, int n_jobs,
                             int32_t* error_flag, double weight_bytes, cudaStream_t s) {
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  if (!mb_shape_ok(ge, gd, gp)) return set_error(AIQ_ERR_SHAPE, "mb_block: unsupported block shape");
  const MbConfig c = mb_config(ge, gd, gp, props.smem_optin);
  if (!c.ok) return set_error(AIQ_ERR_SHAPE, "mb_block: shared or tensor memory does not fit");
  if (c.NH != nh) return set_error(AIQ_ERR_SHAPE, "mb_block: operand images were built for chunks of %d channels, the kernel wants %d", nh, c.NH);
  MbParams p = {};
  p.H = gd.H; p.W = gd.W; p.Ho = gd.Ho; p.Wo = gd.Wo; p.stride = gd.stride;
  p.Cin = ge.Cin; p.Cs_in = padded_channels(ge.Cin); p.Ch = ge.Cout; p.Cout = gp.Cout; p.Cs_out = padded_channels(gp.Cout);
  p.Rb = c.Rb; p.bands = c.bands; p.T1 = c.T1; p.NH = c.NH; p.n_chunks = (p.Ch + c.NH - 1) / c.NH;
  p.tmem_cols = c.tmem_cols;
  p.hid_px = ((c.Rb - 1) * gd.stride + 3) * (gd.W + 2);
  p.act_e = ge.act; p.act_d = gd.act; p.act_p = gp.act;
  p.error_flag = error_flag;
  AIQ_ENSURE_DYNAMIC_SMEM(mb_block_kernel, props.smem_optin);
  {
    const double px_in = (double)ge.B * ge.H * ge.W, px_out = (double)gp.B * gp.Ho * gp.Wo;
    LaunchScope scope(AIQ_KERNEL_CONV_TC, s,
                      n_jobs * (2.0 * px_in * ge.Cin * ge.Cout + 2.0 * px_out * 9.0 * gd.Cout + 2.0 * px_out * gp.Cin * gp.Cout),
                      weight_bytes + 4.0 * n_jobs * (px_in * ge.Cin + px_out * gp.Cout));
    mb_block_kernel<<<dim3((unsigned)(ge.B * c.bands), (unsigned)n_jobs), kMbThreads, c.smem_bytes, s>>>(p, jobs_dev);
  }
  AIQ_LAUNCH_CHECK("mb_block");
  return AIQ_OK;
}

}  // namespace aiq
