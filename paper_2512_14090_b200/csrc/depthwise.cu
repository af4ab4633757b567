// Depthwise 3x3 convolution (stride 1 or 2, pad 1) with bias, residual and activation.
//
// The layer moves 8 bytes per output element for 18 FLOP: it is bound by memory traffic, so
// the kernel is organised around wide, coalesced accesses and input reuse in registers:
//   - a thread owns 8 consecutive channels (16-byte loads: one for the hi and one for the lo
//     half of a split pixel, two for a float32 pixel) and 4 consecutive output columns;
//   - for each of the 3 input rows it loads the 6 (stride 1) or 9 (stride 2) input columns
//     its 4 outputs need once and feeds all taps from registers;
//   - work items (output row, column group, channel octet) are flattened with the channel
//     octet fastest, so consecutive lanes touch consecutive 16-byte units whatever the
//     channel count (32 .. 960 in MobileNetV2);
//   - the 9 x C expanded weights, scales and biases sit in shared memory; blocks are
//     persistent (grid-stride over items).
// Rows 0 and Ho+1 of every output image (the physical padding rows) are written as zeros.
//
// Two kernels share this organisation.  depthwise3x3_kernel gives a thread one output row of
// its columns: every output row re-reads its three input rows (from L1 / L2), which is fine
// for small launches that need the parallelism.  depthwise3x3_walk_kernel gives a thread up to
// 16 consecutive output rows: it walks down the input rows once, each row feeding the (up to
// three) output rows it belongs to.
#include "common.cuh"

namespace aiq {

namespace {

constexpr int kDwThreads = 256;
constexpr int kDwCols = 2;        // output columns per thread
constexpr int kWalkCh = 4;        // channels per thread of the row-walking kernel

template <int FMT>
__device__ __forceinline__ void load8(const void* __restrict__ base, size_t pixel, int c, int Cs, float* v) {
  if (FMT == ACT_SPLIT) {
    const __nv_bfloat16* px = static_cast<const __nv_bfloat16*>(base) + pixel * 2 * Cs;
    const uint4 h = __ldg(reinterpret_cast<const uint4*>(px + c));
    const uint4 l = __ldg(reinterpret_cast<const uint4*>(px + Cs + c));
    const uint32_t hw[4] = {h.x, h.y, h.z, h.w}, lw[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {          // a bfloat16 is the upper half of a float
      v[2 * i] = __uint_as_float(hw[i] << 16) + __uint_as_float(lw[i] << 16);
      v[2 * i + 1] = __uint_as_float(hw[i] & 0xFFFF0000u) + __uint_as_float(lw[i] & 0xFFFF0000u);
    }
  } else {
    const float* px = static_cast<const float*>(base) + pixel * Cs + c;
    const float4 a = __ldg(reinterpret_cast<const float4*>(px)), b = __ldg(reinterpret_cast<const float4*>(px) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}

template <int FMT>
__device__ __forceinline__ void store8(void* __restrict__ base, size_t pixel, int c, int Cs, const float* v) {
  if (FMT == ACT_SPLIT) {
    __nv_bfloat16* px = static_cast<__nv_bfloat16*>(base) + pixel * 2 * Cs;
    uint32_t hw[4], lw[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      // hi = bf16_rn(v), lo = bf16_rn(v - hi), two values per packed conversion (the roundings of split_bf16)
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      hw[i] = *reinterpret_cast<const uint32_t*>(&h);
      const __nv_bfloat162 l = __floats2bfloat162_rn(v[2 * i] - __uint_as_float(hw[i] << 16),
                                                     v[2 * i + 1] - __uint_as_float(hw[i] & 0xFFFF0000u));
      lw[i] = *reinterpret_cast<const uint32_t*>(&l);
    }
    *reinterpret_cast<uint4*>(px + c) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
    *reinterpret_cast<uint4*>(px + Cs + c) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
  } else {
    float* px = static_cast<float*>(base) + pixel * Cs + c;
    *reinterpret_cast<float4*>(px) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(px + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
}

// Expanded weights [9][Cs], scales [Cs] and biases [Cs] of one job -> shared memory.  A thread
// takes whole channels: the first tap brings the packed row (32 elements, 16 .. 128 bytes) into
// L1 and the other eight taps hit it, and the channels of a thread are independent loads.
__device__ __forceinline__ void stage_dw_params(const LayerJob& job, int Cout, int Cs, float* wsm, float* ssm, float* bsm) {
  const int wrow_bytes = 32 * job.bits / 8;              // K = 9 pads to 32 elements
#pragma unroll 4
  for (int c = threadIdx.x; c < Cs; c += kDwThreads) {
    const bool real = c < Cout;
    const uint8_t* row = job.w + (size_t)(real ? c : 0) * wrow_bytes;
#pragma unroll
    for (int tap = 0; tap < 9; ++tap) wsm[tap * Cs + c] = real ? load_element(row, tap, job.bits) : 0.f;
    ssm[c] = real ? job.scale[c] : 0.f;
    bsm[c] = real ? job.bias[c] : 0.f;
  }
}

template <int FMT, int STRIDE>
__global__ void __launch_bounds__(kDwThreads, 4)
depthwise3x3_kernel(ConvGeom g, const LayerJob* __restrict__ jobs) {
  extern __shared__ __align__(16) float dsm[];          // [9][Cs] weights, [Cs] scale, [Cs] bias
  const LayerJob job = jobs[blockIdx.y];
  const int Cs = g.Cs_out;                               // == Cs_in
  float* wsm = dsm;
  float* ssm = dsm + 9 * Cs;
  float* bsm = ssm + Cs;
  stage_dw_params(job, g.Cout, Cs, wsm, ssm, bsm);
  __syncthreads();

  constexpr int IN_COLS = (kDwCols - 1) * STRIDE + 3;    // 6 or 9 input columns per thread
  const int octs = Cs / 8;
  const int col_groups = (g.Wo + kDwCols - 1) / kDwCols;
  const int rows_out = g.B * (g.Ho + 2);
  const long long n_items = (long long)rows_out * col_groups * octs;
  for (long long item = (long long)blockIdx.x * kDwThreads + threadIdx.x; item < n_items;
       item += (long long)gridDim.x * kDwThreads) {
    const int oct = (int)(item % octs);
    const long long rest = item / octs;
    const int cg = (int)(rest % col_groups);
    const int jr = (int)(rest / col_groups);             // padded output row (image, y')
    const int b = jr / (g.Ho + 2), oyp = jr - b * (g.Ho + 2);
    const int c = oct * 8, ox0 = cg * kDwCols;
    float acc[kDwCols][8];
#pragma unroll
    for (int x = 0; x < kDwCols; ++x)
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[x][i] = 0.f;
    const bool interior = oyp >= 1 && oyp <= g.Ho;
    if (interior) {
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        const int iy = (oyp - 1) * STRIDE - 1 + r;       // unpadded input row
        if (iy < 0 || iy >= g.H) continue;
        const size_t row_pix = (size_t)(b * (g.H + 2) + iy + 1) * g.W;
        float in[IN_COLS][8];
#pragma unroll
        for (int xx = 0; xx < IN_COLS; ++xx) {
          const int ix = ox0 * STRIDE - 1 + xx;
          if (ix >= 0 && ix < g.W) {
            load8<FMT>(job.in, row_pix + ix, c, Cs, in[xx]);
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) in[xx][i] = 0.f;
          }
        }
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const float4 w0 = *reinterpret_cast<const float4*>(wsm + (r * 3 + t) * Cs + c);
          const float4 w1 = *reinterpret_cast<const float4*>(wsm + (r * 3 + t) * Cs + c + 4);
          const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
          for (int x = 0; x < kDwCols; ++x)
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[x][i] = fmaf(in[x * STRIDE + t][i], wv[i], acc[x][i]);
        }
      }
    }
    const float4 s0 = *reinterpret_cast<const float4*>(ssm + c), s1 = *reinterpret_cast<const float4*>(ssm + c + 4);
    const float4 b0 = *reinterpret_cast<const float4*>(bsm + c), b1 = *reinterpret_cast<const float4*>(bsm + c + 4);
    const float sc[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    const float bi[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
    for (int x = 0; x < kDwCols; ++x) {
      const int ox = ox0 + x;
      if (ox >= g.Wo) break;
      const size_t opix = (size_t)jr * g.Wo + ox;
      float v[8];
      if (interior) {
        float rs[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (job.res) load8<FMT>(job.res, opix, c, Cs, rs);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          v[i] = (c + i < g.Cout) ? apply_act(fmaf(acc[x][i], sc[i], bi[i]) + rs[i], g.act) : 0.f;
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
      }
      store8<FMT>(job.out, opix, c, Cs, v);
    }
  }
}


// Four channels of one pixel (the unit of the row-walking kernel).  `p` points at the group's
// first channel in the pixel (split format: in the hi half; the lo half is lo_off bytes on).
template <int FMT>
__device__ __forceinline__ void load4(const uint8_t* __restrict__ p, uint32_t lo_off, float* v) {
  if (FMT == ACT_SPLIT) {
    const uint2 h = __ldg(reinterpret_cast<const uint2*>(p));
    const uint2 l = __ldg(reinterpret_cast<const uint2*>(p + lo_off));
    v[0] = __uint_as_float(h.x << 16) + __uint_as_float(l.x << 16);            // a bfloat16 is the upper half of a float
    v[1] = __uint_as_float(h.x & 0xFFFF0000u) + __uint_as_float(l.x & 0xFFFF0000u);
    v[2] = __uint_as_float(h.y << 16) + __uint_as_float(l.y << 16);
    v[3] = __uint_as_float(h.y & 0xFFFF0000u) + __uint_as_float(l.y & 0xFFFF0000u);
  } else {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  }
}

template <int FMT>
__device__ __forceinline__ void store4(uint8_t* __restrict__ p, uint32_t lo_off, const float* v) {
  if (FMT == ACT_SPLIT) {
    uint32_t hw[2], lw[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      // hi = bf16_rn(v), lo = bf16_rn(v - hi), two values per packed conversion (the roundings of split_bf16)
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      hw[i] = *reinterpret_cast<const uint32_t*>(&h);
      const __nv_bfloat162 l = __floats2bfloat162_rn(v[2 * i] - __uint_as_float(hw[i] << 16),
                                                     v[2 * i + 1] - __uint_as_float(hw[i] & 0xFFFF0000u));
      lw[i] = *reinterpret_cast<const uint32_t*>(&l);
    }
    *reinterpret_cast<uint2*>(p) = make_uint2(hw[0], hw[1]);
    *reinterpret_cast<uint2*>(p + lo_off) = make_uint2(lw[0], lw[1]);
  } else {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
}

// Row-walking kernel.  A thread owns kWalkCh = 4 channels x kDwCols output columns and walks down up to
// `rb` consecutive output rows of one image, loading every input row once:
//   stride 1: input row y feeds output rows y - 1 (tap row 2), y (tap row 1) and y + 1 (tap row
//             0), held in three accumulator sets whose roles rotate from row to row;
//   stride 2: output row j takes input rows 2j - 1, 2j, 2j + 1; row 2j + 1 is also the first
//             tap row of output j + 1, whose product is carried over.
// The row loop is a real loop (three rotated copies of the body at stride 1), so the code stays
// small whatever `rb` is.  Input rows -1 and H are the physical padding rows of the image, which
// every kernel writes as zeros: they are loaded like any other row.
// acc[x][i] (+)= sum_t in[x * STRIDE + t][i] * w[(r, t)][c + i]
template <int STRIDE, bool ACCUMULATE>
__device__ __forceinline__ void dw_tap_row(const float* __restrict__ wsm, int Cs, int c, int r,
                                           const float (&in)[(kDwCols - 1) * STRIDE + 3][kWalkCh], float (&acc)[kDwCols][kWalkCh]) {
#pragma unroll
  for (int t = 0; t < 3; ++t) {
    const float4 w0 = *reinterpret_cast<const float4*>(wsm + (r * 3 + t) * Cs + c);
    const float wv[kWalkCh] = {w0.x, w0.y, w0.z, w0.w};
#pragma unroll
    for (int x = 0; x < kDwCols; ++x)
#pragma unroll
      for (int i = 0; i < kWalkCh; ++i) {
        const float prev = (ACCUMULATE || t > 0) ? acc[x][i] : 0.f;
        acc[x][i] = fmaf(in[x * STRIDE + t][i], wv[i], prev);
      }
  }
}

template <int FMT, int STRIDE>
__global__ void __launch_bounds__(kDwThreads, 3)
depthwise3x3_walk_kernel(ConvGeom g, const LayerJob* __restrict__ jobs, int rb) {
  extern __shared__ __align__(16) float dsm[];          // [9][Cs] weights, [Cs] scale, [Cs] bias
  const LayerJob job = jobs[blockIdx.y];
  const int Cs = g.Cs_out;                               // == Cs_in
  float* wsm = dsm;
  float* ssm = dsm + 9 * Cs;
  float* bsm = ssm + Cs;
  stage_dw_params(job, g.Cout, Cs, wsm, ssm, bsm);
  __syncthreads();

  constexpr int IN_COLS = (kDwCols - 1) * STRIDE + 3;    // input columns per thread
  const int octs = Cs / kWalkCh;                         // channel groups
  const int col_groups = (g.Wo + kDwCols - 1) / kDwCols;
  const int row_blocks = (g.Ho + rb - 1) / rb;
  const size_t pix_bytes = (size_t)4 * Cs;               // a pixel: [hi(Cs) | lo(Cs)] bfloat16 or Cs floats
  const uint32_t lo_off = 2u * Cs;                       // split format: bytes from the hi to the lo half
  const uint32_t in_pitch = (uint32_t)(g.W * pix_bytes), out_pitch = (uint32_t)(g.Wo * pix_bytes);
  const bool clamp = g.act != AIQ_ACT_NONE;              // relu: [0, inf), relu6: [0, 6]
  const float act_hi = g.act == AIQ_ACT_RELU6 ? 6.0f : __int_as_float(0x7f800000);
  const long long n_items = (long long)g.B * row_blocks * col_groups * octs;
  for (long long item = (long long)blockIdx.x * kDwThreads + threadIdx.x; item < n_items;
       item += (long long)gridDim.x * kDwThreads) {
    const int oct = (int)(item % octs);
    long long rest = item / octs;
    const int cg = (int)(rest % col_groups);
    rest /= col_groups;
    const int rbk = (int)(rest % row_blocks);
    const int b = (int)(rest / row_blocks);
    const int c = oct * kWalkCh, ox0 = cg * kDwCols;
    const uint32_t ch_off = (uint32_t)c * (FMT == ACT_SPLIT ? 2u : 4u);   // bytes from a pixel to its channel c
    const int oy0 = rbk * rb;                            // first (unpadded) output row of the block
    const int n_out = min(rb, g.Ho - oy0);               // output rows of this block
    const size_t out_row0 = (size_t)b * (g.Ho + 2);      // padded output row 0 of the image
    const size_t in_row0 = (size_t)b * (g.H + 2) + 1;    // padded input row of unpadded row 0
    const int ix0 = ox0 * STRIDE - 1;

    // Addresses are kept as running pointers: one per input column, stepped by a row after every
    // load (a column outside the image points at a pixel of the image's first padding row, which
    // holds zeros, and does not move), one for the output row and one for the residual row.
    const uint8_t* colp[IN_COLS];
    uint32_t colstep[IN_COLS];
    {
      const uint8_t* in_base = static_cast<const uint8_t*>(job.in) + ch_off;
      const size_t first_row = in_row0 + (size_t)(oy0 * STRIDE) - 1;      // padded row of m = 0 (>= in_row0 - 1)
#pragma unroll
      for (int xx = 0; xx < IN_COLS; ++xx) {
        const int ix = ix0 + xx;
        const bool inside = ix >= 0 && ix < g.W;
        colp[xx] = in_base + (inside ? first_row * g.W + ix : (in_row0 - 1) * g.W) * pix_bytes;
        colstep[xx] = inside ? in_pitch : 0u;
      }
    }
    auto load_next_row = [&](float (&in)[IN_COLS][kWalkCh]) {
#pragma unroll
      for (int xx = 0; xx < IN_COLS; ++xx) {
        load4<FMT>(colp[xx], lo_off, in[xx]);
        colp[xx] += colstep[xx];
      }
    };
    uint8_t* outp = static_cast<uint8_t*>(job.out) + ch_off + ((out_row0 + oy0 + 1) * g.Wo + ox0) * pix_bytes;
    const uint8_t* resp = job.res ? static_cast<const uint8_t*>(job.res) + (outp - static_cast<uint8_t*>(job.out)) : nullptr;

    // finish and store the next output row (rows are emitted in order) from its accumulators
    auto emit = [&](const float (&acc)[kDwCols][kWalkCh]) {
      const float4 s0 = *reinterpret_cast<const float4*>(ssm + c);
      const float4 b0 = *reinterpret_cast<const float4*>(bsm + c);
      const float sc[kWalkCh] = {s0.x, s0.y, s0.z, s0.w};
      const float bi[kWalkCh] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
      for (int x = 0; x < kDwCols; ++x) {
        if (ox0 + x >= g.Wo) break;
        float v[kWalkCh];
#pragma unroll
        for (int i = 0; i < kWalkCh; ++i) v[i] = fmaf(acc[x][i], sc[i], bi[i]);
        if (resp) {
          float rs[kWalkCh];
          load4<FMT>(resp + x * pix_bytes, lo_off, rs);
#pragma unroll
          for (int i = 0; i < kWalkCh; ++i) v[i] += rs[i];
        }
        if (clamp) {
#pragma unroll
          for (int i = 0; i < kWalkCh; ++i) v[i] = fminf(fmaxf(v[i], 0.f), act_hi);
        }
        if (c + kWalkCh > g.Cout) {                      // padding channels stay zero
#pragma unroll
          for (int i = 0; i < kWalkCh; ++i)
            if (c + i >= g.Cout) v[i] = 0.f;
        }
        store4<FMT>(outp + x * pix_bytes, lo_off, v);
      }
      outp += out_pitch;
      if (resp) resp += out_pitch;
    };

    if (STRIDE == 1) {
      // k-th input row of the block = unpadded row oy0 - 1 + k, k = 0 .. n_out + 1.  a0 / a1 / a2
      // belong to output rows oy0 + k - 2 / k - 1 / k; a0 is complete after this row.
      auto step = [&](int k, float (&a0)[kDwCols][kWalkCh], float (&a1)[kDwCols][kWalkCh], float (&a2)[kDwCols][kWalkCh]) {
        float in[IN_COLS][kWalkCh];
        load_next_row(in);                               // unpadded row oy0 - 1 + k (-1 .. H)
        // rows that belong to a neighbouring block are accumulated too and never stored
        dw_tap_row<STRIDE, true>(wsm, Cs, c, 2, in, a0);
        dw_tap_row<STRIDE, true>(wsm, Cs, c, 1, in, a1);
        dw_tap_row<STRIDE, false>(wsm, Cs, c, 0, in, a2);
        if (k >= 2) emit(a0);
      };
      float A[kDwCols][kWalkCh], B[kDwCols][kWalkCh], C[kDwCols][kWalkCh];
#pragma unroll
      for (int x = 0; x < kDwCols; ++x)
#pragma unroll
        for (int i = 0; i < kWalkCh; ++i) A[x][i] = B[x][i] = 0.f;
      const int n_rows = n_out + 2;
      for (int k = 0; k < n_rows; k += 3) {
        step(k, A, B, C);
        if (k + 1 < n_rows) step(k + 1, B, C, A);
        if (k + 2 < n_rows) step(k + 2, C, A, B);
      }
    } else {
      // output row j of the block takes unpadded input rows 2 (oy0 + j) - 1, .., + 1
      float acc[kDwCols][kWalkCh], carry[kDwCols][kWalkCh];
      float in[IN_COLS][kWalkCh];
#pragma unroll
      for (int x = 0; x < kDwCols; ++x)
#pragma unroll
        for (int i = 0; i < kWalkCh; ++i) carry[x][i] = 0.f;
      load_next_row(in);                                 // unpadded row 2 oy0 - 1
      dw_tap_row<STRIDE, false>(wsm, Cs, c, 0, in, carry);
      for (int j = 0; j < n_out; ++j) {
        load_next_row(in);                               // rows 2 (oy0 + j) and, below, + 1 (<= H)
#pragma unroll
        for (int x = 0; x < kDwCols; ++x)
#pragma unroll
          for (int i = 0; i < kWalkCh; ++i) acc[x][i] = carry[x][i];
        dw_tap_row<STRIDE, true>(wsm, Cs, c, 1, in, acc);
        load_next_row(in);
        dw_tap_row<STRIDE, true>(wsm, Cs, c, 2, in, acc);
        dw_tap_row<STRIDE, false>(wsm, Cs, c, 0, in, carry);
        emit(acc);
      }
    }
    // the two physical padding rows of the image, by the first and the last row block
    if (rbk == 0 || rbk == row_blocks - 1) {
      const float zero[kWalkCh] = {0, 0, 0, 0};
#pragma unroll
      for (int side = 0; side < 2; ++side) {
        if (side == 0 ? rbk != 0 : rbk != row_blocks - 1) continue;
        const size_t jr = out_row0 + (side == 0 ? 0 : g.Ho + 1);
#pragma unroll
        for (int x = 0; x < kDwCols; ++x)
          if (ox0 + x < g.Wo)
            store4<FMT>(static_cast<uint8_t*>(job.out) + ch_off + (jr * g.Wo + ox0 + x) * pix_bytes, lo_off, zero);
      }
    }
  }
}

}  // namespace

aiq_status_t launch_depthwise(const ConvGeom& g, const LayerJob* jobs_dev, int n_jobs,
                              const float* /*net_input*/, double weight_bytes, cudaStream_t s) {
  if (g.stride != 1 && g.stride != 2) return set_error(AIQ_ERR_SHAPE, "depthwise: stride %d is not supported", g.stride);
  const int Cs = g.Cs_out;
  const size_t smem = (size_t)11 * Cs * sizeof(float);
  DeviceProps props;
  if (aiq_status_t st = current_device_props(&props)) return st;
  const int n_sms = props.n_sms;
  if (smem > 48 * 1024) return set_error(AIQ_ERR_SHAPE, "depthwise: %d channels need %zu bytes of shared memory", g.Cout, smem);
  const int col_groups = (g.Wo + kDwCols - 1) / kDwCols;
  // Rows per thread of the row-walking kernel: the image height cut into the fewest blocks of at
  // most 16 rows, of equal height where it divides.  The kernel is used when it still gives
  // every SM a block of threads; smaller launches need the parallelism of one row per thread.
  const int n_blk = (g.Ho + 15) / 16;
  const int rb = (g.Ho + n_blk - 1) / n_blk;
  const long long items_rows = (long long)g.B * n_blk * col_groups * (Cs / kWalkCh);
  const bool walk_rows = items_rows >= (long long)n_sms * kDwThreads;
  const long long n_items = walk_rows ? items_rows : (long long)g.B * (g.Ho + 2) * col_groups * (Cs / 8);
  long long blocks = (n_items + kDwThreads - 1) / kDwThreads;
  const long long cap = (long long)n_sms * (walk_rows ? 3 : 4);   // persistent: as many blocks as are resident
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  dim3 grid((unsigned)blocks, n_jobs);
  LaunchScope scope(AIQ_KERNEL_DEPTHWISE, s, 18.0 * g.B * g.Ho * g.Wo * g.Cout * n_jobs,
                    weight_bytes + 4.0 * n_jobs * ((double)g.B * g.Cin * g.H * g.W +
                                                   (double)g.B * g.Ho * g.Wo * g.Cout));
  if (walk_rows) {
#define AIQ_DWR(FMT_, ST_) depthwise3x3_walk_kernel<FMT_, ST_><<<grid, kDwThreads, smem, s>>>(g, jobs_dev, rb)
    if (g.act_format == ACT_SPLIT) { if (g.stride == 1) AIQ_DWR(ACT_SPLIT, 1); else AIQ_DWR(ACT_SPLIT, 2); }
    else { if (g.stride == 1) AIQ_DWR(ACT_F32, 1); else AIQ_DWR(ACT_F32, 2); }
#undef AIQ_DWR
    AIQ_LAUNCH_CHECK("depthwise3x3_walk");
    return AIQ_OK;
  }
#define AIQ_DW(FMT_, ST_) depthwise3x3_kernel<FMT_, ST_><<<grid, kDwThreads, smem, s>>>(g, jobs_dev)
  if (g.act_format == ACT_SPLIT) { if (g.stride == 1) AIQ_DW(ACT_SPLIT, 1); else AIQ_DW(ACT_SPLIT, 2); }
  else { if (g.stride == 1) AIQ_DW(ACT_F32, 1); else AIQ_DW(ACT_F32, 2); }
#undef AIQ_DW
  AIQ_LAUNCH_CHECK("depthwise3x3");
  return AIQ_OK;
}

}  // namespace aiq
