// Fake-quantization kernels: Q_w(W * scale) for the group-wise asymmetric setting and the int8
// symmetric row / token quantizers (paper Sec. 2.2 quantizer; Sec. 3.2.1 f_q).
//
// All are streaming kernels whose floor is HBM bandwidth: a tile of the bf16 source is staged once
// in shared memory and re-used for every scale candidate, so the source is read once and each
// candidate's operand is written once.  The arithmetic is kept off the slow conversion / reciprocal
// unit: rounding to an integer is the add-and-subtract of 1.5*2^23 (exact round-half-even in
// binary32 for |x| < 2^22), clamping is done before rounding and in floating point, int8 codes are read out of the low
// mantissa bits, and the per-element quotient value/step is taken as value * (1/step) with an exact
// IEEE division only when the product lies so close to a rounding tie that the two could round
// differently.  The integer produced is therefore always rint(fl32(value / step)), the contract the
// CPU reference uses, at a fraction of the instruction count.
#include "common.cuh"

namespace tlq {

namespace {

constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23

// rint(x) for |x| <= 2^21 without a conversion instruction.
__device__ __forceinline__ float round_magic(float x) { return __fsub_rn(__fadd_rn(x, kMagic), kMagic); }

// Reciprocal to within one ulp (a single instruction on the special-function unit).
__device__ __forceinline__ float rcp_fast(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

// The rare exact path, kept out of line so the common path stays a dozen instructions.
__device__ __noinline__ float exact_quotient_rint(float v, float step, float lo, float hi) {
  const float exact = fminf(fmaxf(__fdiv_rn(v, step), lo), hi);
  return round_magic(exact);
}

// clamp(rint(fl32(v / step)), lo, hi) for integer bounds lo <= hi inside (-1024, 1024), given
// inv ~ 1/step to within one ulp.  Clamping before rounding gives the same integer because the bounds
// are integers and rounding is monotone.  fl32(v * inv) is within |q| * 2.4e-7 of the true quotient
// and fl32(v / step) within |q| * 6e-8, so with |q| < 1024 both lie within 2.5e-4 of it: when the
// product is farther than that from a rounding tie the two round to the same integer, otherwise the
// exact division decides.
__device__ __forceinline__ float quotient_rint_clamped(float v, float step, float inv, float lo, float hi) {
  const float q = fminf(fmaxf(__fmul_rn(v, inv), lo), hi);
  float r = round_magic(q);
  if (fabsf(__fsub_rn(q, r)) > 0.49975f) r = exact_quotient_rint(v, step, lo, hi);
  return r;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// Group-wise asymmetric weights (W4A16 and other widths).
// Tile: kGqRows x 512 channels.  A thread owns 16 consecutive channels, a warp spans the 512 channels
// of one row, the 8 warps of the CTA take 8 rows per pass.  A group of g channels is g/16 adjacent
// lanes: min/max go through xor-shuffles.  grid.z splits the candidates when the matrix alone
// would not fill the machine.
// ------------------------------------------------------------------------------------------------
constexpr int kGqRows = 32;
constexpr int kGqCols = 512;
constexpr int kGqThreads = 256;

__global__ void __launch_bounds__(kGqThreads)
fakequant_group_kernel(const uint16_t* __restrict__ W, const uint16_t* __restrict__ s_tab,
                       const float* __restrict__ rs_tab, int K, int k_per_cta, int64_t C2, int64_t C1, int group,
                       int qmax, uint16_t* __restrict__ dW, uint8_t* __restrict__ codes, float* __restrict__ steps,
                       int32_t* __restrict__ zeros) {
  __shared__ uint4 tile[kGqRows][kGqCols / 8];
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t c0 = (int64_t)blockIdx.x * kGqCols + lane * 16;
  const int64_t row0 = (int64_t)blockIdx.y * kGqRows;
  const bool col_ok = c0 < C1;                    // C1 % 16 == 0 is guaranteed by the group sizes
  const int lanes_per_group = group >> 4;
  const float qmax_f = (float)qmax;
  const int64_t ngroups = C1 / group;
  const int k_begin = blockIdx.z * k_per_cta;
  const int k_end = min(K, k_begin + k_per_cta);

  // stage the W tile (zeros outside the matrix)
#pragma unroll
  for (int p = 0; p < kGqRows / 8; ++p) {
    const int r = p * 8 + warp;
    uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
    if (col_ok && row0 + r < C2) {
      const uint16_t* src = W + (row0 + r) * C1 + c0;
      v0 = ld_nc_16(src);
      v1 = ld_nc_16(src + 8);
    }
    tile[r][lane * 2] = v0;
    tile[r][lane * 2 + 1] = v1;
  }
  __syncthreads();

  for (int k = k_begin; k < k_end; ++k) {
    float sv[16], rsv[16];
    if (s_tab != nullptr && col_ok) {
      const uint16_t* sp = s_tab + (int64_t)k * C1 + c0;
      float a[8], b[8];
      unpack8(*reinterpret_cast<const uint4*>(sp), a);
      unpack8(*reinterpret_cast<const uint4*>(sp + 8), b);
#pragma unroll
      for (int j = 0; j < 8; ++j) { sv[j] = a[j]; sv[8 + j] = b[j]; }
      if (rs_tab != nullptr) {
        const float4* rp = reinterpret_cast<const float4*>(rs_tab + (int64_t)k * C1 + c0);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float4 r4 = rp[j];
          rsv[j * 4] = r4.x; rsv[j * 4 + 1] = r4.y; rsv[j * 4 + 2] = r4.z; rsv[j * 4 + 3] = r4.w;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) rsv[j] = __fdiv_rn(1.0f, sv[j]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) { sv[j] = 1.0f; rsv[j] = 1.0f; }
    }
#pragma unroll 1
    for (int p = 0; p < kGqRows / 8; ++p) {
      const int r = p * 8 + warp;
      float w[16], pr[16];
      {
        float a[8], b[8];
        unpack8(tile[r][lane * 2], a);
        unpack8(tile[r][lane * 2 + 1], b);
#pragma unroll
        for (int j = 0; j < 8; ++j) { w[j] = a[j]; w[8 + j] = b[j]; }
      }
      float mx, mn;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        pr[j] = __fmul_rn(sv[j], w[j]);            // exact: 8-bit x 8-bit significands
        mx = (j == 0) ? pr[0] : fmaxf(mx, pr[j]);
        mn = (j == 0) ? pr[0] : fminf(mn, pr[j]);
      }
      for (int off = 1; off < lanes_per_group; off <<= 1) {
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
        mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, off));
      }
      const float range = fmaxf(__fsub_rn(mx, mn), TLQ_RANGE_FLOOR);
      const float step = __fdiv_rn(range, qmax_f);
      const float inv = rcp_fast(step);
      // zero-point z = clamp(-rint(mn / step), 0, qmax), kept as a float
      const float zf = -quotient_rint_clamped(mn, step, inv, -qmax_f, 0.0f);
      const float lo = -zf, hi = qmax_f - zf;          // bounds of q - z
      uint32_t outw[8];
      uint32_t qpack[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int j = 0; j < 16; j += 2) {
        float d[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float qz = quotient_rint_clamped(pr[j + h], step, inv, lo, hi);     // q - z
          const float dq = __fmul_rn(qz, step);
          const float w_hat = __fmul_rn(dq, rsv[j + h]);
          d[h] = __fsub_rn(w[j + h], w_hat);
          if (codes != nullptr)
            qpack[(j + h) >> 2] |= (__float_as_uint(__fadd_rn(__fadd_rn(qz, zf), kMagic)) & 0xFFu) << (((j + h) & 3) * 8);
        }
        outw[j >> 1] = pack_bf16x2(d[0], d[1]);
      }
      const int64_t row = row0 + r;
      if (col_ok && row < C2) {
        if (dW != nullptr) {
          uint4* dst = reinterpret_cast<uint4*>(dW + ((int64_t)k * C2 + row) * C1 + c0);
          dst[0] = make_uint4(outw[0], outw[1], outw[2], outw[3]);
          dst[1] = make_uint4(outw[4], outw[5], outw[6], outw[7]);
        }
        if (codes != nullptr)
          *reinterpret_cast<uint4*>(codes + row * C1 + c0) = make_uint4(qpack[0], qpack[1], qpack[2], qpack[3]);
        if ((lane % lanes_per_group) == 0) {
          const int64_t g = c0 / group;
          if (steps != nullptr) steps[row * ngroups + g] = step;
          if (zeros != nullptr) zeros[row * ngroups + g] = (int)zf;
        }
      }
    }
  }
}

int launch_fakequant_group(const uint16_t* W, const uint16_t* s, const float* rs, int K, int64_t C2, int64_t C1,
                           int group, int w_bits, uint16_t* dW, uint8_t* codes, float* steps, int32_t* zeros,
                           cudaStream_t st) {
  const int64_t ctas = ceil_div(C1, kGqCols) * ceil_div(C2, kGqRows);
  int64_t kchunks = ceil_div(148 * 6, ctas);        // aim for several CTAs per SM
  if (kchunks > K) kchunks = K;
  if (kchunks < 1) kchunks = 1;
  const int k_per_cta = (int)ceil_div(K, kchunks);
  kchunks = ceil_div(K, k_per_cta);
  dim3 grid((unsigned)ceil_div(C1, kGqCols), (unsigned)ceil_div(C2, kGqRows), (unsigned)kchunks);
  fakequant_group_kernel<<<grid, kGqThreads, 0, st>>>(W, s, rs, K, k_per_cta, C2, C1, group, (1 << w_bits) - 1, dW,
                                                     codes, steps, zeros);
  return after_launch();
}

// ------------------------------------------------------------------------------------------------
// int8 symmetric quantization of whole rows: weights (value = scale * w, exact) or activations
// (value = x * (1/scale), one binary32 rounding).  One CTA owns a row at a time: the bf16 row is
// staged in shared memory, then for every candidate the row maximum is reduced and the codes are
// written, 16 per thread per store.
// ------------------------------------------------------------------------------------------------
constexpr int kRowThreads = 256;

template <bool kActivation>
__device__ __forceinline__ void scaled16(const uint4* row_smem, int64_t c, const uint16_t* s_row, const float* rs_row,
                                         float (&v)[16]) {
  float a[8], b[8];
  unpack8(row_smem[c >> 3], a);
  unpack8(row_smem[(c >> 3) + 1], b);
  if (kActivation) {
    if (rs_row != nullptr) {
      const float4* r4 = reinterpret_cast<const float4*>(rs_row + c);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 r = r4[j];
        float* src = (j < 2) ? a : b;
        const int o = (j & 1) * 4;
        v[j * 4 + 0] = __fmul_rn(src[o + 0], r.x); v[j * 4 + 1] = __fmul_rn(src[o + 1], r.y);
        v[j * 4 + 2] = __fmul_rn(src[o + 2], r.z); v[j * 4 + 3] = __fmul_rn(src[o + 3], r.w);
      }
    } else if (s_row != nullptr) {      // single scale vector given as bf16: take the reciprocal here
      float sa[8], sb[8];
      unpack8(*reinterpret_cast<const uint4*>(s_row + c), sa);
      unpack8(*reinterpret_cast<const uint4*>(s_row + c + 8), sb);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        v[j] = __fmul_rn(a[j], __fdiv_rn(1.0f, sa[j]));
        v[8 + j] = __fmul_rn(b[j], __fdiv_rn(1.0f, sb[j]));
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) { v[j] = a[j]; v[8 + j] = b[j]; }
    }
  } else {
    if (s_row != nullptr) {
      float sa[8], sb[8];
      unpack8(*reinterpret_cast<const uint4*>(s_row + c), sa);
      unpack8(*reinterpret_cast<const uint4*>(s_row + c + 8), sb);
#pragma unroll
      for (int j = 0; j < 8; ++j) { v[j] = __fmul_rn(sa[j], a[j]); v[8 + j] = __fmul_rn(sb[j], b[j]); }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) { v[j] = a[j]; v[8 + j] = b[j]; }
    }
  }
}

template <bool kActivation>
__global__ void __launch_bounds__(kRowThreads)
quant_rows_i8_kernel(const uint16_t* __restrict__ src, const uint16_t* __restrict__ s_tab,
                     const float* __restrict__ rs_tab, int K, int64_t R, int64_t C1, int8_t* __restrict__ q,
                     float* __restrict__ step_out) {
  extern __shared__ uint4 row_smem[];      // C1/8 packets
  __shared__ float warp_max[2][kRowThreads / 32];
  const int t = threadIdx.x;
  for (int64_t row = blockIdx.x; row < R; row += gridDim.x) {
    __syncthreads();
    for (int64_t i = t; i < C1 / 8; i += kRowThreads) row_smem[i] = ld_nc_16(src + row * C1 + i * 8);
    __syncthreads();
    for (int k = 0; k < K; ++k) {
      const uint16_t* s_row = (s_tab != nullptr) ? s_tab + (int64_t)k * C1 : nullptr;
      const float* rs_row = (rs_tab != nullptr) ? rs_tab + (int64_t)k * C1 : nullptr;
      float amax = 0.0f;
      for (int64_t c = (int64_t)t * 16; c < C1; c += kRowThreads * 16) {
        float v[16];
        scaled16<kActivation>(row_smem, c, s_row, rs_row, v);
#pragma unroll
        for (int j = 0; j < 16; ++j) amax = fmaxf(amax, fabsf(v[j]));
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, off));
      float* wm = warp_max[k & 1];          // double-buffered: one barrier per candidate
      if ((t & 31) == 0) wm[t >> 5] = amax;
      __syncthreads();
      float m = wm[0];
#pragma unroll
      for (int w = 1; w < kRowThreads / 32; ++w) m = fmaxf(m, wm[w]);
      const float st = __fdiv_rn(fmaxf(m, TLQ_RANGE_FLOOR), 127.0f);
      const float inv = rcp_fast(st);
      if (t == 0) step_out[(int64_t)k * R + row] = st;
      int8_t* out = q + ((int64_t)k * R + row) * C1;
      for (int64_t c = (int64_t)t * 16; c < C1; c += kRowThreads * 16) {
        float v[16];
        scaled16<kActivation>(row_smem, c, s_row, rs_row, v);
        uint32_t pk[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float qi = quotient_rint_clamped(v[j], st, inv, -128.0f, 127.0f);
          pk[j >> 2] |= (__float_as_uint(__fadd_rn(qi, kMagic)) & 0xFFu) << ((j & 3) * 8);
        }
        *reinterpret_cast<uint4*>(out + c) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      }
    }
  }
}

template <bool kActivation>
static int launch_rows(const uint16_t* src, const uint16_t* s, const float* rs, int K, int64_t R, int64_t C1,
                       int8_t* q, float* step, cudaStream_t st) {
  const size_t smem = (size_t)C1 * 2;
  static bool configured = false;
  if (!configured) {
    TLQ_CUDA_TRY(cudaFuncSetAttribute(quant_rows_i8_kernel<kActivation>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      200 * 1024));
    configured = true;
  }
  int64_t grid = R < 148 * 8 ? R : 148 * 8;
  quant_rows_i8_kernel<kActivation><<<(unsigned)grid, kRowThreads, smem, st>>>(src, s, rs, K, R, C1, q, step);
  return after_launch();
}

int launch_fakequant_rows_i8(const uint16_t* W, const uint16_t* s, int K, int64_t C2, int64_t C1, int8_t* q, float* u,
                             cudaStream_t st) {
  return launch_rows<false>(W, s, nullptr, K, C2, C1, q, u, st);
}

int launch_actquant_i8(const uint16_t* X, const uint16_t* s, const float* rs, int K, int64_t N, int64_t C1, int8_t* q,
                       float* t, cudaStream_t st) {
  return launch_rows<true>(X, s, rs, K, N, C1, q, t, st);
}

}  // namespace tlq
