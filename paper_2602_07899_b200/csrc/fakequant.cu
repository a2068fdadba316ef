// Fake-quantization kernels: Q_w(W * scale) for the group-wise asymmetric setting and the int8
// symmetric row / token quantizers (paper Sec. 2.2 quantizer; Sec. 3.2.1 f_q).
//
// All are HBM-bound streaming kernels: a tile of the bf16 source is staged once in shared memory
// and re-used for every scale candidate, so the source is read once and each candidate's operand
// is written once.  Where floating point decides an integer (step, zero-point, code) the operation
// is a single IEEE binary32 operation written with the *_rn intrinsics, so no contraction or
// approximate division can change a code.
#include "common.cuh"

namespace tlq {

// ------------------------------------------------------------------------------------------------
// Group-wise asymmetric weights (W4A16 and other widths).
// Tile: kGqRows x 512 channels; a thread owns 8 consecutive channels, 64 threads span the 512
// channels of one row, so one pass of the 256-thread CTA covers 4 rows.  A group of g channels is
// g/8 adjacent lanes of one warp: min/max go through xor-shuffles.
// ------------------------------------------------------------------------------------------------
constexpr int kGqRows = 16;
constexpr int kGqCols = 512;
constexpr int kGqThreads = 256;

__global__ void __launch_bounds__(kGqThreads)
fakequant_group_kernel(const uint16_t* __restrict__ W, const uint16_t* __restrict__ s_tab, int K, int64_t C2,
                       int64_t C1, int group, int qmax, uint16_t* __restrict__ dW, uint8_t* __restrict__ codes,
                       float* __restrict__ steps, int32_t* __restrict__ zeros) {
  __shared__ uint4 tile[kGqRows][kGqCols / 8];
  const int t = threadIdx.x;
  const int col8 = t & 63;          // which 8-channel packet of the 512-wide tile
  const int rsub = t >> 6;          // 0..3
  const int64_t c0 = (int64_t)blockIdx.x * kGqCols + col8 * 8;
  const int64_t row0 = (int64_t)blockIdx.y * kGqRows;
  const bool col_ok = c0 < C1;
  const int lanes_per_group = group >> 3;
  const float qmax_f = (float)qmax;
  const int64_t ngroups = C1 / group;

  // stage the W tile (zeros outside the matrix)
#pragma unroll
  for (int p = 0; p < kGqRows / 4; ++p) {
    const int r = p * 4 + rsub;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (col_ok && row0 + r < C2) v = ld_nc_16(W + (row0 + r) * C1 + c0);
    tile[r][col8] = v;
  }
  __syncthreads();

  for (int k = 0; k < K; ++k) {
    float sv[8];
    if (s_tab != nullptr && col_ok) {
      unpack8(*reinterpret_cast<const uint4*>(s_tab + (int64_t)k * C1 + c0), sv);
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) sv[j] = 1.0f;
    }
#pragma unroll
    for (int p = 0; p < kGqRows / 4; ++p) {
      const int r = p * 4 + rsub;
      float w[8], pr[8];
      unpack8(tile[r][col8], w);
      float mx, mn;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        pr[j] = __fmul_rn(sv[j], w[j]);            // exact: 8-bit x 8-bit significands
        mx = (j == 0) ? pr[0] : fmaxf(mx, pr[j]);
        mn = (j == 0) ? pr[0] : fminf(mn, pr[j]);
      }
      for (int off = 1; off < lanes_per_group; off <<= 1) {
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
        mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, off));
      }
      float range = fmaxf(__fsub_rn(mx, mn), TLQ_RANGE_FLOOR);
      const float step = __fdiv_rn(range, qmax_f);
      int z = -__float2int_rn(__fdiv_rn(mn, step));
      z = min(max(z, 0), qmax);
      uint32_t outw[4];
      uint32_t qpack[2] = {0u, 0u};
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        int q = __float2int_rn(__fdiv_rn(pr[j], step)) + z;
        q = min(max(q, 0), qmax);
        const float dq = __fmul_rn((float)(q - z), step);
        const float w_hat = __fdiv_rn(dq, sv[j]);
        const uint32_t b = float_to_bf16_bits(__fsub_rn(w[j], w_hat));
        if (j & 1) outw[j >> 1] |= b << 16; else outw[j >> 1] = b;
        qpack[j >> 2] |= (uint32_t)q << ((j & 3) * 8);
      }
      const int64_t row = row0 + r;
      if (col_ok && row < C2) {
        if (dW != nullptr)
          *reinterpret_cast<uint4*>(dW + ((int64_t)k * C2 + row) * C1 + c0) = make_uint4(outw[0], outw[1], outw[2], outw[3]);
        if (codes != nullptr) *reinterpret_cast<uint2*>(codes + row * C1 + c0) = make_uint2(qpack[0], qpack[1]);
        if ((col8 % lanes_per_group) == 0) {
          const int64_t g = c0 / group;
          if (steps != nullptr) steps[row * ngroups + g] = step;
          if (zeros != nullptr) zeros[row * ngroups + g] = z;
        }
      }
    }
  }
}

int launch_fakequant_group(const uint16_t* W, const uint16_t* s, int K, int64_t C2, int64_t C1, int group,
                           int w_bits, uint16_t* dW, uint8_t* codes, float* steps, int32_t* zeros,
                           cudaStream_t st) {
  dim3 grid((unsigned)ceil_div(C1, kGqCols), (unsigned)ceil_div(C2, kGqRows));
  fakequant_group_kernel<<<grid, kGqThreads, 0, st>>>(W, s, K, C2, C1, group, (1 << w_bits) - 1, dW, codes, steps,
                                                     zeros);
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
  __shared__ float warp_max[kRowThreads / 32];
  __shared__ float row_step;
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
      if ((t & 31) == 0) warp_max[t >> 5] = amax;
      __syncthreads();
      if (t == 0) {
        float m = warp_max[0];
#pragma unroll
        for (int w = 1; w < kRowThreads / 32; ++w) m = fmaxf(m, warp_max[w]);
        const float st = __fdiv_rn(fmaxf(m, TLQ_RANGE_FLOOR), 127.0f);
        row_step = st;
        step_out[(int64_t)k * R + row] = st;
      }
      __syncthreads();
      const float st = row_step;
      int8_t* out = q + ((int64_t)k * R + row) * C1;
      for (int64_t c = (int64_t)t * 16; c < C1; c += kRowThreads * 16) {
        float v[16];
        scaled16<kActivation>(row_smem, c, s_row, rs_row, v);
        uint32_t pk[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          int qi = __float2int_rn(__fdiv_rn(v[j], st));
          qi = min(max(qi, -128), 127);
          pk[j >> 2] |= ((uint32_t)qi & 0xFFu) << ((j & 3) * 8);
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

int launch_actquant_i8(const uint16_t* X, const float* rs, int K, int64_t N, int64_t C1, int8_t* q, float* t,
                       cudaStream_t st) {
  return launch_rows<true>(X, nullptr, rs, K, N, C1, q, t, st);
}

}  // namespace tlq
