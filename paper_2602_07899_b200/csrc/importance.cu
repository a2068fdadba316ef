// Token importance: imp[n] = sum_b norm(g[b,n,:]) and the top-fraction selection (paper Sec. 3.1.2,
// third equation and the Top-50% rule).  HBM-bound: the gradient tensor is read once with 128-bit
// loads.  One CTA owns one token position; its warps take the samples b round-robin, reduce one
// gradient row each with shuffles, and the per-sample norms are added in fp64 in a fixed order.
#include "common.cuh"

namespace tlq {

constexpr int kImpThreads = 256;
constexpr int kImpWarps = kImpThreads / 32;

template <bool kF32, bool kL2>
__global__ void __launch_bounds__(kImpThreads)
token_importance_kernel(const void* __restrict__ G, int64_t B, int64_t N, int64_t C, float* __restrict__ imp) {
  __shared__ double warp_sum[kImpWarps];
  const int64_t n = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  double acc = 0.0;   // this warp's samples, in increasing b
  for (int64_t b = warp; b < B; b += kImpWarps) {
    double row = 0.0;
    if (kF32) {
      const float* g = reinterpret_cast<const float*>(G) + (b * N + n) * C;
      for (int64_t c = (int64_t)lane * 4; c < C; c += 32 * 4) {
        const float4 v = *reinterpret_cast<const float4*>(g + c);
        float part;
        if (kL2) part = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        else part = fabsf(v.x) + fabsf(v.y) + fabsf(v.z) + fabsf(v.w);
        row += (double)part;
      }
    } else {
      const uint16_t* g = reinterpret_cast<const uint16_t*>(G) + (b * N + n) * C;
      int64_t c = (int64_t)lane * 8;
      // four 128-bit loads in flight per lane before any is consumed
      for (; c + 3 * 256 < C; c += 4 * 256) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_nc_16(g + c + u * 256);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          float f[8];
          unpack8(v[u], f);
          float part = 0.0f;
#pragma unroll
          for (int j = 0; j < 8; ++j) part += kL2 ? f[j] * f[j] : fabsf(f[j]);
          row += (double)part;
        }
      }
      for (; c < C; c += 256) {
        float f[8];
        unpack8(ld_nc_16(g + c), f);
        float part = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) part += kL2 ? f[j] * f[j] : fabsf(f[j]);
        row += (double)part;
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) row += __shfl_xor_sync(0xFFFFFFFFu, row, off);
    acc += kL2 ? sqrt(row) : row / (double)C;
  }
  if (lane == 0) warp_sum[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double v = 0.0;
#pragma unroll
    for (int w = 0; w < kImpWarps; ++w) v += warp_sum[w];
    imp[n] = (float)v;
  }
}

// mask[n] = 1 iff fewer than k_sel positions rank ahead of n (larger value, or equal value and lower index).
__global__ void top_mask_kernel(const float* __restrict__ imp, int64_t N, int64_t k_sel, uint8_t* __restrict__ mask) {
  __shared__ float chunk[1024];
  const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const float mine = (n < N) ? imp[n] : 0.0f;
  int64_t ahead = 0;
  for (int64_t base = 0; base < N; base += 1024) {
    __syncthreads();
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) chunk[i] = (base + i < N) ? imp[base + i] : -1.0f;
    __syncthreads();
    const int lim = (int)((N - base < 1024) ? (N - base) : 1024);
    for (int i = 0; i < lim; ++i) {
      const float v = chunk[i];
      ahead += (v > mine) || (v == mine && base + i < n);
    }
  }
  if (n < N) mask[n] = (ahead < k_sel) ? 1 : 0;
}

int launch_token_importance(const void* G, int g_dtype, int64_t B, int64_t N, int64_t C, int norm_kind, float* imp,
                            cudaStream_t st) {
  const unsigned grid = (unsigned)N;
  const bool f32 = g_dtype == TLQ_DTYPE_F32, l2 = norm_kind == TLQ_NORM_L2;
  if (f32 && l2) token_importance_kernel<true, true><<<grid, kImpThreads, 0, st>>>(G, B, N, C, imp);
  else if (f32) token_importance_kernel<true, false><<<grid, kImpThreads, 0, st>>>(G, B, N, C, imp);
  else if (l2) token_importance_kernel<false, true><<<grid, kImpThreads, 0, st>>>(G, B, N, C, imp);
  else token_importance_kernel<false, false><<<grid, kImpThreads, 0, st>>>(G, B, N, C, imp);
  return after_launch();
}

int launch_top_mask(const float* imp, int64_t N, int64_t k_sel, uint8_t* mask, cudaStream_t st) {
  const int threads = 256;
  top_mask_kernel<<<(unsigned)ceil_div(N, threads), threads, 0, st>>>(imp, N, k_sel, mask);
  return after_launch();
}

}  // namespace tlq
