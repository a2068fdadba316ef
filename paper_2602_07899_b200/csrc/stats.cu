// Per-channel activation statistic and the K x C1 table of scale candidates.
//
// x_stat_c is the mean or the maximum of |X_nc| over the calibration tokens, or the maximum over
// the selected tokens (paper Sec. 3.1.2, second equation; Table 2 variants); candidate k is
// scale = x_stat^(k/K) (Sec. 3.1.2, first equation).  HBM-bound: X is read exactly once with
// 128-bit loads, 8 channels per thread; sums are carried in fp64 so that the bf16-rounded scale is
// reproducible bit for bit (sums of bf16 magnitudes are almost always exact in fp64, so the
// reduction order does not leak into the result).  Two stages, both with a fixed order: per-CTA
// column partials, then one thread per channel folds the partials and raises to the grid powers.
#include "common.cuh"

namespace tlq {

constexpr int kStatTx = 32;   // threads across channels (x8 channels each = 256 channels per CTA)
constexpr int kStatTy = 8;    // threads across rows

int64_t stats_row_chunks(int64_t N) {
  int64_t chunks = ceil_div(N, 256);      // 32 rows per thread: enough loads in flight, few enough CTAs to launch fast
  if (chunks > 256) chunks = 256;
  if (chunks < 1) chunks = 1;
  return chunks;
}

template <int kMode>
__global__ void __launch_bounds__(kStatTx * kStatTy)
channel_stats_kernel(const uint16_t* __restrict__ X, int64_t N, int64_t C1, const uint8_t* __restrict__ mask,
                     int64_t rows_per_chunk, double* __restrict__ partials) {
  __shared__ double red[kStatTy][kStatTx][8 + 1];
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int64_t c0 = ((int64_t)blockIdx.x * kStatTx + tx) * 8;
  const int64_t r_begin = (int64_t)blockIdx.y * rows_per_chunk;
  int64_t r_end = r_begin + rows_per_chunk;
  if (r_end > N) r_end = N;

  double acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.0;

  if (c0 < C1) {
    int64_t r = r_begin + ty;
    // four rows in flight per thread before any is consumed (a deselected row is loaded and then ignored)
    for (; r + 3 * kStatTy < r_end; r += 4 * kStatTy) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = ld_nc_16(X + (r + u * kStatTy) * C1 + c0);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (kMode == TLQ_STAT_MASKED_MAX && mask[r + u * kStatTy] == 0) continue;
        float f[8];
        unpack8(v[u], f);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          double a = (double)fabsf(f[j]);
          if (kMode == TLQ_STAT_MEAN_ABS) acc[j] += a; else acc[j] = fmax(acc[j], a);
        }
      }
    }
    for (; r < r_end; r += kStatTy) {
      if (kMode == TLQ_STAT_MASKED_MAX && mask[r] == 0) continue;
      float f[8];
      unpack8(ld_nc_16(X + r * C1 + c0), f);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        double a = (double)fabsf(f[j]);
        if (kMode == TLQ_STAT_MEAN_ABS) acc[j] += a; else acc[j] = fmax(acc[j], a);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) red[ty][tx][j] = acc[j];
  __syncthreads();
  if (ty == 0 && c0 < C1) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      double v = red[0][tx][j];
      for (int y = 1; y < kStatTy; ++y) {
        if (kMode == TLQ_STAT_MEAN_ABS) v += red[y][tx][j]; else v = fmax(v, red[y][tx][j]);
      }
      partials[(int64_t)blockIdx.y * C1 + c0 + j] = v;
    }
  }
}

// One rounding from binary64 to bfloat16 (nearest even), finite positive normal inputs.
__device__ __forceinline__ uint16_t double_to_bf16_bits(double x) {
  unsigned long long u = (unsigned long long)__double_as_longlong(x);
  const unsigned long long lsb = (u >> 45) & 1ull;
  u += ((1ull << 44) - 1ull) + lsb;
  const double r = __longlong_as_double((long long)((u >> 45) << 45));
  return (uint16_t)(__float_as_uint((float)r) >> 16);   // r is exactly representable in binary32
}

// One thread per (channel, candidate): every thread folds the channel's partials in the same fixed order
// (they sit in L2), then raises the statistic to its own grid power.
__global__ void scale_table_kernel(const double* __restrict__ partials, int64_t chunks, int64_t N, int64_t C1,
                                   int stat_mode, int K, double* __restrict__ x_stat, uint16_t* __restrict__ s,
                                   float* __restrict__ rs) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int k = blockIdx.y * blockDim.y + threadIdx.y;
  if (c >= C1 || k >= K) return;
  double v = partials[c];
  for (int64_t j = 1; j < chunks; ++j) {
    const double p = partials[j * C1 + c];
    if (stat_mode == TLQ_STAT_MEAN_ABS) v += p; else v = fmax(v, p);
  }
  if (stat_mode == TLQ_STAT_MEAN_ABS) v = v / (double)N;
  if (x_stat != nullptr && k == 0) x_stat[c] = v;
  const double m = fmax(v, kStatFloor);
  const double r = (double)k / (double)K;
  const uint16_t b = (k == 0) ? (uint16_t)0x3F80 : double_to_bf16_bits(pow(m, r));
  s[(int64_t)k * C1 + c] = b;
  if (rs) rs[(int64_t)k * C1 + c] = __fdiv_rn(1.0f, bf16_bits_to_float(b));
}

int launch_channel_stats(const uint16_t* X, int64_t N, int64_t C1, const uint8_t* mask, int stat_mode,
                         double* partials, cudaStream_t st) {
  const int64_t chunks = stats_row_chunks(N);
  const int64_t rows_per_chunk = ceil_div(N, chunks);
  dim3 grid((unsigned)ceil_div(C1, kStatTx * 8), (unsigned)chunks), block(kStatTx, kStatTy);
  switch (stat_mode) {
    case TLQ_STAT_MEAN_ABS:
      channel_stats_kernel<TLQ_STAT_MEAN_ABS><<<grid, block, 0, st>>>(X, N, C1, mask, rows_per_chunk, partials);
      break;
    case TLQ_STAT_MAX_ABS:
      channel_stats_kernel<TLQ_STAT_MAX_ABS><<<grid, block, 0, st>>>(X, N, C1, mask, rows_per_chunk, partials);
      break;
    default:
      channel_stats_kernel<TLQ_STAT_MASKED_MAX><<<grid, block, 0, st>>>(X, N, C1, mask, rows_per_chunk, partials);
      break;
  }
  return after_launch();
}

int launch_scale_table(const double* partials, int64_t chunks, int64_t N, int64_t C1, int stat_mode, int K,
                       double* x_stat, uint16_t* s, float* rs, cudaStream_t st) {
  const dim3 block(32, 8), grid((unsigned)ceil_div(C1, 32), (unsigned)ceil_div(K, 8));
  scale_table_kernel<<<grid, block, 0, st>>>(partials, chunks, N, C1, stat_mode, K, x_stat, s, rs);
  return after_launch();
}

// ------------------------------------------------------------------------------------------------
// Variant for callers that cannot allocate device memory: the per-chunk column partials live in a
// file-scope device array instead of a caller-provided workspace.  The array belongs to the loaded
// library image: every GPU that loads the library holds these 4 MiB until the process exits.
// ------------------------------------------------------------------------------------------------
constexpr int64_t kStaticScratchDoubles = 524288;     // 4 MiB of fp64 partials
constexpr int64_t kStaticMaxC1 = 32768;               // leaves room for at least 16 row chunks
static __device__ __align__(256) double g_static_partials[kStaticScratchDoubles];

int64_t static_stats_max_c1() { return kStaticMaxC1; }

// In host code `g_static_partials` is only a handle for the symbol, not a device address; the address a
// kernel can use is looked up once per device (with that device current) and cached here.
static double* static_partials_ptr(int* status) {
  constexpr int kMaxDevices = 64;
  static double* cached[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { *status = TLQ_ERR_CUDA; return nullptr; }
  if (cached[dev] == nullptr) {
    double* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      *status = TLQ_ERR_CUDA;
      return nullptr;
    }
    cached[dev] = p;
  }
  *status = TLQ_OK;
  return cached[dev];
}

int launch_scale_candidates_static(const uint16_t* X, int64_t N, int64_t C1, const uint8_t* mask, int stat_mode, int K,
                                   double* x_stat, uint16_t* s, cudaStream_t st) {
  int rc = TLQ_OK;
  double* partials = static_partials_ptr(&rc);
  if (rc != TLQ_OK) return rc;
  // as many row chunks as the regular path would use, capped by what the fixed array can hold
  int64_t chunks = stats_row_chunks(N);
  const int64_t cap = kStaticScratchDoubles / C1;
  if (chunks > cap) chunks = cap;
  const int64_t rows_per_chunk = ceil_div(N, chunks);
  chunks = ceil_div(N, rows_per_chunk);
  dim3 grid((unsigned)ceil_div(C1, kStatTx * 8), (unsigned)chunks), block(kStatTx, kStatTy);
  // every partial in [0, chunks) x [0, C1) is overwritten before the second stage reads it, so nothing
  // left behind by an earlier call can reach the result and nothing needs clearing
  switch (stat_mode) {
    case TLQ_STAT_MEAN_ABS:
      channel_stats_kernel<TLQ_STAT_MEAN_ABS><<<grid, block, 0, st>>>(X, N, C1, mask, rows_per_chunk, partials);
      break;
    case TLQ_STAT_MAX_ABS:
      channel_stats_kernel<TLQ_STAT_MAX_ABS><<<grid, block, 0, st>>>(X, N, C1, mask, rows_per_chunk, partials);
      break;
    default:
      channel_stats_kernel<TLQ_STAT_MASKED_MAX><<<grid, block, 0, st>>>(X, N, C1, mask, rows_per_chunk, partials);
      break;
  }
  if ((rc = after_launch()) != TLQ_OK) return rc;
  return launch_scale_table(partials, chunks, N, C1, stat_mode, K, x_stat, s, nullptr, st);
}

}  // namespace tlq
