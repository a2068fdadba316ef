// Token compaction for importance weights that contain zeros.
//
// The paper forms its token-level calibration set by keeping the half of the tokens with the largest
// gradient importance (Sec. 3.1.2, I = Top50%); as a weight vector that is w_n in {0, 1}.  A token
// with w_n = 0 adds nothing to any candidate's loss, so the quantized layer need not be applied to
// it at all: the live rows of X are packed to the front (original order kept), the GEMM runs over
// ceil(n_live / 128) token tiles, and with the paper's mask the search does half the tensor work.
// The count stays on the device (no host synchronisation): later kernels read it from memory.
#include "common.cuh"

namespace tlq {

constexpr int kScanThreads = 1024;

// One CTA walks the N weights in chunks of 1024 and assigns output slots in token order.
// live[0] = number of live tokens, live[1] = that number rounded up to a multiple of 128.
__global__ void __launch_bounds__(kScanThreads)
compact_index_kernel(const float* __restrict__ w_imp, int64_t N, int32_t* __restrict__ idx, float* __restrict__ wc,
                     int32_t* __restrict__ live) {
  __shared__ int warp_count[kScanThreads / 32];
  __shared__ int base_sh;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  if (t == 0) base_sh = 0;
  __syncthreads();
  for (int64_t n0 = 0; n0 < N; n0 += kScanThreads) {
    const int64_t n = n0 + t;
    const float w = (n < N) ? w_imp[n] : 0.0f;
    const bool keep = w > 0.0f;                       // NaN and negative weights are dropped as well
    const unsigned ballot = __ballot_sync(0xFFFFFFFFu, keep);
    if (lane == 0) warp_count[warp] = __popc(ballot);
    __syncthreads();
    int before = base_sh;
    for (int i = 0; i < warp; ++i) before += warp_count[i];
    if (keep) {
      const int slot = before + __popc(ballot & ((1u << lane) - 1u));
      idx[slot] = (int32_t)n;
      wc[slot] = w;
    }
    __syncthreads();
    if (t == 0) {
      int total = 0;
      for (int i = 0; i < kScanThreads / 32; ++i) total += warp_count[i];
      base_sh += total;
    }
    __syncthreads();
  }
  const int n_live = base_sh;
  const int padded = (n_live + 127) / 128 * 128;
  for (int j = n_live + t; j < padded; j += kScanThreads) wc[j] = 0.0f;   // rows of the last tile (wc holds n_pad)
  if (t == 0) { live[0] = n_live; live[1] = padded; }
}

// One CTA per output row: copy the live row, zero-fill the rest of the last 128-row tile (so that a
// stale row can never put a NaN into a sum that is then multiplied by a zero weight).
__global__ void __launch_bounds__(128)
gather_rows_kernel(const uint16_t* __restrict__ X, const int32_t* __restrict__ idx, const int32_t* __restrict__ live,
                   int64_t C1, uint16_t* __restrict__ Xc) {
  const int64_t j = blockIdx.x;
  const int n_live = live[0], padded = live[1];
  if (j >= padded) return;
  uint4* dst = reinterpret_cast<uint4*>(Xc + j * C1);
  const int64_t packets = C1 / 8;
  if (j < n_live) {
    const uint16_t* src = X + (int64_t)idx[j] * C1;
    for (int64_t i = threadIdx.x; i < packets; i += 128) dst[i] = ld_nc_16(src + i * 8);
  } else {
    for (int64_t i = threadIdx.x; i < packets; i += 128) dst[i] = make_uint4(0, 0, 0, 0);
  }
}

// idx [N], wc [n_pad], live [2], Xc [n_pad, C1] with n_pad = N rounded up to a multiple of 128.
int launch_compact_tokens(const uint16_t* X, const float* w_imp, int64_t N, int64_t n_pad, int64_t C1, int32_t* idx,
                          float* wc, int32_t* live, uint16_t* Xc, cudaStream_t st) {
  compact_index_kernel<<<1, kScanThreads, 0, st>>>(w_imp, N, idx, wc, live);
  int rc = after_launch();
  if (rc != TLQ_OK) return rc;
  gather_rows_kernel<<<(unsigned)n_pad, 128, 0, st>>>(X, idx, live, C1, Xc);
  return after_launch();
}

}  // namespace tlq
