// Final reduction of the search: loss[k] = sum_n w_n e_{k,n} / (C2 * sum_n w_n) (the expectation in
// the objective of paper Sec. 3.2.1 with per-token importance weights), argmin with the lowest index
// on ties, and the copy of the winning scale row.  Latency-bound: one CTA per candidate, fp64, fixed summation
// order (per-thread strided serial sums, then a binary tree in shared memory), so two runs give
// bit-identical losses.
#include "common.cuh"

namespace tlq {

constexpr int kRedThreads = 1024;

__device__ __forceinline__ double block_sum_fixed(double v, double* scratch) {
  const int t = threadIdx.x;
  __syncthreads();
  scratch[t] = v;
  __syncthreads();
  for (int half = kRedThreads / 2; half > 0; half >>= 1) {
    if (t < half) scratch[t] += scratch[t + half];
    __syncthreads();
  }
  return scratch[0];
}

// Refine set: the candidates whose screened loss is within `band` (relative) of the minimum, lowest loss first (equal
// losses: lower index first).  A set of one needs no second look.  A set larger than min(kMaxRefine, K/2) is not
// evaluated either: the screened result stands as a whole, so that losses[] never mixes first and second
// evaluations of candidates that close (the data is then flat to within the screening arithmetic: all scales
// equal, for instance).  Each member gets the delta-weight slot of a candidate outside the set for the low part of
// its split delta weights.
__device__ void refine_select(const double* losses /* a shared-memory copy */, int K, double band,
                              WorkspaceHeader* hdr) {      // one thread
  hdr->refine_count = 0;
  hdr->refine_done = 0;
  if (hdr->status != TLQ_OK || K < 2) return;
  const double lmin = losses[hdr->best_idx];
  if (!(lmin > 0.0) || !isfinite(lmin)) return;
  const double limit = lmin * (1.0 + band);
  const int cap = K / 2 < kMaxRefine ? K / 2 : kMaxRefine;
  int cand[kMaxRefine];
  int n = 0;
  for (int j = 0; j < K; ++j) {
    const double lj = losses[j];
    if (!(lj <= limit)) continue;
    if (n == cap) return;                       // too many to tell apart: keep the screened result
    int pos = n;                                // insertion by (loss, index); j ascends, so equal losses keep their order
    while (pos > 0 && losses[cand[pos - 1]] > lj) { cand[pos] = cand[pos - 1]; --pos; }
    cand[pos] = j;
    ++n;
  }
  if (n < 2) return;
  int slot = 0;
  for (int r = 0; r < n; ++r) {
    bool used = true;
    while (used) {            // next candidate index that is not in the set (K >= 2n: there is one)
      used = false;
      for (int q = 0; q < n; ++q) used = used || cand[q] == slot;
      if (used) ++slot;
    }
    hdr->refine_cand[r] = cand[r];
    hdr->refine_slot[r] = slot++;
  }
  hdr->refine_count = n;
}

// One CTA per candidate; the CTA that finishes last takes the argmin and copies the winning scale row.
__global__ void __launch_bounds__(kRedThreads)
loss_reduce_kernel(const float* __restrict__ partials, int64_t per_k, int K, const float* __restrict__ w_imp,
                   int64_t N, int64_t C2, const uint16_t* __restrict__ s_table, int64_t C1, WorkspaceHeader* hdr,
                   double* __restrict__ losses, int32_t* __restrict__ best_idx, uint16_t* __restrict__ s_best,
                   double refine_band) {
  __shared__ double scratch[kRedThreads];
  __shared__ int best_sh;
  __shared__ int last_sh;
  const int t = threadIdx.x;
  const int k = blockIdx.x;

  double wsum;
  if (w_imp != nullptr) {
    double a = 0.0;
    for (int64_t n = t; n < N; n += kRedThreads) a += (double)w_imp[n];
    wsum = block_sum_fixed(a, scratch);
  } else {
    wsum = (double)N;
  }
  const double denom = (double)C2 * wsum;

  const float* p = partials + (int64_t)k * per_k;
  double a = 0.0;
  for (int64_t i = t; i < per_k; i += kRedThreads) a += (double)p[i];
  const double total = block_sum_fixed(a, scratch);
  if (t == 0) {
    double l = total / denom;
    if (!isfinite(l)) l = __longlong_as_double(0x7FF0000000000000LL);
    losses[k] = l;
    __threadfence();
    last_sh = (atomicAdd(&hdr->reduce_done, 1) == K - 1) ? 1 : 0;
  }
  __syncthreads();
  if (last_sh == 0) return;

  __threadfence();
  if (t < K) scratch[t] = __ldcg(losses + t);      // written by other CTAs: read past L1 (K <= TLQ_MAX_GRID)
  __syncthreads();
  if (t == 0) {
    int best = -1;
    double bv = __longlong_as_double(0x7FF0000000000000LL);
    for (int j = 0; j < K; ++j) {
      const double lj = scratch[j];
      if (lj < bv) { bv = lj; best = j; }
    }
    if (best < 0) {
      if (hdr->status == TLQ_OK) hdr->status = TLQ_ERR_NONFINITE;
      best = 0;
    }
    best_sh = best;
    hdr->best_idx = best;
    hdr->denom = denom;
    *best_idx = best;
    if (refine_band > 0.0) refine_select(scratch, K, refine_band, hdr);
  }
  __syncthreads();
  if (s_best != nullptr) {
    const uint16_t* row = s_table + (int64_t)best_sh * C1;
    for (int64_t c = t; c < C1; c += kRedThreads) s_best[c] = row[c];
  }
}

// One CTA per refined candidate: fixed-order fp64 sum of its partials; the CTA that finishes last takes the argmin
// over the refined candidates (equal losses: lowest candidate index) and copies the winning scale row.
__global__ void __launch_bounds__(kRedThreads)
refine_finish_kernel(const double* __restrict__ partials, int64_t per_r, const uint16_t* __restrict__ s_table,
                     int64_t C1, WorkspaceHeader* hdr, double* __restrict__ losses, int32_t* __restrict__ best_idx,
                     uint16_t* __restrict__ s_best) {
  __shared__ double scratch[kRedThreads];
  __shared__ int best_sh;
  __shared__ int last_sh;
  const int t = threadIdx.x;
  const int r = blockIdx.x;
  const int n = hdr->refine_count;
  if (r >= n || hdr->status != TLQ_OK) return;
  const double* p = partials + (int64_t)r * per_r;
  double a = 0.0;
  for (int64_t i = t; i < per_r; i += kRedThreads) a += p[i];
  const double total = block_sum_fixed(a, scratch);
  if (t == 0) {
    double l = total / hdr->denom;
    if (!isfinite(l)) l = __longlong_as_double(0x7FF0000000000000LL);
    losses[hdr->refine_cand[r]] = l;
    __threadfence();
    last_sh = (atomicAdd(&hdr->refine_done, 1) == n - 1) ? 1 : 0;
  }
  __syncthreads();
  if (last_sh == 0) return;
  if (t == 0) {
    __threadfence();
    int best = -1;
    double bv = __longlong_as_double(0x7FF0000000000000LL);
    for (int q = 0; q < n; ++q) {
      const int j = hdr->refine_cand[q];
      const double lj = __ldcg(losses + j);
      if (lj < bv || (lj == bv && j < best)) { bv = lj; best = j; }
    }
    if (best < 0) best = hdr->best_idx;      // every refined loss non-finite: keep the screened choice
    best_sh = best;
    hdr->best_idx = best;
    *best_idx = best;
  }
  __syncthreads();
  if (s_best != nullptr) {
    const uint16_t* row = s_table + (int64_t)best_sh * C1;
    for (int64_t c = t; c < C1; c += kRedThreads) s_best[c] = row[c];
  }
}

__global__ void per_token_reduce_kernel(const float* __restrict__ ptab, int K, int64_t otiles, int64_t n_pad,
                                        int64_t N, float* __restrict__ per_token) {
  const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int k = blockIdx.y;
  if (n >= N) return;
  double a = 0.0;
  for (int64_t o = 0; o < otiles; ++o) a += (double)ptab[((int64_t)k * otiles + o) * n_pad + n];
  per_token[(int64_t)k * N + n] = (float)a;
}

int launch_loss_reduce(const float* partials, int64_t per_k, int K, const float* w_imp, int64_t N, int64_t C2,
                       const uint16_t* s_table, int64_t C1, WorkspaceHeader* hdr, double* losses, int32_t* best_idx,
                       uint16_t* s_best, double refine_band, cudaStream_t st) {
  loss_reduce_kernel<<<(unsigned)K, kRedThreads, 0, st>>>(partials, per_k, K, w_imp, N, C2, s_table, C1, hdr, losses, best_idx,
                                               s_best, refine_band);
  return after_launch();
}

int launch_refine_finish(const double* partials, int64_t per_r, const uint16_t* s_table, int64_t C1,
                         WorkspaceHeader* hdr, double* losses, int32_t* best_idx, uint16_t* s_best, cudaStream_t st) {
  refine_finish_kernel<<<kMaxRefine, kRedThreads, 0, st>>>(partials, per_r, s_table, C1, hdr, losses, best_idx, s_best);
  return after_launch();
}

int launch_per_token_reduce(const float* ptab, int K, int64_t otiles, int64_t n_pad, int64_t N, float* per_token,
                            cudaStream_t st) {
  dim3 grid((unsigned)ceil_div(N, 256), (unsigned)K);
  per_token_reduce_kernel<<<grid, 256, 0, st>>>(ptab, K, otiles, n_pad, N, per_token);
  return after_launch();
}

}  // namespace tlq
