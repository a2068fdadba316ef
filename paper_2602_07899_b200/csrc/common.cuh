// Shared declarations of the libtlq kernels (device helpers, launch bookkeeping, stage launchers).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <math.h>
#include <stdint.h>

#include "tlq.h"

namespace tlq {

// ---------------------------------------------------------------------------------------------
// Host-side bookkeeping
// ---------------------------------------------------------------------------------------------
extern long long g_launch_count;  // kernels launched since load

#define TLQ_CUDA_TRY(expr)                         \
  do {                                             \
    cudaError_t e__ = (expr);                      \
    if (e__ != cudaSuccess) return TLQ_ERR_CUDA;   \
  } while (0)

inline int after_launch() {
  ++g_launch_count;
  return cudaGetLastError() == cudaSuccess ? TLQ_OK : TLQ_ERR_CUDA;
}

// Host-side state that belongs to a device (kernel attributes, SM counts) is kept per device index: one process
// may drive several GPUs, each call acting on the device that is current when it is made.
constexpr int kMaxDevices = 64;
inline int current_device_index() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}
int device_sm_count();   // multiprocessors of the current device (looked up once per device); 0 on error
struct OncePerDevice {
  bool done[kMaxDevices] = {};
};
// Runs `configure` (returning a cudaError_t) the first time it is reached with a given device current.
template <typename F>
inline int once_per_device(OncePerDevice& state, F configure) {
  const int dev = current_device_index();
  if (dev < 0) return TLQ_ERR_CUDA;
  if (!state.done[dev]) {
    if (configure() != cudaSuccess) {
      cudaGetLastError();
      return TLQ_ERR_CUDA;
    }
    state.done[dev] = true;
  }
  return TLQ_OK;
}

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Floors on degenerate statistics (a dead channel, a flat group, a zero row).
constexpr double kStatFloor = 9.5367431640625e-07;  // 2^-20
#define TLQ_RANGE_FLOOR 1e-5f

// ---------------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

// float -> bf16 bits, round to nearest even (finite inputs).
__device__ __forceinline__ uint32_t float_to_bf16_bits(float f) {
  uint32_t u = __float_as_uint(f);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return u >> 16;
}

// Unpack 8 bf16 values held in a uint4 (little-endian pairs).
__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
  f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
  f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}

__device__ __forceinline__ uint4 ld_nc_16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// ---------------------------------------------------------------------------------------------
// Walk order of the (token tile, output tile) grid of one GEMM.  The persistent CTAs take tiles
// round-robin from one linear order, so the tiles in flight at any moment are a run of consecutive
// indices.  With a = mtiles the order is "all token tiles of one output tile, then the next output
// tile": a run touches every activation tile and two or three weight tiles, which reads the weights
// from HBM once as long as the activations stay in L2.  When they cannot (the wide down-projection),
// a run is made a block of `a` token tiles x `b` output tiles instead, blocks advancing along the
// tokens first: the run then needs a activation tiles and b weight tiles, and measured HBM traffic
// of the 18944-channel case drops by a quarter.  (Measured the other way round for activations that do
// fit, where the blocked walk re-reads weight tiles: hence the switch.)
// ---------------------------------------------------------------------------------------------
struct TileRaster {
  int mtiles, otiles, a, b;
  __host__ __device__ void decode(int64_t t, int& mt, int& ot) const {
    const int64_t band_tiles = (int64_t)mtiles * b;
    const int oband = (int)(t / band_tiles);
    const int b_eff = (otiles - oband * b) < b ? (otiles - oband * b) : b;
    int64_t r = t - (int64_t)oband * band_tiles;
    const int mgroup = (int)(r / ((int64_t)a * b_eff));
    const int a_eff = (mtiles - mgroup * a) < a ? (mtiles - mgroup * a) : a;
    r -= (int64_t)mgroup * a * b_eff;
    ot = oband * b + (int)(r / a_eff);
    mt = mgroup * a + (int)(r % a_eff);
  }
};
// `act_bytes`: bytes of the activation operand one candidate streams (bf16 X, or one candidate's int8 codes);
// `tile_tokens`: token rows of one tile (128, or 256 for the wide kernel and the CTA pairs).
// The block is 2048 tokens high: measured on the 72B-class shapes (16384 x 8192 activations, 256-token tiles),
// 8 token tiles x 18 output tiles per wave moved 26-35 % fewer HBM bytes than 16 x 9 and ran 5-15 % faster
// (4, 6, 12 and 32 token tiles per block all measured worse); the weight block (18 tiles of 256 rows) is what stays
// in L2 from wave to wave while the activations stream past it.
inline TileRaster make_raster(int64_t mtiles, int64_t otiles, int grid, int64_t act_bytes, int tile_tokens) {
  TileRaster r;
  r.mtiles = (int)mtiles; r.otiles = (int)otiles;
  if (act_bytes <= (64ll << 20)) {      // fits in half of L2 with room for the weight stream
    r.a = (int)mtiles; r.b = 1;
  } else {
    r.a = 2048 / tile_tokens;
    r.b = grid / r.a > 0 ? grid / r.a : 1;
  }
  return r;
}

// ---------------------------------------------------------------------------------------------
// Work items of the tile-resident kernel (one CTA keeps an output tile for all of its candidates)
// ---------------------------------------------------------------------------------------------
// What one CTA does next.  Whole waves of tiles run all K candidates per tile; the tiles left over for the last,
// partial wave are split by candidates over the CTAs that would otherwise idle (each split recomputes the
// candidate-free tile, two pass-equivalents, against up to K passes saved): with 896 tiles on 148 SMs the seventh
// wave of 8 tiles costs 3 pass-times instead of 22.
struct TailSplit {
  int full;        // tiles handled whole (a multiple of the grid size)
  int chunks;      // candidate chunks per left-over tile
  int per;         // candidates per chunk
  int items;       // left-over tiles x chunks (<= grid size)
};
__host__ __device__ inline TailSplit make_tail_split(int num_tiles, int grid, int K) {
  TailSplit t;
  t.full = (num_tiles / grid) * grid;
  const int rest = num_tiles - t.full;
  int splits = rest > 0 ? grid / rest : 1;
  if (splits > K) splits = K;
  if (splits < 1) splits = 1;
  t.per = (K + splits - 1) / splits;
  t.chunks = (K + t.per - 1) / t.per;
  t.items = rest * t.chunks;
  return t;
}
// Work item number w of this launch -> (tile, candidates [k0, k1)); false when there is none.
__host__ __device__ inline bool work_item(const TailSplit& t, int w, int K, int& tile, int& k0, int& k1) {
  if (w < t.full) { tile = w; k0 = 0; k1 = K; return true; }
  const int j = w - t.full;
  if (j >= t.items) return false;
  tile = t.full + j / t.chunks;
  k0 = (j % t.chunks) * t.per;
  k1 = k0 + t.per < K ? k0 + t.per : K;
  return true;
}

// ---------------------------------------------------------------------------------------------
// Workspace header (first 256 bytes of every workspace)
// ---------------------------------------------------------------------------------------------
constexpr int kMaxRefine = 4;            // candidates the refine pass re-evaluates at most
struct WorkspaceHeader {
  int32_t status;     // TLQ_OK / TLQ_ERR_TIMEOUT / TLQ_ERR_NONFINITE
  int32_t where;      // diagnostic: which wait gave up
  int32_t best_idx;   // device copy of the argmin
  int32_t reduce_done; // CTAs of the loss reduction that have finished (the header is zeroed by every call)
  int32_t selftest;    // set by the bounded-wait self-test when its abort flag reached the other lanes
  int32_t slot_count[2]; // tile-walk slots claimed so far in each L2 partition by the CTAs of the search GEMM
  // refine pass (reduce.cu, search_refine.cu): the candidates whose screened losses lie within the band of the
  // minimum, lowest loss first, and for each the slot of the delta-weight buffer (a candidate outside the list, whose
  // delta weights are no longer needed) that receives the low part of its split delta weights
  int32_t refine_count;
  int32_t refine_cand[kMaxRefine];
  int32_t refine_slot[kMaxRefine];
  int32_t refine_done;   // CTAs of the refine reduction that have finished
  int32_t pad0;
  double denom;          // C2 * sum of the token weights: what the weighted partial sums are divided by
  int32_t pad[44];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header is 256 bytes");

// ---------------------------------------------------------------------------------------------
// Stage launchers (each enqueues on `st`, returns TLQ_OK or TLQ_ERR_CUDA)
// ---------------------------------------------------------------------------------------------

// stats.cu
int64_t stats_row_chunks(int64_t N);
int launch_channel_stats(const uint16_t* X, int64_t N, int64_t C1, const uint8_t* mask, int stat_mode,
                         double* partials /*[chunks,C1]*/, cudaStream_t st);
int launch_scale_table(const double* partials, int64_t chunks, int64_t N, int64_t C1, int stat_mode, int K,
                       double* x_stat /*[C1] or null*/, uint16_t* s /*[K,C1]*/, float* rs /*[K,C1] or null*/,
                       cudaStream_t st);

int64_t static_stats_max_c1();
int launch_scale_candidates_static(const uint16_t* X, int64_t N, int64_t C1, const uint8_t* mask, int stat_mode, int K,
                                   double* x_stat /*[C1] or null*/, uint16_t* s /*[K,C1]*/, cudaStream_t st);

// fakequant.cu
int launch_fakequant_group(const uint16_t* W, const uint16_t* s /*[K,C1] or null*/, const float* rs /*[K,C1] or null: 1/s*/,
                           int K, int64_t C2, int64_t C1,
                           int group, int w_bits, uint16_t* dW /*[K,C2,C1] or null*/, uint8_t* codes, float* steps,
                           int32_t* zeros, cudaStream_t st);
// symmetric `bits`-wide codes (2..8) in int8 containers
int launch_fakequant_rows_i8(const uint16_t* W, const uint16_t* s /*[K,C1] or null*/, int K, int64_t C2, int64_t C1,
                             int bits, int8_t* q /*[K,C2,C1]*/, float* u /*[K,C2]*/, cudaStream_t st);
// activations: x * (1/s); give the reciprocal table rs [K,C1], or a bf16 scale s [K,C1] to invert on the fly, or neither
// n_rows_dev: optional device int32 holding how many leading rows are live (the rest are skipped)
int launch_actquant_i8(const uint16_t* X, const uint16_t* s, const float* rs, int K, int64_t N, int64_t C1, int bits,
                       int8_t* q /*[K,N,C1]*/, float* t /*[K,N]*/, const int32_t* n_rows_dev, cudaStream_t st);

// compact.cu: pack the rows of X whose weight is > 0 to the front (order kept); live[0] = count, live[1] = count
// rounded up to 128.  idx [N], wc [n_pad], Xc [n_pad, C1].
int launch_compact_tokens(const uint16_t* X, const float* w_imp, int64_t N, int64_t n_pad, int64_t C1, int32_t* idx,
                          float* wc, int32_t* live, uint16_t* Xc, cudaStream_t st);

// 4-bit codes, two per byte (even channel in the low nibble); n_codes a multiple of 32
int launch_pack_codes4(const uint8_t* codes, int64_t n_codes, uint8_t* packed, cudaStream_t st);

// importance.cu
int launch_token_importance(const void* G, int g_dtype, int64_t B, int64_t N, int64_t C, int norm_kind,
                            float* imp, cudaStream_t st);
int launch_top_mask(const float* imp, int64_t N, int64_t k_sel, uint8_t* mask, cudaStream_t st);

// reduce.cu
int launch_loss_reduce(const float* partials, int64_t per_k, int K, const float* w_imp, int64_t N, int64_t C2,
                       const uint16_t* s_table, int64_t C1, WorkspaceHeader* hdr, double* losses, int32_t* best_idx,
                       uint16_t* s_best, double refine_band /* > 0: also fill hdr's refine set with the candidates
                       within this relative distance of the minimum: 2 .. min(kMaxRefine, K/2) of them, or none */,
                       cudaStream_t st);
int launch_per_token_reduce(const float* ptab /*[K,otiles,Npad]*/, int K, int64_t otiles, int64_t Npad, int64_t N,
                            float* per_token /*[K,N]*/, cudaStream_t st);

// Refine pass of the group-mode search (16-bit activations).  The screening GEMM sees delta weights rounded to bf16
// and accumulates each output over all of C1 in the tensor core's fp32 accumulator.  The accumulation pulls a loss
// down by up to 6e-5 relative (C1 up to 29568).  The rounding of a delta weight is shared by every token, so it
// averages out over the C2 output channels only: about 2 * 2^-9 / sqrt(3 * C2) of the loss when one input channel
// dominates (2.3e-4 measured at C2 = 72, at most 6e-5 in total at C2 >= 256 on 7B/72B-class layers).  Candidates
// closer to the minimum than refine_band(C2) are evaluated again with split delta weights (bf16 high + bf16 low
// part) and short accumulation chunks summed outside the tensor core, and the argmin is taken on those values.
inline double refine_band(int64_t C2) {
  const double by_rows = 3.2e-3 / sqrt((double)C2);      // 1e-4 from 1024 output channels on, 2e-4 at 256
  return by_rows > 1.0e-4 ? by_rows : 1.0e-4;
}
// reduce.cu: refined losses from the fp64 partials [kMaxRefine][per_r]; rewrites losses[k] of the refined
// candidates, the argmin and the winning scale row
int launch_refine_finish(const double* partials, int64_t per_r, const uint16_t* s_table, int64_t C1,
                         WorkspaceHeader* hdr, double* losses, int32_t* best_idx, uint16_t* s_best, cudaStream_t st);
// fakequant.cu: for each refined candidate r, bf16(dW - bf16(dW)) of candidate hdr->refine_cand[r] into slot
// hdr->refine_slot[r] of dW [K,C2,C1]
int launch_fakequant_group_residual(const uint16_t* W, const uint16_t* s, const float* rs, int64_t C2, int64_t C1,
                                    int group, int w_bits, uint16_t* dW, const WorkspaceHeader* hdr, cudaStream_t st);
// search_refine.cu: partials [kMaxRefine][refine_partials_per_candidate] (fp64; zeroed by the caller when n_live is
// given, since token tiles without live tokens are not written)
int64_t refine_partials_per_candidate(int64_t N, int64_t C2);
int launch_search_gemm_refine(const uint16_t* X, const uint16_t* dW, const float* w_imp, int64_t N, int64_t C1,
                              int64_t C2, int K, double* partials, WorkspaceHeader* hdr, const int32_t* n_live,
                              cudaStream_t st);

// selftest.cu: guard words between the regions of a workspace (TLQ_FLAG_DEBUG_CANARIES).  fill writes a pattern that
// depends on the guard's index and the word's position; check compares and, on the first difference it sees, sets
// hdr->status = TLQ_ERR_OVERRUN and hdr->where = 100 + index of the guard (unless an earlier error is recorded).
constexpr int kMaxGuards = 32;
constexpr size_t kGuardBytes = 256;
struct GuardList {
  int n;
  unsigned long long off[kMaxGuards];      // byte offset of each guard from the start of the workspace
};
int launch_canary_fill(void* workspace, const GuardList& guards, cudaStream_t st);
int launch_canary_check(const void* workspace, const GuardList& guards, WorkspaceHeader* hdr, cudaStream_t st);

// selftest.cu: one warp waits `limit_cycles` on a barrier nobody arrives on, then reports TLQ_ERR_TIMEOUT in `hdr`
int launch_bounded_wait_selftest(WorkspaceHeader* hdr, long long limit_cycles, cudaStream_t st);

// search_gemm.cu
struct GemmPlan {
  int64_t N, C1, C2;
  int K;
  int64_t mtiles, otiles;   // tiles along tokens / output channels
  int64_t partials_per_k;   // floats per candidate in the partial buffer
  int64_t n_pad;            // mtiles * 128
};
GemmPlan plan_search_gemm(int64_t N, int64_t C1, int64_t C2, int K);
// W4A16 search: partials[K][mtiles*otiles*4] (+ ptab[K][otiles][n_pad] if non-null)
// n_live: optional device int32: only the first *n_live rows of X are tokens (the partial buffer must be zeroed)
int launch_search_gemm_bf16(const uint16_t* X, const uint16_t* dW, const float* w_imp, const GemmPlan& plan,
                            float* partials, float* ptab, WorkspaceHeader* hdr, const int32_t* n_live, cudaStream_t st);
// search_gemm_pair.cu: the same search on CTA pairs (cta_group::2), same partial / per-token layout
int search_gemm_pair_capacity();
int launch_search_gemm_bf16_pair(const uint16_t* X, const uint16_t* dW, const float* w_imp, const GemmPlan& plan,
                                 float* partials, float* ptab, WorkspaceHeader* hdr, const int32_t* n_live,
                                 cudaStream_t st);
// search_gemm_wide.cu: the same search on 256-token x 256-channel tiles per CTA (weight tile shared by two halves);
// l2map: the device's SM -> L2 partition table (l2part.cuh) or null
struct L2PartMap;
int launch_search_gemm_bf16_wide(const uint16_t* X, const uint16_t* dW, const float* w_imp, const GemmPlan& plan,
                                 float* partials, float* ptab, WorkspaceHeader* hdr, const int32_t* n_live,
                                 const L2PartMap* l2map, cudaStream_t st);
// Apply: Yq[N,C2] = X W^T - X dW^T (+bias), bf16 out
int launch_apply_gemm_bf16(const uint16_t* X, const uint16_t* W, const uint16_t* dW, const uint16_t* bias,
                           int64_t N, int64_t C1, int64_t C2, uint16_t* Yq, WorkspaceHeader* hdr, cudaStream_t st);

// search_gemm_i8.cu
GemmPlan plan_search_gemm_i8(int64_t N, int64_t C1, int64_t C2, int K);   // partials_per_k = mtiles*otiles*8
// W8A8 search: partials[K][mtiles*otiles*8] (+ ptab[K][otiles*2][n_pad] if non-null)
int launch_search_gemm_i8(const uint16_t* X, const uint16_t* W, const int8_t* Xq, const int8_t* Wq, const float* t,
                          const float* u, const float* w_imp, const GemmPlan& plan, float* partials, float* ptab,
                          WorkspaceHeader* hdr, const int32_t* n_live, cudaStream_t st);
// Two-stream search with 16-bit activations (reference from Xfp, quantized side from Xq); plan = plan_search_gemm_i8
int launch_search_gemm_dual_bf16(const uint16_t* Xq, const uint16_t* Xfp, const uint16_t* W, const uint16_t* dW,
                                 const float* w_imp, const GemmPlan& plan, float* partials, float* ptab,
                                 WorkspaceHeader* hdr, cudaStream_t st);
// Apply: Yq[N,C2] = t[n] * u[o] * (Xq Wq^T) (+bias), bf16 out
int launch_apply_gemm_i8(const int8_t* Xq, const int8_t* Wq, const float* t, const float* u, const uint16_t* bias,
                         int64_t N, int64_t C1, int64_t C2, uint16_t* Yq, WorkspaceHeader* hdr, cudaStream_t st);

}  // namespace tlq
