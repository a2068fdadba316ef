// The fused bf16 search GEMM on CTA pairs (tcgen05 cta_group::2).
//
// Same contraction and the same fused epilogue as search_gemm.cu (per-token squared output error of
// E_k = X dW_k^T, importance-weighted, paper Sec. 3.2.1 objective), but two CTAs of a cluster work on
// one 256-token x 256-channel tile: each holds 128 token rows of X, HALF of the 256 dW rows and its
// own 128 x 256 fp32 accumulator; the even CTA issues one 256 x 256 x 16 MMA for both.  Per unit of
// tensor work a CTA now stages 32 KB instead of 48 KB (the weight tile is split, not duplicated), so
// the same shared memory holds six stages instead of four and the traffic L2 -> SM drops by a third.
// No multicast loads: every CTA fetches its own tiles; completion bytes of both CTAs are counted on
// the even CTA's barrier.
//
// Roles per CTA (192 threads): warp 0 TMA producer, warp 1 tensor-memory owner (and MMA issuer in the
// even CTA), warps 2..5 epilogue.  Barriers: full[s] (even CTA, 1 arrival + 64 KB), empty[s] (each
// CTA, released by the MMA commit multicast), tfull[a] (each CTA, commit multicast), tempty[a] (even
// CTA, 8 arrivals: four epilogue warps of each CTA).  Every wait is bounded.
#include "common.cuh"
#include "umma.cuh"

namespace tlq {

namespace {

constexpr int BM = 128;                  // token rows per CTA (256 per pair)
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int kStages = 6;
constexpr int kThreads = 192;
constexpr uint32_t kABytes = BM * BK * 2;          // 16 KB
constexpr uint32_t kBBytes = (BN / 2) * BK * 2;    // 16 KB: this CTA's half of the weight tile
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kTmemCols = 512;
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 256;
constexpr uint32_t kIdescPair = ptx::make_idesc(1, 1, 2 * BM, BN, false);

struct PairArgs {
  int64_t N, C2;
  int num_kb;
  int K;
  int64_t mtiles;          // 128-row token tiles (layout of the partial buffer)
  int64_t mpairs;          // 256-row token tiles
  int64_t otiles;
  int64_t n_pad;
  TileRaster raster;       // over (mpairs, otiles)
  const float* w_imp;
  float* partials;         // [K][otiles*mtiles*4]
  float* ptab;             // [K][otiles][n_pad] or null
  WorkspaceHeader* hdr;
  const int32_t* n_live;   // device: live token count after compaction, or null
};

__device__ __forceinline__ void report_timeout(WorkspaceHeader* hdr, int where) {
  hdr->where = where;
  hdr->status = TLQ_ERR_TIMEOUT;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const PairArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + kStages * kStageBytes + 8 * (2 * kStages + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();       // 0 = the CTA that issues the MMAs
  const int64_t pair = blockIdx.x >> 1;
  const int64_t npairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), 8);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
  }
  if (warp == 1) ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), kTmemCols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();          // both CTAs' barriers exist before anything is signalled across
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int num_kb = args.num_kb;
  int64_t n_tokens = args.N, mpairs = args.mpairs;
  TileRaster raster = args.raster;
  if (args.n_live != nullptr) {
    n_tokens = *args.n_live;
    mpairs = (n_tokens + 2 * BM - 1) / (2 * BM);
    raster.mtiles = (int)mpairs;
    if (raster.b == 1) raster.a = mpairs > 0 ? (int)mpairs : 1;
  }
  const int64_t tiles_per_k = args.otiles * mpairs;
  const int64_t num_tiles = (int64_t)args.K * tiles_per_k;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int64_t tile = pair; tile < num_tiles && ok; tile += npairs) {
        const int k = (int)(tile / tiles_per_k);
        int mp, ot;
        raster.decode(tile - (int64_t)k * tiles_per_k, mp, ot);
        const int row_a = (mp * 2 + (int)rank) * BM;
        const int row_b = ot * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
            report_timeout(args.hdr, 21);
            ok = false;
            break;
          }
          const uint32_t a_dst = smem_base + stage * kStageBytes;
          const uint32_t bar = ptx::map_to_cta(full_bar(stage), 0);
          if (rank == 0) ptx::mbar_expect_tx(full_bar(stage), 2 * kStageBytes);
          ptx::tma_load_2d_pair(a_dst, &tmA, bar, kb * BK, row_a);
          ptx::tma_load_3d_pair(a_dst + kABytes, &tmB, bar, kb * BK, row_b, k);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA only)
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int64_t it = 0;
      bool ok = true;
      for (int64_t tile = pair; tile < num_tiles && ok; tile += npairs, ++it) {
        const int acc = (int)(it & 1);
        const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
        if (!ptx::mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) {
          report_timeout(args.hdr, 22);
          break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        uint32_t accumulate = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait(full_bar(stage), phase, abort_flag)) {
            report_timeout(args.hdr, 23);
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t a_addr = smem_base + stage * kStageBytes;
          const uint64_t adesc = ptx::smem_desc_sw128(a_addr);
          const uint64_t bdesc = ptx::smem_desc_sw128(a_addr + kABytes);
#pragma unroll
          for (int ks = 0; ks < BK / UMMA_K; ++ks) {
            ptx::mma_bf16_ss_pair(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), kIdescPair, accumulate);
            accumulate = 1;
          }
          ptx::mma_commit_pair(empty_bar(stage), 3);      // frees the stage in both CTAs
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) ptx::mma_commit_pair(tfull_bar(acc), 3);  // accumulators of both CTAs are complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    int64_t it = 0;
    for (int64_t tile = pair; tile < num_tiles; tile += npairs, ++it) {
      const int k = (int)(tile / tiles_per_k);
      int mp, ot;
      raster.decode(tile - (int64_t)k * tiles_per_k, mp, ot);
      const int64_t mt = (int64_t)mp * 2 + rank;          // this CTA's 128-row token tile
      const int acc = (int)(it & 1);
      const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
      if (!ptx::mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) {
        if (lane == 0) report_timeout(args.hdr, 24);
        break;
      }
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN;
      const int64_t n = mt * BM + row_in_tile;
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        ptx::tmem_ld32(taddr + c * 32, r);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float v0 = __uint_as_float(r[j]), v1 = __uint_as_float(r[j + 1]);
          const float v2 = __uint_as_float(r[j + 2]), v3 = __uint_as_float(r[j + 3]);
          s0 = fmaf(v0, v0, s0); s1 = fmaf(v1, v1, s1); s2 = fmaf(v2, v2, s2); s3 = fmaf(v3, v3, s3);
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(tempty_bar(acc), 0));
      const float e = (s0 + s1) + (s2 + s3);
      // an odd count of 128-row tiles leaves the second CTA of the last pair without tokens: it has nothing to add
      // (after compaction its rows may even be stale memory, which must not reach a sum)
      if (mt < args.mtiles && mt * BM < n_tokens) {
        if (args.ptab != nullptr) args.ptab[((int64_t)k * args.otiles + ot) * args.n_pad + n] = e;
        float wn = 0.0f;
        if (n < n_tokens) wn = (args.w_imp != nullptr) ? args.w_imp[n] : 1.0f;
        float v = wn * e;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
        if (lane == 0)
          args.partials[((int64_t)k * args.otiles + ot) * args.mtiles * 4 + mt * 4 + quarter] = v;
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag != 0) {
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();          // neither CTA leaves while the other may still read its memory or barriers
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

int max_pairs() {
  static int pairs_of[kMaxDevices];
  static bool known[kMaxDevices] = {};
  const int dev = current_device_index();
  if (dev < 0) return 0;
  int& pairs = pairs_of[dev];
  if (!known[dev]) {
    if (cudaFuncSetAttribute(gemm_bf16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) !=
        cudaSuccess)
      return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_bf16_pair_kernel, &cfg) != cudaSuccess) {
      cudaGetLastError();
      return 0;
    }
    pairs = n;
    known[dev] = true;
  }
  return pairs;
}

}  // namespace

// How many CTA pairs the device can keep resident at once (0: pairs cannot be launched here).
int search_gemm_pair_capacity() { return max_pairs(); }

int launch_search_gemm_bf16_pair(const uint16_t* X, const uint16_t* dW, const float* w_imp, const GemmPlan& plan,
                                 float* partials, float* ptab, WorkspaceHeader* hdr, const int32_t* n_live,
                                 cudaStream_t st) {
  const int cap = max_pairs();
  if (cap <= 0) return TLQ_ERR_CUDA;
  CUtensorMap tmA, tmB;
  const uint64_t adims[2] = {(uint64_t)plan.C1, (uint64_t)plan.N};
  const uint64_t astr[1] = {(uint64_t)plan.C1 * 2};
  const uint32_t abox[2] = {BK, BM};
  const uint64_t bdims[3] = {(uint64_t)plan.C1, (uint64_t)plan.C2, (uint64_t)plan.K};
  const uint64_t bstr[2] = {(uint64_t)plan.C1 * 2, (uint64_t)plan.C1 * (uint64_t)plan.C2 * 2};
  const uint32_t bbox[3] = {BK, BN / 2, 1};
  if (!encode_tensor_map(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, adims, astr, abox) ||
      !encode_tensor_map(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, dW, bdims, bstr, bbox))
    return TLQ_ERR_CUDA;
  PairArgs a{};
  a.N = plan.N; a.C2 = plan.C2;
  a.num_kb = (int)ceil_div(plan.C1, BK);
  a.K = plan.K;
  a.mtiles = plan.mtiles;
  a.mpairs = ceil_div(plan.N, 2 * BM);
  a.otiles = plan.otiles;
  a.n_pad = plan.n_pad;
  a.raster = make_raster(a.mpairs, a.otiles, cap, plan.N * plan.C1 * 2, 2 * BM);
  a.w_imp = w_imp; a.partials = partials; a.ptab = ptab; a.hdr = hdr; a.n_live = n_live;
  const int64_t pair_tiles = (int64_t)plan.K * a.otiles * a.mpairs;
  const unsigned pairs = (unsigned)(pair_tiles < cap ? pair_tiles : cap);
  gemm_bf16_pair_kernel<<<2 * pairs, kThreads, kSmemBytes, st>>>(tmA, tmB, a);
  return after_launch();
}

}  // namespace tlq
