// The fused bf16 search GEMM on 256-token x 256-channel tiles per CTA.
//
// Same contraction and fused epilogue as search_gemm.cu (per-token squared output error of
// E_k = X dW_k^T, importance-weighted, paper Sec. 3.2.1 objective).  One CTA works on two 128-token
// halves against the SAME 256-row weight tile: per 64-wide k-block it stages 32 KB of X (one 256-row
// box) and 32 KB of dW and issues eight MMAs, four into each of the two 256-column accumulators in
// tensor memory.  Per unit of tensor work that is 32 KB staged instead of 48 KB (the weight tile is
// fetched once for both halves), a third less L2 -> shared-memory traffic, with no second SM involved.
// The price: both accumulators belong to the tile in flight, so the epilogue overlaps the next tile
// only half by half (the MMAs into a half wait until that half has been drained).
//
// Roles (192 threads): warp 0 TMA producer (3 stages of 64 KB), warp 1 tensor-memory owner and MMA
// issuer, warps 2..5 epilogue (each owns a quarter of the 128 lanes, first of half 0, then of half 1).
// Barriers: full[s] / empty[s] per stage, tfull (both accumulators complete), tempty[h] per half
// (four epilogue warps).  Every wait is bounded.
#include "common.cuh"
#include "l2part.cuh"
#include "umma.cuh"

namespace tlq {

namespace {

constexpr int BM = 128;                  // rows of one half
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int kStages = 3;
constexpr int kThreads = 192;
constexpr uint32_t kABytes = 2 * BM * BK * 2;      // 32 KB: both halves, one box
constexpr uint32_t kBBytes = BN * BK * 2;          // 32 KB
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kTmemCols = 512;
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 256;
constexpr uint32_t kIdesc = ptx::make_idesc(1, 1, BM, BN, false);

struct WideArgs {
  int64_t N, C2;
  int num_kb;
  int K;
  int64_t mtiles;          // 128-row token tiles (layout of the partial buffer)
  int64_t mpairs;          // 256-row token tiles
  int64_t otiles;
  int64_t n_pad;
  bool blocked;            // walk by blocks of `block_a` token tiles (activations too large to stay in L2)
  int block_a;
  const L2PartMap* l2map;  // which L2 partition each SM sits next to (may be null or not yet measured)
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

__global__ void __launch_bounds__(kThreads, 1)
gemm_bf16_wide_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const WideArgs args) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  const uint32_t tfull_bar = bar_base + 8u * (2 * kStages);
  auto tempty_bar = [&](int h) { return bar_base + 8u * (2 * kStages + 1 + h); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + kStages * kStageBytes + 8 * (2 * kStages + 3));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  TileWalk* walk_sh = reinterpret_cast<TileWalk*>(smem_gen + kStages * kStageBytes + 128);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  int64_t n_tokens = args.N, mpairs = args.mpairs;
  if (args.n_live != nullptr) {
    n_tokens = *args.n_live;
    mpairs = (n_tokens + 2 * BM - 1) / (2 * BM);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(tfull_bar, 1);
    ptx::mbar_init(tempty_bar(0), 4);
    ptx::mbar_init(tempty_bar(1), 4);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    // this CTA's share of the tiles: its L2 partition's token tiles when the partitions are known
    make_tile_walk(args.l2map, args.hdr, (int)mpairs, (int)args.otiles, args.K, args.blocked, args.block_a, *walk_sh);
  }
  if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), kTmemCols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const TileWalk walk = *walk_sh;
  const int num_kb = args.num_kb;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int k = 0;
      for (int64_t tile = walk.first; tile < walk.count && ok; tile += walk.stride) {
        int mp, ot;
        walk.decode(tile, k, mp, ot);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
            report_timeout(args.hdr, 31);
            ok = false;
            break;
          }
          const uint32_t a_dst = smem_base + stage * kStageBytes;
          ptx::mbar_expect_tx(full_bar(stage), kStageBytes);
          ptx::tma_load_2d(a_dst, &tmA, full_bar(stage), kb * BK, mp * 2 * BM);
          ptx::tma_load_3d(a_dst + kABytes, &tmB, full_bar(stage), kb * BK, ot * BN, k);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int64_t it = 0;
      bool ok = true;
      for (int64_t tile = walk.first; tile < walk.count && ok; tile += walk.stride, ++it) {
        const uint32_t drained_phase = (uint32_t)(it & 1) ^ 1u;     // halves were drained once per earlier tile
        for (int kb = 0; kb < num_kb && ok; ++kb) {
          if (!ptx::mbar_wait(full_bar(stage), phase, abort_flag)) {
            report_timeout(args.hdr, 33);
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t a_addr = smem_base + stage * kStageBytes;
          const uint64_t bdesc = ptx::smem_desc_sw128(a_addr + kABytes);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            if (kb == 0) {      // the first write into a half needs the epilogue of the previous tile out of it
              if (!ptx::mbar_wait(tempty_bar(h), drained_phase, abort_flag)) {
                report_timeout(args.hdr, 32);
                ok = false;
                break;
              }
              ptx::tc_fence_after();
            }
            const uint64_t adesc = ptx::smem_desc_sw128(a_addr + (uint32_t)h * (BM * BK * 2));
            const uint32_t d_tmem = tmem_base + (uint32_t)h * BN;
#pragma unroll
            for (int ks = 0; ks < BK / UMMA_K; ++ks)
              ptx::mma_bf16_ss(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), kIdesc,
                               (kb > 0 || ks > 0) ? 1u : 0u);
          }
          if (!ok) break;
          ptx::mma_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) ptx::mma_commit(tfull_bar);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;
    const int row_in_half = quarter * 32 + lane;
    int64_t it = 0;
    int k = 0;
    for (int64_t tile = walk.first; tile < walk.count; tile += walk.stride, ++it) {
      int mp, ot;
      walk.decode(tile, k, mp, ot);
      if (!ptx::mbar_wait(tfull_bar, (uint32_t)(it & 1), abort_flag)) {
        if (lane == 0) report_timeout(args.hdr, 34);
        break;
      }
      ptx::tc_fence_after();
#pragma unroll 1
      for (int h = 0; h < 2; ++h) {
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)h * BN;
        const int64_t mt = (int64_t)mp * 2 + h;
        const int64_t n = mt * BM + row_in_half;
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
        if (lane == 0) ptx::mbar_arrive(tempty_bar(h));     // this half may be overwritten by the next tile
        const float e = (s0 + s1) + (s2 + s3);
        // a half past the last token has nothing to add (after compaction its rows may be stale memory)
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
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag != 0) {
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

int wide_sm_count() { return device_sm_count(); }

}  // namespace

int launch_search_gemm_bf16_wide(const uint16_t* X, const uint16_t* dW, const float* w_imp, const GemmPlan& plan,
                                 float* partials, float* ptab, WorkspaceHeader* hdr, const int32_t* n_live,
                                 const L2PartMap* l2map, cudaStream_t st) {
  static OncePerDevice once;
  const int rc_cfg = once_per_device(once, [] {
    return cudaFuncSetAttribute(gemm_bf16_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  });
  if (rc_cfg != TLQ_OK) return rc_cfg;
  CUtensorMap tmA, tmB;
  const uint64_t adims[2] = {(uint64_t)plan.C1, (uint64_t)plan.N};
  const uint64_t astr[1] = {(uint64_t)plan.C1 * 2};
  const uint32_t abox[2] = {BK, 2 * BM};
  const uint64_t bdims[3] = {(uint64_t)plan.C1, (uint64_t)plan.C2, (uint64_t)plan.K};
  const uint64_t bstr[2] = {(uint64_t)plan.C1 * 2, (uint64_t)plan.C1 * (uint64_t)plan.C2 * 2};
  const uint32_t bbox[3] = {BK, BN, 1};
  if (!encode_tensor_map(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, adims, astr, abox) ||
      !encode_tensor_map(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, dW, bdims, bstr, bbox))
    return TLQ_ERR_CUDA;
  const int sms = wide_sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  WideArgs a{};
  a.N = plan.N; a.C2 = plan.C2;
  a.num_kb = (int)ceil_div(plan.C1, BK);
  a.K = plan.K;
  a.mtiles = plan.mtiles;
  a.mpairs = ceil_div(plan.N, 2 * BM);
  a.otiles = plan.otiles;
  a.n_pad = plan.n_pad;
  const TileRaster shape = make_raster(a.mpairs, a.otiles, sms, plan.N * plan.C1 * 2, 2 * BM);
  a.blocked = shape.b != 1;
  a.block_a = 2048 / (2 * BM);
  a.w_imp = w_imp; a.partials = partials; a.ptab = ptab; a.hdr = hdr; a.n_live = n_live;
  const int64_t tiles = (int64_t)plan.K * a.otiles * a.mpairs;
  const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
  // The partition-aware walk needs one CTA on every SM and enough tiles for the split to balance.  It is for
  // activations that can stay in L2 (measured on the 7B-class layer: HBM bytes of the q / k / gate launches about 1690 /
  // 340 / 10460 MB -> 576 / 133 / 2813 MB, i.e. the operands once); where they cannot, splitting the tokens only shortens the weight block a
  // wave shares (18944-channel down-projection: 24.5 -> 45 GB), so the blocked walk stays whole.
  a.l2map = (grid == (unsigned)sms && tiles >= 8 * (int64_t)sms && !a.blocked) ? l2map : nullptr;
  gemm_bf16_wide_kernel<<<grid, kThreads, kSmemBytes, st>>>(tmA, tmB, a);
  return after_launch();
}

}  // namespace tlq
