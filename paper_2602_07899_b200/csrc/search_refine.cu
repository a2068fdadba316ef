// Refine pass of the group-mode search: a second, more exact evaluation of the few candidates whose screened losses
// are too close to call (objective of paper Sec. 3.2.1; the argmin of its last equation must not depend on how the
// error is accumulated).
//
// The screening GEMM deviates from the exact per-token error in two ways: the delta weights are rounded to bf16
// (2^-9 relative per element, random sign: it averages out over a loss), and every output element is accumulated
// over all of C1 inside the tensor core, whose fp32 accumulator drops the bits below its unit in the last place at
// every instruction (a systematic pull towards zero that grows with C1: 2e-5 to 6e-5 of the loss at 3584..29568
// channels).  This kernel removes both for the candidates listed in the workspace header:
//   * delta weights enter as two bf16 operands, hi = bf16(d) (the screening operand, still in place) and
//     lo = bf16(d - hi) (written by the residual mode of the group fake-quant kernel): products with the bf16
//     activations are exact, what is left out is 2^-18 |d|;
//   * the hi products are accumulated in the tensor core over chunks of kChunkKb k-blocks only (16 instructions),
//     each chunk is added to per-thread fp32 sums in registers with round-to-nearest (unbiased), and the lo
//     products, 2^-9 as large, get an accumulator of their own over the whole row;
//   * squares, token weighting and all sums from there on are fp64.
// Tile 128 tokens x 128 output channels (one fp32 register per output channel and thread), otherwise the structure
// of the screening kernels: one persistent CTA per SM, a TMA producer warp, an MMA warp, four epilogue warps, all
// waits bounded.  Reads the candidate list from device memory, so it is launched unconditionally and returns at once
// when the list is empty.
#include "common.cuh"
#include "umma.cuh"

namespace tlq {

bool encode_tensor_map(CUtensorMap* out, CUtensorMapDataType dtype, int rank, const void* base, const uint64_t* dims,
                       const uint64_t* strides_bytes, const uint32_t* box);

namespace {

constexpr int BM = 128;
constexpr int BN = 128;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kThreads = 192;
constexpr int kChunkKb = 4;              // k-blocks (of 64 channels) per tensor-core accumulation chunk
constexpr uint32_t kABytes = BM * BK * 2;
constexpr uint32_t kBBytes = BN * BK * 2;
constexpr uint32_t kStageBytes = kABytes + 2 * kBBytes;      // X tile, hi tile, lo tile
constexpr uint32_t kTmemCols = 512;      // columns 0..255: two chunk accumulators, 256..383: the lo accumulator
constexpr uint32_t kLoCol = 2 * BN;
constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kStages * kStageBytes + 256 /*barriers*/;
constexpr uint32_t kIdesc = ptx::make_idesc(1, 1, BM, BN, false);

struct RefineArgs {
  int64_t N;
  int num_kb;              // ceil(C1 / 64)
  int64_t mtiles, otiles;
  TileRaster raster;       // walk order inside one candidate (whole token range, or 2048-token blocks)
  const int32_t* n_live;   // device: live token count after compaction, or null (= N)
  const float* w_imp;      // [N] or null (uniform)
  double* partials;        // [kMaxRefine][otiles*mtiles*4]
  WorkspaceHeader* hdr;
};

__device__ __forceinline__ void report_timeout(WorkspaceHeader* hdr, int where) {
  hdr->where = where;
  hdr->status = TLQ_ERR_TIMEOUT;
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_refine_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const RefineArgs args) {
  const int n_refine = args.hdr->refine_count;      // written by the selection kernel before this launch
  if (n_refine <= 0 || args.hdr->status != TLQ_OK) return;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto hfull_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto hempty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  const uint32_t lfull_bar = bar_base + 8u * (2 * kStages + 4);
  const uint32_t lempty_bar = bar_base + 8u * (2 * kStages + 5);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + kStages * kStageBytes + 8 * (2 * kStages + 6));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(hfull_bar(a), 1);
      ptx::mbar_init(hempty_bar(a), 4);
    }
    ptx::mbar_init(lfull_bar, 1);
    ptx::mbar_init(lempty_bar, 4);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
  }
  if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), kTmemCols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int num_kb = args.num_kb;
  const int num_chunks = (num_kb + kChunkKb - 1) / kChunkKb;
  const int64_t n_tokens = args.n_live != nullptr ? (int64_t)*args.n_live : args.N;
  const int64_t mt_live = (n_tokens + BM - 1) / BM;          // token tiles that hold tokens
  const int64_t tiles_per_r = args.otiles * mt_live;
  const int64_t num_tiles = (int64_t)n_refine * tiles_per_r;
  // tile -> (entry of the refine set, then the screening kernels' walk inside the candidate: token tiles fastest
  // while the activations fit in L2, blocks of 2048 tokens x 9 output tiles when they do not)
  TileRaster raster = args.raster;
  raster.mtiles = (int)mt_live;
  if (raster.b == 1) raster.a = mt_live > 0 ? (int)mt_live : 1;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int r = (int)(tile / tiles_per_r);
        const int64_t rem = tile - (int64_t)r * tiles_per_r;
        int mt, ot;
        raster.decode(rem, mt, ot);
        const int k_hi = args.hdr->refine_cand[r], k_lo = args.hdr->refine_slot[r];
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
            report_timeout(args.hdr, 51);
            ok = false;
            break;
          }
          const uint32_t a_dst = smem_base + stage * kStageBytes;
          ptx::mbar_expect_tx(full_bar(stage), kStageBytes);
          ptx::tma_load_2d(a_dst, &tmA, full_bar(stage), kb * BK, mt * BM);
          ptx::tma_load_3d(a_dst + kABytes, &tmB, full_bar(stage), kb * BK, ot * BN, k_hi);
          ptx::tma_load_3d(a_dst + kABytes + kBBytes, &tmB, full_bar(stage), kb * BK, ot * BN, k_lo);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int64_t it = 0, cc = 0;       // tiles and chunks handled so far by this CTA
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
        if (!ptx::mbar_wait(lempty_bar, (uint32_t)(it & 1) ^ 1u, abort_flag)) {
          report_timeout(args.hdr, 52);
          break;
        }
        const uint32_t d_lo = tmem_base + kLoCol;
        uint32_t acc_lo = 0;
        for (int c = 0; c < num_chunks && ok; ++c, ++cc) {
          const int acc = (int)(cc & 1);
          if (!ptx::mbar_wait(hempty_bar(acc), (uint32_t)((cc >> 1) & 1) ^ 1u, abort_flag)) {
            report_timeout(args.hdr, 53);
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t d_hi = tmem_base + (uint32_t)acc * BN;
          uint32_t acc_hi = 0;
          const int kb_end = (c + 1) * kChunkKb < num_kb ? (c + 1) * kChunkKb : num_kb;
          for (int kb = c * kChunkKb; kb < kb_end; ++kb) {
            if (!ptx::mbar_wait(full_bar(stage), phase, abort_flag)) {
              report_timeout(args.hdr, 54);
              ok = false;
              break;
            }
            ptx::tc_fence_after();
            const uint32_t a_addr = smem_base + stage * kStageBytes;
            const uint64_t adesc = ptx::smem_desc_sw128(a_addr);
            const uint64_t hdesc = ptx::smem_desc_sw128(a_addr + kABytes);
            const uint64_t ldesc = ptx::smem_desc_sw128(a_addr + kABytes + kBBytes);
#pragma unroll
            for (int ks = 0; ks < BK / UMMA_K; ++ks) {
              ptx::mma_bf16_ss(d_hi, adesc + (uint64_t)(ks * 2), hdesc + (uint64_t)(ks * 2), kIdesc, acc_hi);
              ptx::mma_bf16_ss(d_lo, adesc + (uint64_t)(ks * 2), ldesc + (uint64_t)(ks * 2), kIdesc, acc_lo);
              acc_hi = 1;
              acc_lo = 1;
            }
            ptx::mma_commit(empty_bar(stage));
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) ptx::mma_commit(hfull_bar(acc));
        }
        if (ok) ptx::mma_commit(lfull_bar);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;                 // tensor-memory lanes [32*quarter, 32*quarter+32)
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
    int64_t it = 0, cc = 0;
    bool ok = true;
    for (int64_t tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int r = (int)(tile / tiles_per_r);
      const int64_t rem = tile - (int64_t)r * tiles_per_r;
      int mt, ot;
      raster.decode(rem, mt, ot);
      float sums[BN];
#pragma unroll
      for (int j = 0; j < BN; ++j) sums[j] = 0.0f;
      for (int c = 0; c < num_chunks; ++c, ++cc) {
        const int acc = (int)(cc & 1);
        if (!ptx::mbar_wait(hfull_bar(acc), (uint32_t)((cc >> 1) & 1), abort_flag)) {
          if (lane == 0) report_timeout(args.hdr, 55);
          ok = false;
          break;
        }
        ptx::tc_fence_after();
#pragma unroll
        for (int q = 0; q < BN / 16; ++q) {
          uint32_t v[16];
          ptx::tmem_ld16(lane_base + (uint32_t)acc * BN + q * 16, v);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) sums[q * 16 + j] = __fadd_rn(sums[q * 16 + j], __uint_as_float(v[j]));
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(hempty_bar(acc));
      }
      if (!ok) break;
      if (!ptx::mbar_wait(lfull_bar, (uint32_t)(it & 1), abort_flag)) {
        if (lane == 0) report_timeout(args.hdr, 56);
        break;
      }
      ptx::tc_fence_after();
      double e = 0.0;                              // sum over the tile's 128 output channels of E[n,o]^2
#pragma unroll
      for (int q = 0; q < BN / 8; ++q) {
        uint32_t v[8];
        ptx::tmem_ld8(lane_base + kLoCol + q * 8, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const double x = (double)sums[q * 8 + j] + (double)__uint_as_float(v[j]);
          e = fma(x, x, e);
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(lempty_bar);
      const int64_t n = (int64_t)mt * BM + row_in_tile;
      double wn = 0.0;
      if (n < n_tokens) wn = (args.w_imp != nullptr) ? (double)args.w_imp[n] : 1.0;
      double v = wn * e;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
      if (lane == 0)
        args.partials[((int64_t)r * args.otiles + ot) * args.mtiles * 4 + (int64_t)mt * 4 + quarter] = v;
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag != 0) {
    // a wait expired somewhere: give copies and MMAs in flight time to land before releasing memory
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

int64_t refine_partials_per_candidate(int64_t N, int64_t C2) { return ceil_div(C2, BN) * ceil_div(N, BM) * 4; }

int launch_search_gemm_refine(const uint16_t* X, const uint16_t* dW, const float* w_imp, int64_t N, int64_t C1,
                              int64_t C2, int K, double* partials, WorkspaceHeader* hdr, const int32_t* n_live,
                              cudaStream_t st) {
  CUtensorMap tmA, tmB;
  const uint64_t adims[2] = {(uint64_t)C1, (uint64_t)N};
  const uint64_t astr[1] = {(uint64_t)C1 * 2};
  const uint32_t abox[2] = {BK, BM};
  const uint64_t bdims[3] = {(uint64_t)C1, (uint64_t)C2, (uint64_t)K};
  const uint64_t bstr[2] = {(uint64_t)C1 * 2, (uint64_t)C1 * (uint64_t)C2 * 2};
  const uint32_t bbox[3] = {BK, BN, 1};
  if (!encode_tensor_map(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, adims, astr, abox) ||
      !encode_tensor_map(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, dW, bdims, bstr, bbox))
    return TLQ_ERR_CUDA;
  static OncePerDevice once;
  const int rc = once_per_device(once, [] {
    return cudaFuncSetAttribute(gemm_refine_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  });
  if (rc != TLQ_OK) return rc;
  RefineArgs a{};
  a.N = N;
  a.num_kb = (int)ceil_div(C1, BK);
  a.mtiles = ceil_div(N, BM);
  a.otiles = ceil_div(C2, BN);
  a.n_live = n_live;
  a.w_imp = w_imp;
  a.partials = partials;
  a.hdr = hdr;
  const int sms = device_sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  const int64_t max_tiles = (int64_t)kMaxRefine * a.mtiles * a.otiles;
  const unsigned grid = (unsigned)(max_tiles < sms ? max_tiles : sms);
  a.raster = make_raster(a.mtiles, a.otiles, sms, N * C1 * 2, BM);
  gemm_refine_kernel<<<grid, kThreads, kSmemBytes, st>>>(tmA, tmB, a);
  return after_launch();
}

}  // namespace tlq
