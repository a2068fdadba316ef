// The fused search GEMM for 16-bit activations (W4A16 and other weight widths with Q_a = identity).
//
// With unquantized activations f_fp(x) - f_q(x; scale_k) = (W - W_hat_k) x (paper Sec. 3.2.1, f_fp and
// f_q with Q_a = id; W_hat_k = dequant(Q_w(W*scale_k)) / scale_k by the smoothing identity of
// Sec. 2.2), so the per-token squared output error of candidate k is the squared row norm of
// E_k = X dW_k^T.  All K candidates are one batched GEMM  [N x C1] x [K*C2 x C1]^T  on the 5th-gen
// tensor cores; the epilogue never stores E: each epilogue thread owns one token row of the fp32
// accumulator in tensor memory, squares and adds its 256 columns, multiplies by the token's
// importance weight and the four epilogue warps emit one partial each per tile.
//
// Structure (one persistent CTA per SM, 192 threads):
//   warp 0      TMA producer: 128x64 X tile + 256x64 dW tile per stage (128-byte swizzle), 4 stages
//   warp 1      tensor-memory owner and tcgen05.mma issuer (128x256x16 per instruction, fp32 accumulate),
//               two 256-column accumulators so the epilogue of tile i overlaps the main loop of tile i+1
//   warps 2..5  epilogue: tcgen05.ld 32 columns at a time, sum of squares, weighting, partial store
// The same main loop serves tlq_apply_layer: two passes over K (W, then dW with the negate-B bit)
// accumulate X W^T - X dW^T = X W_hat^T, and the epilogue stores bf16 (+bias).
#include "common.cuh"
#include "umma.cuh"

namespace tlq {

namespace {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;                   // 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kThreads = 192;
constexpr uint32_t kABytes = BM * BK * 2;
constexpr uint32_t kBBytes = BN * BK * 2;
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kTmemCols = 512;      // two 256-column fp32 accumulators
constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kStages * kStageBytes + 256 /*barriers*/;

constexpr uint32_t kIdesc = ptx::make_idesc(1, 1, BM, BN, false);
constexpr uint32_t kIdescNegB = ptx::make_idesc(1, 1, BM, BN, true);

struct GemmArgs {
  int64_t N, C2;
  int num_kb;              // ceil(C1 / 64)
  int64_t mtiles, otiles;
  int64_t num_tiles;       // K * otiles * mtiles
  int64_t tiles_per_k;     // otiles * mtiles
  TileRaster raster;       // walk order inside one candidate
  const int32_t* n_live;   // device: live token count after compaction, or null (= N)
  int64_t n_pad;
  const float* w_imp;      // [N] or null (uniform)
  float* partials;         // [K][otiles*mtiles*4]
  float* ptab;             // [K][otiles][n_pad] or null
  const uint16_t* bias;    // apply: [C2] or null
  uint16_t* yq;            // apply: [N,C2]
  WorkspaceHeader* hdr;
};

__device__ __forceinline__ void report_timeout(WorkspaceHeader* hdr, int where) {
  hdr->where = where;
  hdr->status = TLQ_ERR_TIMEOUT;
}

template <bool kApply>
__global__ void __launch_bounds__(kThreads, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmB2, const GemmArgs args) {
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

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), 4);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    if (kApply) ptx::prefetch_tensormap(&tmB2);
  }
  if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), kTmemCols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int passes = kApply ? 2 : 1;
  const int num_kb = args.num_kb;
  // token count and tile walk: fixed by the host, or read from the device when the tokens were compacted
  int64_t n_tokens = args.N, tiles_per_k = args.tiles_per_k, num_tiles = args.num_tiles;
  TileRaster raster = args.raster;
  if (args.n_live != nullptr) {
    n_tokens = *args.n_live;
    const int64_t mt_live = (n_tokens + BM - 1) / BM;
    raster.mtiles = (int)mt_live;
    if (raster.b == 1) raster.a = mt_live > 0 ? (int)mt_live : 1;
    tiles_per_k = args.otiles * mt_live;
    num_tiles = (args.num_tiles / args.tiles_per_k) * tiles_per_k;
  }

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int k = (int)(tile / tiles_per_k);
        int mt, ot;
        raster.decode(tile - (int64_t)k * tiles_per_k, mt, ot);
        for (int pass = 0; pass < passes && ok; ++pass) {
          const CUtensorMap* tb = (kApply && pass == 1) ? &tmB2 : &tmB;
          for (int kb = 0; kb < num_kb; ++kb) {
            if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
              report_timeout(args.hdr, 1);
              ok = false;
              break;
            }
            const uint32_t a_dst = smem_base + stage * kStageBytes;
            ptx::mbar_expect_tx(full_bar(stage), kStageBytes);
            ptx::tma_load_2d(a_dst, &tmA, full_bar(stage), kb * BK, mt * BM);
            ptx::tma_load_3d(a_dst + kABytes, tb, full_bar(stage), kb * BK, ot * BN, k);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
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
      for (int64_t tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = (int)(it & 1);
        const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
        if (!ptx::mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) {
          report_timeout(args.hdr, 2);
          break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        uint32_t accumulate = 0;
        for (int pass = 0; pass < passes && ok; ++pass) {
          const uint32_t idesc = (kApply && pass == 1) ? kIdescNegB : kIdesc;
          for (int kb = 0; kb < num_kb; ++kb) {
            if (!ptx::mbar_wait(full_bar(stage), phase, abort_flag)) {
              report_timeout(args.hdr, 3);
              ok = false;
              break;
            }
            ptx::tc_fence_after();
            const uint32_t a_addr = smem_base + stage * kStageBytes;
            const uint64_t adesc = ptx::smem_desc_sw128(a_addr);
            const uint64_t bdesc = ptx::smem_desc_sw128(a_addr + kABytes);
#pragma unroll
            for (int ks = 0; ks < BK / UMMA_K; ++ks) {
              // +32 bytes along K per step: the start-address field counts 16-byte units
              ptx::mma_bf16_ss(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, accumulate);
              accumulate = 1;
            }
            ptx::mma_commit(empty_bar(stage));
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
        if (ok) ptx::mma_commit(tfull_bar(acc));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;                 // tensor-memory lanes [32*quarter, 32*quarter+32)
    const int row_in_tile = quarter * 32 + lane;
    int64_t it = 0;
    for (int64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
      const int k = (int)(tile / tiles_per_k);
      int mt, ot;
      raster.decode(tile - (int64_t)k * tiles_per_k, mt, ot);
      const int acc = (int)(it & 1);
      const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
      if (!ptx::mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) {
        if (lane == 0) report_timeout(args.hdr, 4);
        break;
      }
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN;
      const int64_t n = (int64_t)mt * BM + row_in_tile;
      if (!kApply) {
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
        if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
        const float e = (s0 + s1) + (s2 + s3);      // sum_o E[n,o]^2 over this tile's 256 output channels
        if (args.ptab != nullptr) args.ptab[((int64_t)k * args.otiles + ot) * args.n_pad + n] = e;
        float wn = 0.0f;
        if (n < n_tokens) wn = (args.w_imp != nullptr) ? args.w_imp[n] : 1.0f;
        float v = wn * e;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
        if (lane == 0)
          args.partials[((int64_t)k * args.otiles + ot) * args.mtiles * 4 + mt * 4 + quarter] = v;
      } else {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          ptx::tmem_ld32(taddr + c * 32, r);
          ptx::tmem_ld_wait();
          const int64_t col0 = (int64_t)ot * BN + c * 32;
          if (n < n_tokens) {
#pragma unroll
            for (int p = 0; p < 4; ++p) {
              const int64_t col = col0 + p * 8;
              if (col < args.C2) {
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  float v = __uint_as_float(r[p * 8 + j]);
                  if (args.bias != nullptr) v += bf16_bits_to_float(args.bias[col + j]);
                  const uint32_t b = float_to_bf16_bits(v);
                  if (j & 1) o[j >> 1] |= b << 16; else o[j >> 1] = b;
                }
                *reinterpret_cast<uint4*>(args.yq + n * args.C2 + col) = make_uint4(o[0], o[1], o[2], o[3]);
              }
            }
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
      }
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

int num_sms() { return device_sm_count(); }

template <bool kApply>
int configure_kernel() {
  static OncePerDevice once;
  return once_per_device(once, [] {
    return cudaFuncSetAttribute(gemm_bf16_kernel<kApply>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  });
}

}  // namespace

bool encode_tensor_map(CUtensorMap* out, CUtensorMapDataType dtype, int rank, const void* base, const uint64_t* dims,
                       const uint64_t* strides_bytes, const uint32_t* box) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || p == nullptr)
      return false;
    fn = reinterpret_cast<EncodeFn>(p);
  }
  cuuint64_t gdim[5], gstr[5];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
  return fn(out, dtype, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

GemmPlan plan_search_gemm(int64_t N, int64_t C1, int64_t C2, int K) {
  GemmPlan p;
  p.N = N; p.C1 = C1; p.C2 = C2; p.K = K;
  p.mtiles = ceil_div(N, BM);
  p.otiles = ceil_div(C2, BN);
  p.partials_per_k = p.mtiles * p.otiles * 4;
  p.n_pad = p.mtiles * BM;
  return p;
}

static bool make_maps_bf16(const uint16_t* X, int64_t N, int64_t C1, const uint16_t* B, int64_t C2, int K,
                           CUtensorMap* tmA, CUtensorMap* tmB) {
  const uint64_t adims[2] = {(uint64_t)C1, (uint64_t)N};
  const uint64_t astr[1] = {(uint64_t)C1 * 2};
  const uint32_t abox[2] = {BK, BM};
  const uint64_t bdims[3] = {(uint64_t)C1, (uint64_t)C2, (uint64_t)K};
  const uint64_t bstr[2] = {(uint64_t)C1 * 2, (uint64_t)C1 * (uint64_t)C2 * 2};
  const uint32_t bbox[3] = {BK, BN, 1};
  return encode_tensor_map(tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, adims, astr, abox) &&
         encode_tensor_map(tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, B, bdims, bstr, bbox);
}

int launch_search_gemm_bf16(const uint16_t* X, const uint16_t* dW, const float* w_imp, const GemmPlan& plan,
                            float* partials, float* ptab, WorkspaceHeader* hdr, const int32_t* n_live, cudaStream_t st) {
  CUtensorMap tmA, tmB;
  if (!make_maps_bf16(X, plan.N, plan.C1, dW, plan.C2, plan.K, &tmA, &tmB)) return TLQ_ERR_CUDA;
  int rc = configure_kernel<false>();
  if (rc != TLQ_OK) return rc;
  GemmArgs a{};
  a.N = plan.N; a.C2 = plan.C2;
  a.num_kb = (int)ceil_div(plan.C1, BK);
  a.mtiles = plan.mtiles; a.otiles = plan.otiles;
  a.tiles_per_k = plan.otiles * plan.mtiles;
  a.num_tiles = (int64_t)plan.K * a.tiles_per_k;
  a.n_pad = plan.n_pad;
  a.w_imp = w_imp; a.partials = partials; a.ptab = ptab; a.bias = nullptr; a.yq = nullptr; a.hdr = hdr;
  a.n_live = n_live;
  const int sms = num_sms();
  if (sms <= 0) return TLQ_ERR_CUDA;
  const unsigned grid = (unsigned)(a.num_tiles < sms ? a.num_tiles : sms);
  a.raster = make_raster(plan.mtiles, plan.otiles, sms, plan.N * plan.C1 * 2, BM);
  gemm_bf16_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(tmA, tmB, tmB, a);
  return after_launch();
}

int launch_apply_gemm_bf16(const uint16_t* X, const uint16_t* W, const uint16_t* dW, const uint16_t* bias, int64_t N,
                           int64_t C1, int64_t C2, uint16_t* Yq, WorkspaceHeader* hdr, cudaStream_t st) {
  CUtensorMap tmA, tmW, tmD;
  if (!make_maps_bf16(X, N, C1, W, C2, 1, &tmA, &tmW)) return TLQ_ERR_CUDA;
  if (!make_maps_bf16(X, N, C1, dW, C2, 1, &tmA, &tmD)) return TLQ_ERR_CUDA;
  int rc = configure_kernel<true>();
  if (rc != TLQ_OK) return rc;
  GemmPlan plan = plan_search_gemm(N, C1, C2, 1);
  GemmArgs a{};
  a.N = N; a.C2 = C2;
  a.num_kb = (int)ceil_div(C1, BK);
  a.mtiles = plan.mtiles; a.otiles = plan.otiles;
  a.tiles_per_k = plan.otiles * plan.mtiles;
  a.num_tiles = a.tiles_per_k;
  a.n_pad = plan.n_pad;
  a.w_imp = nullptr; a.partials = nullptr; a.ptab = nullptr; a.bias = bias; a.yq = Yq; a.hdr = hdr;
  const int sms = num_sms();
  if (sms <= 0) return TLQ_ERR_CUDA;
  const unsigned grid = (unsigned)(a.num_tiles < sms ? a.num_tiles : sms);
  a.raster = make_raster(plan.mtiles, plan.otiles, sms, plan.N * plan.C1 * 2, BM);
  gemm_bf16_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(tmA, tmW, tmD, a);
  return after_launch();
}

}  // namespace tlq
