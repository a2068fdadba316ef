// The fused search GEMM for the W8A8 setting: int8 weights per output channel, int8 activations per
// token, both symmetric (paper Sec. 2.2 quantizer; Sec. 3.2.1 f_q = Q_w(W*scale) Q_a(x/scale)).
//
// With quantized activations the output error is no longer linear in a weight difference, so each
// candidate needs the integer product itself:
//     E_k[n,o] = (X W^T)[n,o] - t_k[n] * u_k[o] * (Xq_k Wq_k^T)[n,o].
// One CTA owns a 128-token x 256-channel output tile for ALL candidates: pass 0 accumulates the
// full-precision tile X W^T with bf16 tcgen05.mma (fp32 in tensor memory) and the epilogue threads
// pull their share of it into registers, where it stays; passes 1..K run the int8 tcgen05.mma
// (kind::i8, int32 accumulators) for one candidate each, and the epilogue forms the difference, the
// per-token sum of squares and the importance-weighted partial without the quantized output ever
// leaving the SM.  Two 256-column accumulators alternate, so the epilogue of one pass overlaps the
// main loop of the next.
//
// Structure (one persistent CTA per SM, 320 threads):
//   warp 0      TMA producer (4 stages of 16 KB + 32 KB, 128-byte swizzle; bf16 k-blocks are 64 wide,
//               int8 k-blocks 128 wide, both 128 bytes per row)
//   warp 1      tensor-memory owner and MMA issuer
//   warps 2..9  epilogue: two warps per tensor-memory lane quarter, 128 columns each
// The same kernel serves tlq_apply_layer for W8A8 (a single int8 pass, bf16 store of t*u*acc + bias).
#include "common.cuh"
#include "umma.cuh"

namespace tlq {

namespace {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK16 = 64;                 // bf16 elements per k-block (128 bytes)
constexpr int BK8 = 128;                 // int8 elements per k-block (128 bytes)
constexpr int kStages = 4;
constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;
constexpr uint32_t kABytes = BM * 128;
constexpr uint32_t kBBytes = BN * 128;
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kTmemCols = 512;
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 256;

constexpr uint32_t kIdescBf16 = ptx::make_idesc(1, 1, BM, BN, false);   // bf16 x bf16 -> f32
constexpr uint32_t kIdescBf16NegB = ptx::make_idesc(1, 1, BM, BN, true);
constexpr uint32_t kIdescI8 = ptx::make_idesc(2, 1, BM, BN, false);     // s8 x s8 -> s32

struct I8Args {
  int64_t N, C2;
  int num_kb16, num_kb8;
  int K;
  int64_t mtiles, otiles;
  int64_t num_tiles;       // otiles * mtiles (every tile runs all passes)
  TileRaster raster;       // walk order of the tiles
  const int32_t* n_live;   // device: live token count after compaction, or null (= N)
  int64_t n_pad;
  const float* w_imp;      // [N] or null
  const float* t;          // [K,N] activation steps
  const float* u;          // [K,C2] weight steps
  float* partials;         // [K][otiles*mtiles*8]
  float* ptab;             // [K][otiles*2][n_pad] or null
  const uint16_t* bias;    // apply
  uint16_t* yq;            // apply
  WorkspaceHeader* hdr;
};

__device__ __forceinline__ void report_timeout(WorkspaceHeader* hdr, int where) {
  hdr->where = where;
  hdr->status = TLQ_ERR_TIMEOUT;
}

// kMode 0: W8A8-style search (one bf16 pass for the full-precision tile, then K int8 passes)
// kMode 1: apply (a single int8 pass, bf16 store)
// kMode 2: two-stream search with 16-bit activations (first propagation strategy of paper Sec. 3.2.1):
//          || f_fp(x_fp) - f_q(x_q) ||^2 with f_fp - f_q = (X_fp - X_q) W^T + X_q dW_k^T.  The candidate-free
//          part is accumulated once per tile by two bf16 passes into one accumulator (X_fp W^T, then X_q W^T
//          with the negate bit) and kept in registers; every candidate adds its bf16 pass X_q dW_k^T to it.
//          Tensor maps: tmX = X_fp, tmW = W, tmXq = X_q (bf16, 3-D with a single slice), tmWq = dW (bf16, 3-D).
template <int kMode>
__global__ void __launch_bounds__(kThreads, 1)
gemm_w8a8_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmXq, const __grid_constant__ CUtensorMap tmWq,
                 const I8Args args) {
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
  constexpr bool kApply = kMode == 1;
  constexpr bool kDual = kMode == 2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), kEpiWarps);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmX);
    ptx::prefetch_tensormap(&tmW);
    ptx::prefetch_tensormap(&tmXq);
    ptx::prefetch_tensormap(&tmWq);
  }
  if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), kTmemCols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // pass 0 of a search tile is the full-precision product; apply has the single int8 pass only
  const int n_cand = kApply ? 1 : args.K;      // passes of one work item: its candidates (+ the candidate-free pass)
  // token count and tile walk: fixed by the host, or read from the device when the tokens were compacted
  int64_t n_tokens = args.N, num_tiles = args.num_tiles;
  TileRaster raster = args.raster;
  if (args.n_live != nullptr) {
    n_tokens = *args.n_live;
    const int64_t mt_live = (n_tokens + BM - 1) / BM;
    raster.mtiles = (int)mt_live;
    if (raster.b == 1) raster.a = mt_live > 0 ? (int)mt_live : 1;
    num_tiles = args.otiles * mt_live;
  }

  const TailSplit split = make_tail_split((int)num_tiles, (int)gridDim.x, n_cand);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int w = blockIdx.x; ok; w += gridDim.x) {
        int tile, k0, k1;
        if (!work_item(split, w, n_cand, tile, k0, k1)) break;
        const int passes = kApply ? 1 : k1 - k0 + 1;
        int mt, ot;
        raster.decode(tile, mt, ot);
        for (int pass = 0; pass < passes && ok; ++pass) {
          const bool fp = !kApply && pass == 0;
          const int k = kApply ? 0 : k0 + pass - 1;
          const int nkb = fp ? (kDual ? 2 * args.num_kb16 : args.num_kb16) : (kDual ? args.num_kb16 : args.num_kb8);
          for (int kb = 0; kb < nkb; ++kb) {
            if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
              report_timeout(args.hdr, 11);
              ok = false;
              break;
            }
            const uint32_t a_dst = smem_base + stage * kStageBytes;
            ptx::mbar_expect_tx(full_bar(stage), kStageBytes);
            if (fp && kDual && kb >= args.num_kb16) {        // second half of the reference pass: X_q against W
              const int kq = kb - args.num_kb16;
              ptx::tma_load_3d(a_dst, &tmXq, full_bar(stage), kq * BK16, mt * BM, 0);
              ptx::tma_load_2d(a_dst + kABytes, &tmW, full_bar(stage), kq * BK16, ot * BN);
            } else if (fp) {
              ptx::tma_load_2d(a_dst, &tmX, full_bar(stage), kb * BK16, mt * BM);
              ptx::tma_load_2d(a_dst + kABytes, &tmW, full_bar(stage), kb * BK16, ot * BN);
            } else if (kDual) {                              // a candidate: X_q against its delta weights
              ptx::tma_load_3d(a_dst, &tmXq, full_bar(stage), kb * BK16, mt * BM, 0);
              ptx::tma_load_3d(a_dst + kABytes, &tmWq, full_bar(stage), kb * BK16, ot * BN, k);
            } else {
              ptx::tma_load_3d(a_dst, &tmXq, full_bar(stage), kb * BK8, mt * BM, k);
              ptx::tma_load_3d(a_dst + kABytes, &tmWq, full_bar(stage), kb * BK8, ot * BN, k);
            }
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
      int64_t it = 0;                      // passes issued so far: selects the accumulator
      bool ok = true;
      for (int w = blockIdx.x; ok; w += gridDim.x) {
        int tile, k0, k1;
        if (!work_item(split, w, n_cand, tile, k0, k1)) break;
        const int passes = kApply ? 1 : k1 - k0 + 1;
        for (int pass = 0; pass < passes && ok; ++pass, ++it) {
          const bool fp = !kApply && pass == 0;
          const int nkb = fp ? (kDual ? 2 * args.num_kb16 : args.num_kb16) : (kDual ? args.num_kb16 : args.num_kb8);
          const int acc = (int)(it & 1);
          const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
          if (!ptx::mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) {
            report_timeout(args.hdr, 12);
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
          uint32_t accumulate = 0;
          for (int kb = 0; kb < nkb; ++kb) {
            if (!ptx::mbar_wait(full_bar(stage), phase, abort_flag)) {
              report_timeout(args.hdr, 13);
              ok = false;
              break;
            }
            ptx::tc_fence_after();
            const uint32_t a_addr = smem_base + stage * kStageBytes;
            const uint64_t adesc = ptx::smem_desc_sw128(a_addr);
            const uint64_t bdesc = ptx::smem_desc_sw128(a_addr + kABytes);
            // four instructions per k-block either way: 16 bf16 or 32 int8 along K = 32 bytes per step
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              if (fp || kDual)
                ptx::mma_bf16_ss(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2),
                                 (fp && kDual && kb >= args.num_kb16) ? kIdescBf16NegB : kIdescBf16, accumulate);
              else ptx::mma_i8_ss(d_tmem, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), kIdescI8, accumulate);
              accumulate = 1;
            }
            ptx::mma_commit(empty_bar(stage));
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) ptx::mma_commit(tfull_bar(acc));
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int ew = warp - 2;                      // 0..7
    const int quarter = warp & 3;                 // tensor-memory lanes [32*quarter, +32)
    const int half = ew >> 2;                     // columns [128*half, +128) of the tile
    const int row_in_tile = quarter * 32 + lane;
    float yfp[128];                               // this thread's share of the full-precision tile
    int64_t it = 0;
    bool ok = true;
    for (int w = blockIdx.x; ok; w += gridDim.x) {
      int tile, k0, k1;
      if (!work_item(split, w, n_cand, tile, k0, k1)) break;
      const int passes = kApply ? 1 : k1 - k0 + 1;
      int mt, ot;
      raster.decode(tile, mt, ot);
      const int64_t n = (int64_t)mt * BM + row_in_tile;
      const int64_t col_base = (int64_t)ot * BN + half * 128;
      for (int pass = 0; pass < passes; ++pass, ++it) {
        const int acc = (int)(it & 1);
        const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
        if (!ptx::mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) {
          if (lane == 0) report_timeout(args.hdr, 14);
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN + (uint32_t)half * 128;
        if (!kApply && pass == 0) {
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            uint32_t r[16];
            ptx::tmem_ld16(taddr + c * 16, r);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) yfp[c * 16 + j] = __uint_as_float(r[j]);
          }
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
          continue;
        }
        const int k = kApply ? 0 : k0 + pass - 1;
        const float tn = (!kDual && n < n_tokens) ? args.t[(int64_t)k * args.N + n] : 0.0f;
        const float* u_row = kDual ? nullptr : args.u + (int64_t)k * args.C2;
        if (!kApply) {
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            uint32_t r[8];
            ptx::tmem_ld8(taddr + c * 8, r);
            float tu[8];
            if (!kDual) {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const int64_t col = col_base + c * 8 + j;
                tu[j] = (col < args.C2) ? tn * __ldg(u_row + col) : 0.0f;
              }
            }
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
              float e0, e1;
              if (kDual) {       // (X_fp - X_q) W^T + X_q dW_k^T, both fp32
                e0 = yfp[c * 8 + j] + __uint_as_float(r[j]);
                e1 = yfp[c * 8 + j + 1] + __uint_as_float(r[j + 1]);
              } else {
                e0 = fmaf(-(float)(int)r[j], tu[j], yfp[c * 8 + j]);
                e1 = fmaf(-(float)(int)r[j + 1], tu[j + 1], yfp[c * 8 + j + 1]);
              }
              s0 = fmaf(e0, e0, s0);
              s1 = fmaf(e1, e1, s1);
            }
          }
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
          const float e = s0 + s1;                // sum over this warp's 128 output channels
          if (args.ptab != nullptr) args.ptab[((int64_t)k * args.otiles * 2 + ot * 2 + half) * args.n_pad + n] = e;
          float wn = 0.0f;
          if (n < n_tokens) wn = (args.w_imp != nullptr) ? args.w_imp[n] : 1.0f;
          float v = wn * e;
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
          if (lane == 0)
            args.partials[(int64_t)k * args.otiles * args.mtiles * 8 + ((int64_t)ot * args.mtiles + mt) * 8 + ew] = v;
        } else {
#pragma unroll 1
          for (int c = 0; c < 8; ++c) {
            uint32_t r[16];
            ptx::tmem_ld16(taddr + c * 16, r);
            ptx::tmem_ld_wait();
            if (n < n_tokens) {
#pragma unroll
              for (int p = 0; p < 2; ++p) {
                const int64_t col = col_base + c * 16 + p * 8;
                if (col < args.C2) {
                  uint32_t o[4];
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    float v = (float)(int)r[p * 8 + j] * (tn * __ldg(u_row + col + j));
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

int sm_count() { return device_sm_count(); }

template <int kMode>
int configure_kernel() {
  static OncePerDevice once;
  return once_per_device(once, [] {
    return cudaFuncSetAttribute(gemm_w8a8_kernel<kMode>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  });
}

bool map_bf16_2d(CUtensorMap* tm, const uint16_t* p, int64_t rows, int64_t C1, uint32_t box_rows) {
  const uint64_t dims[2] = {(uint64_t)C1, (uint64_t)rows};
  const uint64_t str[1] = {(uint64_t)C1 * 2};
  const uint32_t box[2] = {BK16, box_rows};
  return encode_tensor_map(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p, dims, str, box);
}

bool map_i8_3d(CUtensorMap* tm, const int8_t* p, int64_t rows, int64_t C1, int K, uint32_t box_rows) {
  const uint64_t dims[3] = {(uint64_t)C1, (uint64_t)rows, (uint64_t)K};
  const uint64_t str[2] = {(uint64_t)C1, (uint64_t)C1 * (uint64_t)rows};
  const uint32_t box[3] = {BK8, box_rows, 1};
  return encode_tensor_map(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, p, dims, str, box);
}

}  // namespace

GemmPlan plan_search_gemm_i8(int64_t N, int64_t C1, int64_t C2, int K) {
  GemmPlan p;
  p.N = N; p.C1 = C1; p.C2 = C2; p.K = K;
  p.mtiles = ceil_div(N, BM);
  p.otiles = ceil_div(C2, BN);
  p.partials_per_k = p.mtiles * p.otiles * 8;
  p.n_pad = p.mtiles * BM;
  return p;
}

int launch_search_gemm_i8(const uint16_t* X, const uint16_t* W, const int8_t* Xq, const int8_t* Wq, const float* t,
                          const float* u, const float* w_imp, const GemmPlan& plan, float* partials, float* ptab,
                          WorkspaceHeader* hdr, const int32_t* n_live, cudaStream_t st) {
  CUtensorMap tmX, tmW, tmXq, tmWq;
  if (!map_bf16_2d(&tmX, X, plan.N, plan.C1, BM) || !map_bf16_2d(&tmW, W, plan.C2, plan.C1, BN) ||
      !map_i8_3d(&tmXq, Xq, plan.N, plan.C1, plan.K, BM) || !map_i8_3d(&tmWq, Wq, plan.C2, plan.C1, plan.K, BN))
    return TLQ_ERR_CUDA;
  int rc = configure_kernel<0>();
  if (rc != TLQ_OK) return rc;
  I8Args a{};
  a.N = plan.N; a.C2 = plan.C2;
  a.num_kb16 = (int)ceil_div(plan.C1, BK16);
  a.num_kb8 = (int)ceil_div(plan.C1, BK8);
  a.K = plan.K;
  a.mtiles = plan.mtiles; a.otiles = plan.otiles;
  a.num_tiles = plan.mtiles * plan.otiles;
  a.n_pad = plan.n_pad;
  a.w_imp = w_imp; a.t = t; a.u = u; a.partials = partials; a.ptab = ptab; a.bias = nullptr; a.yq = nullptr;
  a.hdr = hdr;
  a.n_live = n_live;
  const int sms = sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  const unsigned grid = (unsigned)(a.num_tiles < sms ? a.num_tiles : sms);
  // Every candidate's int8 operands are read once and never again, so nothing is worth keeping in L2 between
  // passes and what counts is how many distinct operand rows the CTAs of a wave share: always the blocked walk
  // (16 token tiles x 9 output tiles: 15.6 MB per wave and pass on the 7B-class gate projection against 31.4 MB for
  // all 64 token tiles x 2.3 output tiles).
  a.raster = make_raster(plan.mtiles, plan.otiles, sms, (int64_t)1 << 40, BM);
  gemm_w8a8_kernel<0><<<grid, kThreads, kSmemBytes, st>>>(tmX, tmW, tmXq, tmWq, a);
  return after_launch();
}

int launch_apply_gemm_i8(const int8_t* Xq, const int8_t* Wq, const float* t, const float* u, const uint16_t* bias,
                         int64_t N, int64_t C1, int64_t C2, uint16_t* Yq, WorkspaceHeader* hdr, cudaStream_t st) {
  CUtensorMap tmXq, tmWq;
  if (!map_i8_3d(&tmXq, Xq, N, C1, 1, BM) || !map_i8_3d(&tmWq, Wq, C2, C1, 1, BN)) return TLQ_ERR_CUDA;
  int rc = configure_kernel<1>();
  if (rc != TLQ_OK) return rc;
  GemmPlan plan = plan_search_gemm_i8(N, C1, C2, 1);
  I8Args a{};
  a.N = N; a.C2 = C2;
  a.num_kb16 = 0;
  a.num_kb8 = (int)ceil_div(C1, BK8);
  a.K = 1;
  a.mtiles = plan.mtiles; a.otiles = plan.otiles;
  a.num_tiles = plan.mtiles * plan.otiles;
  a.n_pad = plan.n_pad;
  a.t = t; a.u = u; a.bias = bias; a.yq = Yq; a.hdr = hdr;
  const int sms = sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  const unsigned grid = (unsigned)(a.num_tiles < sms ? a.num_tiles : sms);
  a.raster = make_raster(plan.mtiles, plan.otiles, sms, plan.N * plan.C1, BM);
  gemm_w8a8_kernel<1><<<grid, kThreads, kSmemBytes, st>>>(tmXq, tmWq, tmXq, tmWq, a);
  return after_launch();
}

// Two-stream search with 16-bit activations: partials / per-token layout as in the int8 search.
int launch_search_gemm_dual_bf16(const uint16_t* Xq, const uint16_t* Xfp, const uint16_t* W, const uint16_t* dW,
                                 const float* w_imp, const GemmPlan& plan, float* partials, float* ptab,
                                 WorkspaceHeader* hdr, cudaStream_t st) {
  CUtensorMap tmX, tmW, tmXq, tmD;
  const uint64_t xdims[3] = {(uint64_t)plan.C1, (uint64_t)plan.N, 1};
  const uint64_t xstr[2] = {(uint64_t)plan.C1 * 2, (uint64_t)plan.C1 * (uint64_t)plan.N * 2};
  const uint32_t xbox[3] = {BK16, BM, 1};
  const uint64_t ddims[3] = {(uint64_t)plan.C1, (uint64_t)plan.C2, (uint64_t)plan.K};
  const uint64_t dstr[2] = {(uint64_t)plan.C1 * 2, (uint64_t)plan.C1 * (uint64_t)plan.C2 * 2};
  const uint32_t dbox[3] = {BK16, BN, 1};
  if (!map_bf16_2d(&tmX, Xfp, plan.N, plan.C1, BM) || !map_bf16_2d(&tmW, W, plan.C2, plan.C1, BN) ||
      !encode_tensor_map(&tmXq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, Xq, xdims, xstr, xbox) ||
      !encode_tensor_map(&tmD, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, dW, ddims, dstr, dbox))
    return TLQ_ERR_CUDA;
  int rc = configure_kernel<2>();
  if (rc != TLQ_OK) return rc;
  I8Args a{};
  a.N = plan.N; a.C2 = plan.C2;
  a.num_kb16 = (int)ceil_div(plan.C1, BK16);
  a.num_kb8 = 0;
  a.K = plan.K;
  a.mtiles = plan.mtiles; a.otiles = plan.otiles;
  a.num_tiles = plan.mtiles * plan.otiles;
  a.n_pad = plan.n_pad;
  a.w_imp = w_imp; a.t = nullptr; a.u = nullptr; a.partials = partials; a.ptab = ptab; a.bias = nullptr; a.yq = nullptr;
  a.hdr = hdr;
  a.n_live = nullptr;
  const int sms = sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  const unsigned grid = (unsigned)(a.num_tiles < sms ? a.num_tiles : sms);
  a.raster = make_raster(plan.mtiles, plan.otiles, sms, plan.N * plan.C1 * 2, BM);
  gemm_w8a8_kernel<2><<<grid, kThreads, kSmemBytes, st>>>(tmX, tmW, tmXq, tmD, a);
  return after_launch();
}

}  // namespace tlq
