// C ABI of libtlq: argument validation, workspace carving and stage sequencing.  All arithmetic of
// the hot path lives in the kernels; nothing here computes on the host.
#include <math.h>
#include <string.h>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"
#include "l2part.cuh"

namespace tlq {

long long g_launch_count = 0;

int device_sm_count() {
  static int sms[kMaxDevices] = {};
  const int dev = current_device_index();
  if (dev < 0) return 0;
  if (sms[dev] == 0 && cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    sms[dev] = 0;
  }
  return sms[dev];
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_cfg(const tlq_config* cfg, int64_t C1, bool need_quantizer = true) {
  if (cfg == nullptr || cfg->struct_size != sizeof(tlq_config)) return TLQ_ERR_INVALID_ARG;
  if ((cfg->flags & ~(uint32_t)(TLQ_FLAG_SKIP_ZERO_WEIGHT_TOKENS | TLQ_FLAG_GEMM_CTA_PAIRS | TLQ_FLAG_GEMM_NARROW_TILES |
                                 TLQ_FLAG_NO_REFINE | TLQ_FLAG_DEBUG_CANARIES)) != 0)
    return TLQ_ERR_INVALID_ARG;
  if (cfg->n_grid < 1 || cfg->n_grid > TLQ_MAX_GRID) return TLQ_ERR_SHAPE;
  if (cfg->stat_mode < TLQ_STAT_MEAN_ABS || cfg->stat_mode > TLQ_STAT_MASKED_MAX) return TLQ_ERR_INVALID_ARG;
  if (C1 < 8 || (C1 % 8) != 0) return TLQ_ERR_SHAPE;
  if (!need_quantizer) return TLQ_OK;
  if (cfg->mode == TLQ_W4A16_ASYM_GROUP) {
    if (cfg->w_bits < 2 || cfg->w_bits > 8 || cfg->a_bits != 16) return TLQ_ERR_UNSUPPORTED;
    const int g = cfg->group_size;
    if (g != 32 && g != 64 && g != 128 && g != 256) return TLQ_ERR_UNSUPPORTED;
    if ((C1 % g) != 0) return TLQ_ERR_SHAPE;
  } else if (cfg->mode == TLQ_W8A8_SYM) {
    if (cfg->w_bits < 2 || cfg->w_bits > 8 || cfg->a_bits < 2 || cfg->a_bits > 8) return TLQ_ERR_UNSUPPORTED;
    if ((C1 % 16) != 0) return TLQ_ERR_SHAPE;
  } else {
    return TLQ_ERR_INVALID_ARG;
  }
  return TLQ_OK;
}

int have_device() {
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || n < 1) {
    cudaGetLastError();
    return TLQ_ERR_CUDA;
  }
  return TLQ_OK;
}

// Carves consecutive 256-byte aligned regions out of a workspace (or only measures when base is null).
// With `guarded` every region is followed by kGuardBytes that no kernel may write (TLQ_FLAG_DEBUG_CANARIES): a
// pattern is put there when a call starts and verified when it ends.
struct Carver {
  uint8_t* base;
  size_t off;
  bool guarded;
  GuardList guards;
  Carver(void* b, bool with_guards) : base(reinterpret_cast<uint8_t*>(b)), off(0), guarded(with_guards) { guards.n = 0; }
  template <typename T>
  T* take(size_t count, size_t align = 256) {
    off = align_up(off, align);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    if (guarded && guards.n < kMaxGuards) {
      off = align_up(off, 16);
      guards.off[guards.n++] = off;
      off += kGuardBytes;
    }
    return p;
  }
};

struct SearchLayout {
  WorkspaceHeader* hdr;
  double* stat_partials;
  double* x_stat;
  uint16_t* s;
  float* rs;
  float* partials;
  float* ptab;
  uint16_t* dW;
  int8_t* Wq;
  float* u;
  int8_t* Xq;
  float* t;
  int32_t* live;         // token compaction: live[0] = live tokens, live[1] = rounded up to 128
  int32_t* live_idx;     // [N] source row of each packed row
  float* wc;             // [n_pad] packed weights
  uint16_t* Xc;          // [n_pad, C1] packed activations
  double* refine_partials; // group mode: [kMaxRefine][refine_per_r] weighted tile sums of the refine pass
  int64_t refine_per_r;
  GuardList guards;      // TLQ_FLAG_DEBUG_CANARIES: where the guard words between the regions are
  size_t bytes;
  GemmPlan plan;         // the mode's own GEMM
  GemmPlan plan_resident; // the tile-resident kernel's (all candidates per tile): symmetric modes and the two-stream search
  int64_t ptab_slices;   // per-candidate slices of the per-token table as the buffers are sized (2 per column tile)
};

SearchLayout carve_search(void* ws, int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg) {
  SearchLayout L{};
  const int K = cfg->n_grid;
  Carver c(ws, (cfg->flags & TLQ_FLAG_DEBUG_CANARIES) != 0);
  const bool i8 = cfg->mode == TLQ_W8A8_SYM;
  L.plan_resident = plan_search_gemm_i8(N, C1, C2, K);
  L.plan = i8 ? L.plan_resident : plan_search_gemm(N, C1, C2, K);
  L.ptab_slices = L.plan.otiles * 2;
  L.hdr = c.take<WorkspaceHeader>(1);
  L.stat_partials = c.take<double>((size_t)stats_row_chunks(N) * C1);
  L.x_stat = c.take<double>((size_t)C1);
  L.s = c.take<uint16_t>((size_t)K * C1);
  L.rs = c.take<float>((size_t)K * C1);
  L.partials = c.take<float>((size_t)K * L.plan_resident.partials_per_k);
  L.ptab = c.take<float>((size_t)K * L.ptab_slices * L.plan.n_pad);
  if (cfg->mode == TLQ_W4A16_ASYM_GROUP) {
    L.dW = c.take<uint16_t>((size_t)K * C2 * C1, 1024);
    L.refine_per_r = refine_partials_per_candidate(N, C2);
    L.refine_partials = c.take<double>((size_t)kMaxRefine * L.refine_per_r);
  } else {
    L.Wq = c.take<int8_t>((size_t)K * C2 * C1, 1024);
    L.u = c.take<float>((size_t)K * C2);
    L.Xq = c.take<int8_t>((size_t)K * N * C1, 1024);
    L.t = c.take<float>((size_t)K * N);
  }
  if (cfg->flags & TLQ_FLAG_SKIP_ZERO_WEIGHT_TOKENS) {
    L.live = c.take<int32_t>(2);
    L.live_idx = c.take<int32_t>((size_t)N);
    L.wc = c.take<float>((size_t)L.plan.n_pad);
    L.Xc = c.take<uint16_t>((size_t)L.plan.n_pad * C1, 1024);
  }
  L.guards = c.guards;
  L.bytes = align_up(c.off, 256);
  return L;
}

// ---------------------------------------------------------------------------------------------- stage timing
// A fixed pool of event sets, one per recorded call; calls beyond the pool are not recorded.
constexpr int kMaxTimedCalls = 512;
bool g_timing_on = false;
cudaEvent_t (*g_ev)[TLQ_N_STAGES + 1] = nullptr;   // [kMaxTimedCalls][5], created on first use
int g_ev_made = 0;      // sets whose events exist
int g_calls = 0;        // calls recorded since the last enable
int g_cur = -1;         // set being recorded by the call in progress

// Stage boundaries of a search call: a named range for timeline profilers (host side: the range covers the
// enqueueing of the stage; free when no tool is attached) and, when stage timing is on, an event on the stream.
const char* const kStageNames[TLQ_N_STAGES] = {"tlq.stats", "tlq.fakequant", "tlq.gemm", "tlq.reduce"};

int timing_mark(int i, cudaStream_t st) {
  if (i > 0) nvtxRangePop();
  if (i < TLQ_N_STAGES) nvtxRangePushA(kStageNames[i]);
  if (!g_timing_on) return TLQ_OK;
  if (i == 0) {
    if (g_calls >= kMaxTimedCalls) { g_cur = -1; return TLQ_OK; }
    if (g_ev == nullptr) g_ev = new cudaEvent_t[kMaxTimedCalls][TLQ_N_STAGES + 1];
    if (g_calls >= g_ev_made) {
      for (int j = 0; j <= TLQ_N_STAGES; ++j) TLQ_CUDA_TRY(cudaEventCreate(&g_ev[g_ev_made][j]));
      ++g_ev_made;
    }
    g_cur = g_calls;
  }
  if (g_cur < 0) return TLQ_OK;
  TLQ_CUDA_TRY(cudaEventRecord(g_ev[g_cur][i], st));
  if (i == TLQ_N_STAGES) { ++g_calls; g_cur = -1; }
  return TLQ_OK;
}

}  // namespace
}  // namespace tlq

using namespace tlq;

extern "C" {

const char* tlq_status_string(int status) {
  switch (status) {
    case TLQ_OK: return "ok";
    case TLQ_ERR_INVALID_ARG: return "invalid argument";
    case TLQ_ERR_SHAPE: return "unsupported shape";
    case TLQ_ERR_ALIGN: return "pointer not 16-byte aligned";
    case TLQ_ERR_UNSUPPORTED: return "unsupported mode or bit width";
    case TLQ_ERR_WORKSPACE: return "workspace too small";
    case TLQ_ERR_CUDA: return "CUDA error or no CUDA device";
    case TLQ_ERR_TIMEOUT: return "device-side wait timed out";
    case TLQ_ERR_NONFINITE: return "all candidate losses are non-finite";
    case TLQ_ERR_OVERRUN: return "a guard word between workspace regions was overwritten";
    default: return "unknown status";
  }
}

int tlq_version(void) { return 1009; }   // 1.9: refine pass (TLQ_FLAG_NO_REFINE), workspace guard words (TLQ_FLAG_DEBUG_CANARIES)

int64_t tlq_kernel_launch_count(void) { return (int64_t)g_launch_count; }

int tlq_token_importance(const void* G, int g_dtype, int64_t B, int64_t N, int64_t C, int norm_kind, float top_frac,
                         float* imp_out, uint8_t* mask_out, void* stream) {
  if (G == nullptr || imp_out == nullptr) return TLQ_ERR_INVALID_ARG;
  if (g_dtype != TLQ_DTYPE_BF16 && g_dtype != TLQ_DTYPE_F32) return TLQ_ERR_INVALID_ARG;
  if (norm_kind != TLQ_NORM_MEAN_ABS && norm_kind != TLQ_NORM_L2) return TLQ_ERR_INVALID_ARG;
  if (B < 1 || N < 1 || C < 8 || (C % 8) != 0 || N > 0x7FFFFFFFLL) return TLQ_ERR_SHAPE;
  if (!(top_frac >= 0.0f) || top_frac > 1.0f) return TLQ_ERR_INVALID_ARG;
  if (!aligned16(G)) return TLQ_ERR_ALIGN;
  int rc = have_device();
  if (rc != TLQ_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  rc = launch_token_importance(G, g_dtype, B, N, C, norm_kind, imp_out, st);
  if (rc != TLQ_OK) return rc;
  if (mask_out != nullptr && top_frac > 0.0f) {
    int64_t k_sel = (int64_t)floor((double)top_frac * (double)N);
    if (k_sel < 1) k_sel = 1;
    rc = launch_top_mask(imp_out, N, k_sel, mask_out, st);
  }
  return rc;
}

size_t tlq_scale_candidates_workspace_bytes(int64_t N, int64_t C1) {
  if (N < 1 || C1 < 1) return 0;
  return align_up((size_t)stats_row_chunks(N) * (size_t)C1 * sizeof(double), 256);
}

int tlq_scale_candidates(const void* X, int64_t N, int64_t C1, const uint8_t* mask, const tlq_config* cfg,
                         void* workspace, size_t workspace_bytes, double* x_stat_out, void* s_out, void* stream) {
  if (X == nullptr || workspace == nullptr || s_out == nullptr) return TLQ_ERR_INVALID_ARG;
  if (N < 1) return TLQ_ERR_SHAPE;
  int rc = check_cfg(cfg, C1, false);   // only the grid and the statistic are used here
  if (rc != TLQ_OK) return rc;
  if (cfg->stat_mode == TLQ_STAT_MASKED_MAX && mask == nullptr) return TLQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(workspace) || !aligned16(s_out)) return TLQ_ERR_ALIGN;
  if (workspace_bytes < tlq_scale_candidates_workspace_bytes(N, C1)) return TLQ_ERR_WORKSPACE;
  rc = have_device();
  if (rc != TLQ_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  double* partials = reinterpret_cast<double*>(workspace);
  rc = launch_channel_stats(reinterpret_cast<const uint16_t*>(X), N, C1, mask, cfg->stat_mode, partials, st);
  if (rc != TLQ_OK) return rc;
  return launch_scale_table(partials, stats_row_chunks(N), N, C1, cfg->stat_mode, cfg->n_grid, x_stat_out,
                            reinterpret_cast<uint16_t*>(s_out), nullptr, st);
}

int tlq_scale_candidates_noalloc(const void* X, int64_t N, int64_t C1, const uint8_t* mask, const tlq_config* cfg,
                                 double* x_stat_out, void* s_out, void* stream) {
  if (X == nullptr || s_out == nullptr) return TLQ_ERR_INVALID_ARG;
  if (N < 1) return TLQ_ERR_SHAPE;
  int rc = check_cfg(cfg, C1, false);
  if (rc != TLQ_OK) return rc;
  if (C1 > static_stats_max_c1()) return TLQ_ERR_SHAPE;   // beyond the built-in scratch
  if (cfg->stat_mode == TLQ_STAT_MASKED_MAX && mask == nullptr) return TLQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(s_out)) return TLQ_ERR_ALIGN;
  rc = have_device();
  if (rc != TLQ_OK) return rc;
  return launch_scale_candidates_static(reinterpret_cast<const uint16_t*>(X), N, C1, mask, cfg->stat_mode, cfg->n_grid,
                                        x_stat_out, reinterpret_cast<uint16_t*>(s_out),
                                        reinterpret_cast<cudaStream_t>(stream));
}

int tlq_quantize_weights(const void* W, const void* s, int64_t C2, int64_t C1, const tlq_config* cfg, uint8_t* codes,
                         float* steps, int32_t* zeros, void* dW_out, void* stream) {
  if (W == nullptr) return TLQ_ERR_INVALID_ARG;
  if (C2 < 1) return TLQ_ERR_SHAPE;
  int rc = check_cfg(cfg, C1);
  if (rc != TLQ_OK) return rc;
  if (!aligned16(W) || (s != nullptr && !aligned16(s)) || (codes != nullptr && !aligned16(codes)) ||
      (dW_out != nullptr && !aligned16(dW_out)))
    return TLQ_ERR_ALIGN;
  rc = have_device();
  if (rc != TLQ_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint16_t* Wb = reinterpret_cast<const uint16_t*>(W);
  const uint16_t* sb = reinterpret_cast<const uint16_t*>(s);
  if (cfg->mode == TLQ_W4A16_ASYM_GROUP)
    return launch_fakequant_group(Wb, sb, nullptr, 1, C2, C1, cfg->group_size, cfg->w_bits, reinterpret_cast<uint16_t*>(dW_out),
                                  codes, steps, zeros, st);
  if (dW_out != nullptr || codes == nullptr || steps == nullptr) return TLQ_ERR_INVALID_ARG;
  return launch_fakequant_rows_i8(Wb, sb, 1, C2, C1, cfg->w_bits, reinterpret_cast<int8_t*>(codes), steps, st);
}

int tlq_pack_codes4(const uint8_t* codes, int64_t rows, int64_t cols, uint8_t* packed, void* stream) {
  if (codes == nullptr || packed == nullptr) return TLQ_ERR_INVALID_ARG;
  if (rows < 1 || cols < 32 || (cols % 32) != 0) return TLQ_ERR_SHAPE;
  if (!aligned16(codes) || !aligned16(packed)) return TLQ_ERR_ALIGN;
  int rc = have_device();
  if (rc != TLQ_OK) return rc;
  return launch_pack_codes4(codes, rows * cols, packed, reinterpret_cast<cudaStream_t>(stream));
}

int tlq_quantize_activations(const void* X, const void* s, int64_t N, int64_t C1, const tlq_config* cfg, int8_t* codes,
                             float* steps, void* stream) {
  if (X == nullptr || codes == nullptr || steps == nullptr) return TLQ_ERR_INVALID_ARG;
  if (N < 1) return TLQ_ERR_SHAPE;
  int rc = check_cfg(cfg, C1);
  if (rc != TLQ_OK) return rc;
  if (cfg->mode != TLQ_W8A8_SYM) return TLQ_ERR_UNSUPPORTED;
  if (!aligned16(X) || (s != nullptr && !aligned16(s)) || !aligned16(codes)) return TLQ_ERR_ALIGN;
  rc = have_device();
  if (rc != TLQ_OK) return rc;
  return launch_actquant_i8(reinterpret_cast<const uint16_t*>(X), reinterpret_cast<const uint16_t*>(s), nullptr, 1, N,
                            C1, cfg->a_bits, codes, steps, nullptr, reinterpret_cast<cudaStream_t>(stream));
}

size_t tlq_scale_search_workspace_bytes(int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg) {
  if (N < 1 || C2 < 1 || check_cfg(cfg, C1) != TLQ_OK) return 0;
  return carve_search(nullptr, N, C1, C2, cfg).bytes;
}

}  // extern "C"

// X is what the quantized layer (and the scale statistic) sees; X_ref, when given, is what the full-precision
// layer sees (two-stream objective).
static int search_impl(const void* X, const void* X_ref, int64_t N, int64_t C1, const void* W, int64_t C2,
                       const float* w_imp, const uint8_t* mask, const tlq_config* cfg, void* workspace,
                       size_t workspace_bytes, int32_t* best_idx, double* losses, void* s_best, float* per_token_err,
                       void* stream) {
  if (X == nullptr || W == nullptr || workspace == nullptr || best_idx == nullptr || losses == nullptr)
    return TLQ_ERR_INVALID_ARG;
  if (N < 1 || C2 < 1 || N > 0x7FFFFF00LL || C2 > 0x7FFFFF00LL) return TLQ_ERR_SHAPE;
  int rc = check_cfg(cfg, C1);
  if (rc != TLQ_OK) return rc;
  if (cfg->stat_mode == TLQ_STAT_MASKED_MAX && mask == nullptr) return TLQ_ERR_INVALID_ARG;
  // skipping needs weights to look at; per-token errors of skipped tokens would not exist
  const bool compact = (cfg->flags & TLQ_FLAG_SKIP_ZERO_WEIGHT_TOKENS) != 0;
  if (compact && (w_imp == nullptr || per_token_err != nullptr)) return TLQ_ERR_INVALID_ARG;
  const bool two_stream = X_ref != nullptr;
  if (two_stream &&
      (cfg->flags & (TLQ_FLAG_SKIP_ZERO_WEIGHT_TOKENS | TLQ_FLAG_GEMM_CTA_PAIRS | TLQ_FLAG_GEMM_NARROW_TILES)) != 0)
    return TLQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W) || !aligned16(workspace) || !aligned16(X_ref)) return TLQ_ERR_ALIGN;
  SearchLayout L = carve_search(workspace, N, C1, C2, cfg);
  if (workspace_bytes < L.bytes) return TLQ_ERR_WORKSPACE;
  rc = have_device();
  if (rc != TLQ_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint16_t* Xb = reinterpret_cast<const uint16_t*>(X);
  const uint16_t* Wb = reinterpret_cast<const uint16_t*>(W);
  const int K = cfg->n_grid;

  TLQ_CUDA_TRY(cudaMemsetAsync(L.hdr, 0, sizeof(WorkspaceHeader), st));
  if (L.guards.n > 0 && (rc = launch_canary_fill(workspace, L.guards, st)) != TLQ_OK) return rc;
  if ((rc = timing_mark(0, st)) != TLQ_OK) return rc;
  if ((rc = launch_channel_stats(Xb, N, C1, mask, cfg->stat_mode, L.stat_partials, st)) != TLQ_OK) return rc;
  if ((rc = launch_scale_table(L.stat_partials, stats_row_chunks(N), N, C1, cfg->stat_mode, K, L.x_stat, L.s, L.rs,
                               st)) != TLQ_OK)
    return rc;
  if ((rc = timing_mark(1, st)) != TLQ_OK) return rc;
  float* ptab = (per_token_err != nullptr) ? L.ptab : nullptr;
  // tokens of zero weight cannot change any loss: pack the others to the front and run the layer on those only
  const uint16_t* Xg = Xb;          // what the quantized layer is applied to
  const float* wg = w_imp;
  const int32_t* n_live = nullptr;
  if (compact) {
    if ((rc = launch_compact_tokens(Xb, w_imp, N, L.plan.n_pad, C1, L.live_idx, L.wc, L.live, L.Xc, st)) != TLQ_OK)
      return rc;
    TLQ_CUDA_TRY(cudaMemsetAsync(L.partials, 0, (size_t)K * L.plan_resident.partials_per_k * sizeof(float), st));
    Xg = L.Xc; wg = L.wc; n_live = L.live;
  }
  if (cfg->mode == TLQ_W4A16_ASYM_GROUP) {
    // which L2 partition each SM sits next to: measured once per device, in the not yet written delta-weight region
    const L2PartMap* l2map = l2_partition_map(L.dW, (size_t)K * C2 * C1 * sizeof(uint16_t), st);
    if ((rc = launch_fakequant_group(Wb, L.s, L.rs, K, C2, C1, cfg->group_size, cfg->w_bits, L.dW, nullptr, nullptr,
                                     nullptr, st)) != TLQ_OK)
      return rc;
    if ((rc = timing_mark(2, st)) != TLQ_OK) return rc;
    if (two_stream) {
      if ((rc = launch_search_gemm_dual_bf16(Xb, reinterpret_cast<const uint16_t*>(X_ref), Wb, L.dW, w_imp,
                                             L.plan_resident, L.partials, ptab, L.hdr, st)) != TLQ_OK)
        return rc;
    } else if (cfg->flags & TLQ_FLAG_GEMM_CTA_PAIRS) {
      if ((rc = launch_search_gemm_bf16_pair(Xg, L.dW, wg, L.plan, L.partials, ptab, L.hdr, n_live, st)) != TLQ_OK)
        return rc;
    } else if ((cfg->flags & TLQ_FLAG_GEMM_NARROW_TILES) || N <= 128) {
      if ((rc = launch_search_gemm_bf16(Xg, L.dW, wg, L.plan, L.partials, ptab, L.hdr, n_live, st)) != TLQ_OK) return rc;
    } else if ((rc = launch_search_gemm_bf16_wide(Xg, L.dW, wg, L.plan, L.partials, ptab, L.hdr, n_live, l2map, st)) !=
               TLQ_OK) {
      return rc;
    }
  } else {
    if ((rc = launch_fakequant_rows_i8(Wb, L.s, K, C2, C1, cfg->w_bits, L.Wq, L.u, st)) != TLQ_OK) return rc;
    if ((rc = launch_actquant_i8(Xg, nullptr, L.rs, K, N, C1, cfg->a_bits, L.Xq, L.t, n_live, st)) != TLQ_OK) return rc;
    if ((rc = timing_mark(2, st)) != TLQ_OK) return rc;
    // the full-precision tile comes from the reference stream when there is one (compaction excludes that case)
    const uint16_t* Xfp = two_stream ? reinterpret_cast<const uint16_t*>(X_ref) : Xg;
    if ((rc = launch_search_gemm_i8(Xfp, Wb, L.Xq, L.Wq, L.t, L.u, wg, L.plan, L.partials, ptab, L.hdr, n_live, st)) !=
        TLQ_OK)
      return rc;
  }
  if ((rc = timing_mark(3, st)) != TLQ_OK) return rc;
  const bool resident = two_stream || cfg->mode != TLQ_W4A16_ASYM_GROUP;
  const GemmPlan& used = resident ? L.plan_resident : L.plan;
  const bool refine =
      cfg->mode == TLQ_W4A16_ASYM_GROUP && !two_stream && K >= 2 && (cfg->flags & TLQ_FLAG_NO_REFINE) == 0;
  if ((rc = launch_loss_reduce(L.partials, used.partials_per_k, K, w_imp, N, C2, L.s, C1, L.hdr, losses, best_idx,
                               reinterpret_cast<uint16_t*>(s_best), refine ? refine_band(C2) : 0.0, st)) != TLQ_OK)
    return rc;
  // Candidates too close to the minimum for the screening arithmetic to order are evaluated again, more exactly; the
  // set is chosen on the device, so the kernels are enqueued regardless and return at once when it is empty.
  if (refine) {
    if (compact)      // token tiles without live tokens are not visited
      TLQ_CUDA_TRY(cudaMemsetAsync(L.refine_partials, 0, (size_t)kMaxRefine * L.refine_per_r * sizeof(double), st));
    if ((rc = launch_fakequant_group_residual(Wb, L.s, L.rs, C2, C1, cfg->group_size, cfg->w_bits, L.dW, L.hdr, st)) !=
        TLQ_OK)
      return rc;
    if ((rc = launch_search_gemm_refine(Xg, L.dW, wg, N, C1, C2, K, L.refine_partials, L.hdr, n_live, st)) != TLQ_OK)
      return rc;
    if ((rc = launch_refine_finish(L.refine_partials, L.refine_per_r, L.s, C1, L.hdr, losses, best_idx,
                                   reinterpret_cast<uint16_t*>(s_best), st)) != TLQ_OK)
      return rc;
  }
  if (per_token_err != nullptr)
    if ((rc = launch_per_token_reduce(L.ptab, K, used.otiles * (resident ? 2 : 1), used.n_pad, N, per_token_err, st)) != TLQ_OK)
      return rc;
  if (L.guards.n > 0 && (rc = launch_canary_check(workspace, L.guards, L.hdr, st)) != TLQ_OK) return rc;
  return timing_mark(4, st);
}

extern "C" {

int tlq_scale_search_layer(const void* X, int64_t N, int64_t C1, const void* W, int64_t C2, const float* w_imp,
                           const uint8_t* mask, const tlq_config* cfg, void* workspace, size_t workspace_bytes,
                           int32_t* best_idx, double* losses, void* s_best, float* per_token_err, void* stream) {
  return search_impl(X, nullptr, N, C1, W, C2, w_imp, mask, cfg, workspace, workspace_bytes, best_idx, losses, s_best,
                     per_token_err, stream);
}

int tlq_scale_search_layer_two_stream(const void* X_q, const void* X_fp, int64_t N, int64_t C1, const void* W,
                                      int64_t C2, const float* w_imp, const uint8_t* mask, const tlq_config* cfg,
                                      void* workspace, size_t workspace_bytes, int32_t* best_idx, double* losses,
                                      void* s_best, float* per_token_err, void* stream) {
  if (X_fp == nullptr) return TLQ_ERR_INVALID_ARG;
  return search_impl(X_q, X_fp, N, C1, W, C2, w_imp, mask, cfg, workspace, workspace_bytes, best_idx, losses, s_best,
                     per_token_err, stream);
}

}  // extern "C"

namespace {
struct ApplyLayout {
  WorkspaceHeader* hdr;
  uint16_t* dW;
  int8_t* Wq;
  float* u;
  int8_t* Xq;
  float* t;
  GuardList guards;
  size_t bytes;
};
ApplyLayout carve_apply(void* ws, int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg) {
  ApplyLayout L{};
  Carver c(ws, (cfg->flags & TLQ_FLAG_DEBUG_CANARIES) != 0);
  L.hdr = c.take<WorkspaceHeader>(1);
  if (cfg->mode == TLQ_W4A16_ASYM_GROUP) {
    L.dW = c.take<uint16_t>((size_t)C2 * C1, 1024);
  } else {
    L.Wq = c.take<int8_t>((size_t)C2 * C1, 1024);
    L.u = c.take<float>((size_t)C2);
    L.Xq = c.take<int8_t>((size_t)N * C1, 1024);
    L.t = c.take<float>((size_t)N);
  }
  L.guards = c.guards;
  L.bytes = align_up(c.off, 256);
  return L;
}
}  // namespace

extern "C" {

size_t tlq_apply_layer_workspace_bytes(int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg) {
  if (N < 1 || C2 < 1 || check_cfg(cfg, C1) != TLQ_OK) return 0;
  return carve_apply(nullptr, N, C1, C2, cfg).bytes;
}

int tlq_apply_layer(const void* X, int64_t N, int64_t C1, const void* W, int64_t C2, const void* s, const void* bias,
                    const tlq_config* cfg, void* workspace, size_t workspace_bytes, uint8_t* codes, float* steps,
                    int32_t* zeros, void* Yq, void* stream) {
  if (X == nullptr || W == nullptr || workspace == nullptr || Yq == nullptr) return TLQ_ERR_INVALID_ARG;
  if (N < 1 || C2 < 8 || (C2 % 8) != 0 || N > 0x7FFFFF00LL) return TLQ_ERR_SHAPE;
  int rc = check_cfg(cfg, C1);
  if (rc != TLQ_OK) return rc;
  if (!aligned16(X) || !aligned16(W) || !aligned16(workspace) || !aligned16(Yq) || (s != nullptr && !aligned16(s)) ||
      (codes != nullptr && !aligned16(codes)))
    return TLQ_ERR_ALIGN;
  ApplyLayout L = carve_apply(workspace, N, C1, C2, cfg);
  if (workspace_bytes < L.bytes) return TLQ_ERR_WORKSPACE;
  rc = have_device();
  if (rc != TLQ_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const uint16_t* Xb = reinterpret_cast<const uint16_t*>(X);
  const uint16_t* Wb = reinterpret_cast<const uint16_t*>(W);
  const uint16_t* sb = reinterpret_cast<const uint16_t*>(s);
  const uint16_t* bb = reinterpret_cast<const uint16_t*>(bias);
  TLQ_CUDA_TRY(cudaMemsetAsync(L.hdr, 0, sizeof(WorkspaceHeader), st));
  if (L.guards.n > 0 && (rc = launch_canary_fill(workspace, L.guards, st)) != TLQ_OK) return rc;
  if (cfg->mode == TLQ_W4A16_ASYM_GROUP) {
    if ((rc = launch_fakequant_group(Wb, sb, nullptr, 1, C2, C1, cfg->group_size, cfg->w_bits, L.dW, codes, steps,
                                     zeros, st)) != TLQ_OK)
      return rc;
    rc = launch_apply_gemm_bf16(Xb, Wb, L.dW, bb, N, C1, C2, reinterpret_cast<uint16_t*>(Yq), L.hdr, st);
  } else {
    if ((rc = launch_fakequant_rows_i8(Wb, sb, 1, C2, C1, cfg->w_bits, L.Wq, L.u, st)) != TLQ_OK) return rc;
    if ((rc = launch_actquant_i8(Xb, sb, nullptr, 1, N, C1, cfg->a_bits, L.Xq, L.t, nullptr, st)) != TLQ_OK) return rc;
    if (codes != nullptr) TLQ_CUDA_TRY(cudaMemcpyAsync(codes, L.Wq, (size_t)C2 * C1, cudaMemcpyDeviceToDevice, st));
    if (steps != nullptr)
      TLQ_CUDA_TRY(cudaMemcpyAsync(steps, L.u, (size_t)C2 * sizeof(float), cudaMemcpyDeviceToDevice, st));
    rc = launch_apply_gemm_i8(L.Xq, L.Wq, L.t, L.u, bb, N, C1, C2, reinterpret_cast<uint16_t*>(Yq), L.hdr, st);
  }
  if (rc != TLQ_OK) return rc;
  if (L.guards.n > 0) rc = launch_canary_check(workspace, L.guards, L.hdr, st);
  return rc;
}

// The guard words of a workspace laid out for (kind, N, C1, C2, cfg): kind 0 = search, 1 = apply.
static int guards_of(int kind, int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg, void* ws, GuardList* out,
                     size_t* bytes) {
  if (kind != 0 && kind != 1) return TLQ_ERR_INVALID_ARG;
  if (N < 1 || C2 < 1) return TLQ_ERR_SHAPE;
  const int rc = check_cfg(cfg, C1);
  if (rc != TLQ_OK) return rc;
  if ((cfg->flags & TLQ_FLAG_DEBUG_CANARIES) == 0) return TLQ_ERR_INVALID_ARG;
  if (kind == 0) {
    const SearchLayout L = carve_search(ws, N, C1, C2, cfg);
    *out = L.guards; *bytes = L.bytes;
  } else {
    const ApplyLayout L = carve_apply(ws, N, C1, C2, cfg);
    *out = L.guards; *bytes = L.bytes;
  }
  return TLQ_OK;
}

int tlq_debug_canary_offsets(int kind, int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg, uint64_t* offsets,
                             int max_offsets) {
  GuardList g;
  size_t bytes = 0;
  const int rc = guards_of(kind, N, C1, C2, cfg, nullptr, &g, &bytes);
  if (rc != TLQ_OK) return rc;
  for (int i = 0; i < g.n && i < max_offsets && offsets != nullptr; ++i) offsets[i] = g.off[i];
  return g.n;
}

int tlq_debug_check_canaries(int kind, int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg, void* workspace,
                             size_t workspace_bytes, void* stream) {
  if (workspace == nullptr) return TLQ_ERR_INVALID_ARG;
  if (!aligned16(workspace)) return TLQ_ERR_ALIGN;
  GuardList g;
  size_t bytes = 0;
  int rc = guards_of(kind, N, C1, C2, cfg, workspace, &g, &bytes);
  if (rc != TLQ_OK) return rc;
  if (workspace_bytes < bytes) return TLQ_ERR_WORKSPACE;
  if ((rc = have_device()) != TLQ_OK) return rc;
  return launch_canary_check(workspace, g, reinterpret_cast<WorkspaceHeader*>(workspace),
                             reinterpret_cast<cudaStream_t>(stream));
}

int tlq_read_status(const void* workspace, void* stream) {
  if (workspace == nullptr) return TLQ_ERR_INVALID_ARG;
  if (have_device() != TLQ_OK) return TLQ_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return TLQ_ERR_CUDA;
  int32_t status = 0;
  if (cudaMemcpy(&status, workspace, sizeof(status), cudaMemcpyDeviceToHost) != cudaSuccess) return TLQ_ERR_CUDA;
  return status;
}

int tlq_selftest_bounded_wait(void* workspace, size_t workspace_bytes, int64_t limit_cycles, void* stream) {
  if (workspace == nullptr) return TLQ_ERR_INVALID_ARG;
  if (!aligned16(workspace)) return TLQ_ERR_ALIGN;
  if (workspace_bytes < sizeof(WorkspaceHeader)) return TLQ_ERR_WORKSPACE;
  if (limit_cycles < 1 || limit_cycles > 2000000000LL) return TLQ_ERR_INVALID_ARG;   // at most about a second
  int rc = have_device();
  if (rc != TLQ_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  TLQ_CUDA_TRY(cudaMemsetAsync(workspace, 0, sizeof(WorkspaceHeader), st));
  return launch_bounded_wait_selftest(reinterpret_cast<WorkspaceHeader*>(workspace), (long long)limit_cycles, st);
}

int tlq_l2_partition_info(int32_t* info, uint8_t* part) {
  if (info == nullptr) return TLQ_ERR_INVALID_ARG;
  int rc = have_device();
  if (rc != TLQ_OK) return rc;
  L2PartMap m;
  if ((rc = l2_partition_read(&m)) != TLQ_OK) return rc;
  info[0] = m.valid; info[1] = m.n_sms; info[2] = m.count[0]; info[3] = m.count[1];
  if (part != nullptr) memcpy(part, m.part, sizeof(m.part));
  return TLQ_OK;
}

int tlq_debug_tile_walk(int64_t mtiles, int64_t otiles, int32_t K, int32_t n0, int32_t n1, int32_t blocked,
                        int32_t block_a, int32_t* visits) {
  if (visits == nullptr) return TLQ_ERR_INVALID_ARG;
  if (mtiles < 1 || otiles < 1 || K < 1 || K > TLQ_MAX_GRID || n0 < 1 || n1 < 0 || block_a < 1 ||
      mtiles > 0x7FFFFF || otiles > 0x7FFFFF)
    return TLQ_ERR_SHAPE;
  const bool split = n1 > 0;
  if (split && (blocked != 0 || mtiles < 4 || n0 * 4 < n0 + n1 || n1 * 4 < n0 + n1)) return TLQ_ERR_UNSUPPORTED;
  const int grid = n0 + n1;
  for (int part = split ? 0 : -1; part < (split ? 2 : 0); ++part) {
    const int n_part = split ? (part == 0 ? n0 : n1) : grid;
    for (int rank = 0; rank < n_part; ++rank) {
      TileWalk w;
      fill_tile_walk(w, part, rank, n_part, (int)mtiles, (int)otiles, K, blocked != 0, block_a, n0, grid);
      int k = 0;
      for (int64_t item = w.first; item < w.count; item += w.stride) {
        int mt, ot;
        w.decode(item, k, mt, ot);
        if (k < 0 || k >= K || mt < 0 || mt >= mtiles || ot < 0 || ot >= otiles) return TLQ_ERR_INVALID_ARG;
        visits[((int64_t)k * otiles + ot) * mtiles + mt] += 1;
      }
    }
  }
  return TLQ_OK;
}

int tlq_debug_resident_walk(int64_t mtiles, int64_t otiles, int32_t K, int32_t grid, int32_t blocked, int32_t* visits) {
  if (visits == nullptr) return TLQ_ERR_INVALID_ARG;
  if (mtiles < 1 || otiles < 1 || K < 1 || K > TLQ_MAX_GRID || grid < 1 || mtiles * otiles > 0x7FFFFFFF)
    return TLQ_ERR_SHAPE;
  const int num_tiles = (int)(mtiles * otiles);
  const TileRaster raster = make_raster(mtiles, otiles, grid, blocked ? ((int64_t)1 << 40) : 0, 128);
  const TailSplit split = make_tail_split(num_tiles, grid, K);
  for (int cta = 0; cta < grid; ++cta) {
    for (int w = cta;; w += grid) {
      int tile, k0, k1;
      if (!work_item(split, w, K, tile, k0, k1)) break;
      int mt, ot;
      raster.decode(tile, mt, ot);
      if (tile < 0 || tile >= num_tiles || mt < 0 || mt >= mtiles || ot < 0 || ot >= otiles || k0 < 0 || k1 > K)
        return TLQ_ERR_INVALID_ARG;
      for (int k = k0; k < k1; ++k) visits[((int64_t)k * otiles + ot) * mtiles + mt] += 1;
    }
  }
  return TLQ_OK;
}

int tlq_stage_timing_enable(int on) {
  g_timing_on = on != 0;
  g_calls = 0;
  g_cur = -1;
  return TLQ_OK;
}

int tlq_stage_timing_drain(float* ms_out, int max_calls) {
  if (ms_out == nullptr || max_calls < 0) return TLQ_ERR_INVALID_ARG;
  if (!g_timing_on) return TLQ_ERR_INVALID_ARG;
  const int n = g_calls < max_calls ? g_calls : max_calls;
  for (int c = 0; c < n; ++c) {
    if (cudaEventSynchronize(g_ev[c][TLQ_N_STAGES]) != cudaSuccess) return TLQ_ERR_CUDA;
    for (int i = 0; i < TLQ_N_STAGES; ++i)
      if (cudaEventElapsedTime(&ms_out[c * TLQ_N_STAGES + i], g_ev[c][i], g_ev[c][i + 1]) != cudaSuccess)
        return TLQ_ERR_CUDA;
  }
  g_calls = 0;
  return n;
}

}  // extern "C"
