// Fake-quantization kernels: Q_w(W * scale) for the group-wise asymmetric setting and the int8
// symmetric row / token quantizers (paper Sec. 2.2 quantizer; Sec. 3.2.1 f_q).
//
// All are streaming kernels whose floor is HBM bandwidth: a tile of the bf16 source is staged once
// in shared memory and re-used for every scale candidate, so the source is read once and each
// candidate's operand is written once.  The arithmetic is kept off the slow conversion / reciprocal
// unit: rounding to an integer is the add-and-subtract of 1.5*2^23 (exact round-half-even in
// binary32 for |x| < 2^22), clamping is done before rounding and in floating point, int8 codes are read out of the low
// mantissa bits, and the per-element quotient value/step is taken as value * (1/step) with an exact
// IEEE division only when the product lies so close to a rounding tie that the two could round
// differently.  The integer produced is therefore always rint(fl32(value / step)), the contract the
// CPU reference uses, at a fraction of the instruction count.
#include "common.cuh"

namespace tlq {

namespace {

constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23

// rint(x) for |x| <= 2^21 without a conversion instruction.
__device__ __forceinline__ float round_magic(float x) { return __fsub_rn(__fadd_rn(x, kMagic), kMagic); }

// Reciprocal to within one ulp (a single instruction on the special-function unit).
__device__ __forceinline__ float rcp_fast(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

// The rare exact path, kept out of line so the common path stays a dozen instructions.
__device__ __noinline__ float exact_quotient_rint(float v, float step, float lo, float hi) {
  const float exact = fminf(fmaxf(__fdiv_rn(v, step), lo), hi);
  return round_magic(exact);
}

// clamp(rint(fl32(v / step)), lo, hi) for integer bounds lo <= hi inside (-1024, 1024), given
// inv ~ 1/step to within one ulp.  Clamping before rounding gives the same integer because the bounds
// are integers and rounding is monotone.  fl32(v * inv) is within |q| * 2.4e-7 of the true quotient
// and fl32(v / step) within |q| * 6e-8, so with |q| < 1024 both lie within 2.5e-4 of it: when the
// product is farther than that from a rounding tie the two round to the same integer, otherwise the
// exact division decides.
__device__ __forceinline__ float quotient_rint_clamped(float v, float step, float inv, float lo, float hi) {
  const float q = fminf(fmaxf(__fmul_rn(v, inv), lo), hi);
  float r = round_magic(q);
  if (fabsf(__fsub_rn(q, r)) > 0.49975f) r = exact_quotient_rint(v, step, lo, hi);
  return r;
}

// ---- packed binary32 pairs: one instruction carries two independent IEEE round-to-nearest operations.
// A pair travels in ONE 64-bit register from its first use to its last: re-pairing two 32-bit registers around
// every operation costs two moves per operand, more than the packed instruction saves (measured: 45 % of the
// executed instructions of the row quantizers were such moves).
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pair_of(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ float2 halves(f32x2 v) {
  float2 r;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(r.x), "=f"(r.y) : "l"(v));
  return r;
}
__device__ __forceinline__ f32x2 pmul(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 padd(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2 psub(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
// two bf16 values packed in a 32-bit word -> their binary32 values as a pair (low half first)
__device__ __forceinline__ f32x2 bf16x2_to_pair(uint32_t v) {
  return pair_of(__uint_as_float(v << 16), __uint_as_float(v & 0xFFFF0000u));
}
__device__ __forceinline__ void unpack16_pairs(const uint4& t0, const uint4& t1, f32x2 (&w)[8]) {
  w[0] = bf16x2_to_pair(t0.x); w[1] = bf16x2_to_pair(t0.y); w[2] = bf16x2_to_pair(t0.z); w[3] = bf16x2_to_pair(t0.w);
  w[4] = bf16x2_to_pair(t1.x); w[5] = bf16x2_to_pair(t1.y); w[6] = bf16x2_to_pair(t1.z); w[7] = bf16x2_to_pair(t1.w);
}
// sixteen consecutive binary32 table entries (64-byte aligned) as eight pairs
__device__ __forceinline__ void load_pairs16(const float* p, f32x2 (&m)[8]) {
  const ulonglong2* q = reinterpret_cast<const ulonglong2*>(p);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const ulonglong2 v = q[j];
    m[2 * j] = v.x;
    m[2 * j + 1] = v.y;
  }
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
  float r;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// Group-wise asymmetric weights (W4A16 and other widths).
// Tile: kGqRows x 512 channels.  A thread owns 16 consecutive channels, a warp spans the 512 channels
// of one row, the 8 warps of the CTA take 8 rows per pass.  A group of g channels is g/16 adjacent
// lanes: min/max go through xor-shuffles.  grid.z splits the candidates when the matrix alone
// would not fill the machine.
// ------------------------------------------------------------------------------------------------
constexpr int kGqRows = 32;      // tile height of the general one-scale kernel (static shared memory)
constexpr int kHotRows = 64;     // tile height of the delta-weight kernel: 64 KB of dynamic shared memory, so the
                                 // per-candidate scale tables are fetched once per 8 rows of a warp, not per 4
constexpr int kGqCols = 512;
constexpr int kGqThreads = 256;
constexpr size_t kHotSmem = (size_t)kHotRows * kGqCols * 2;

// ------------------------------------------------------------------------------------------------
// The search's own fake-quant pass: delta weights of ALL candidates, nothing else.  Same tile and
// thread mapping as the general kernel below, but the inner loop is straight-line code on packed
// binary32 pairs with no clamps and no per-element branch:
//   * a group whose extreme quotients mn/step and mx/step round to integers ra <= 0 <= rb with
//     -ra <= qmax and rb - ra <= qmax cannot clip: every element's quotient lies between the two
//     (division and rounding are monotone), so code = rint(p/step) - ra is already inside [0, qmax]
//     and q - z is just rint(p/step);
//   * rint(p * (1/step)) equals rint(fl32(p/step)) unless the product lies within `tie_eps` of a
//     rounding tie; the distance to the nearest integer is folded into one running maximum per
//     thread and checked once per 16 elements.
// A group that can clip, and a thread that met a near-tie, redo their 16 elements on the general
// path (clamps, exact division), which computes the contract literally.  Both cases are rare.
// ------------------------------------------------------------------------------------------------
// One thread's 16 elements on the literal path (clamps, exact division near ties): the group's step,
// its reciprocal and its minimum are given, the rest is re-read from the staged tile and the tables.
__device__ __noinline__ void delta16_general(const uint4* tile16, const uint16_t* s16, const float* rs16, float mn,
                                             float step, float inv, float qmax_f, uint4* dst) {
  const float zf = -quotient_rint_clamped(mn, step, inv, -qmax_f, 0.0f);
  const float lo = -zf, hi = qmax_f - zf;
#pragma unroll 1
  for (int h = 0; h < 2; ++h) {
    float w[8], sv[8];
    unpack8(tile16[h], w);
    unpack8(*reinterpret_cast<const uint4*>(s16 + h * 8), sv);
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 8; j += 2) {
      float d[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float qz = quotient_rint_clamped(__fmul_rn(sv[j + e], w[j + e]), step, inv, lo, hi);
        d[e] = __fsub_rn(w[j + e], __fmul_rn(__fmul_rn(qz, step), rs16[h * 8 + j + e]));
      }
      o[j >> 1] = pack_bf16x2(d[0], d[1]);
    }
    dst[h] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// What the head of a row leaves for its tail: the unpacked weights, the group's minimum, step and reciprocal, and
// whether the group can clip.
struct RowHead {
  f32x2 w[8];
  float mn, step, inv;
  bool fast;
};

__device__ __forceinline__ void row_head(const uint4& t0, const uint4& t1, const f32x2 (&sv)[8], int lanes_per_group,
                                         float qmax_f, float tie_lim, RowHead& h) {
  unpack16_pairs(t0, t1, h.w);
  float mx, mn;
  {
    const float2 p0 = halves(pmul(sv[0], h.w[0]));       // exact: 8-bit x 8-bit significands
    mx = fmaxf(p0.x, p0.y);
    mn = fminf(p0.x, p0.y);
#pragma unroll
    for (int j = 1; j < 8; ++j) {
      const float2 pj = halves(pmul(sv[j], h.w[j]));
      mx = max3(mx, pj.x, pj.y);
      mn = min3(mn, pj.x, pj.y);
    }
  }
  for (int off = 1; off < lanes_per_group; off <<= 1) {
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
    mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, off));
  }
  const float range = fmaxf(__fsub_rn(mx, mn), TLQ_RANGE_FLOOR);
  const float step = __fdiv_rn(range, qmax_f);
  const float inv = rcp_fast(step);
  const float qa = __fmul_rn(mn, inv), qb = __fmul_rn(mx, inv);
  float ra = round_magic(qa), rb = round_magic(qb);
  if (fmaxf(fabsf(__fsub_rn(qa, ra)), fabsf(__fsub_rn(qb, rb))) > tie_lim) {
    // an extreme sits on a rounding tie (common for bf16 weights: mx == -mn puts both on +-qmax/2): decide exactly
    ra = round_magic(__fdiv_rn(mn, step));
    rb = round_magic(__fdiv_rn(mx, step));
  }
  h.mn = mn; h.step = step; h.inv = inv;
  h.fast = ra <= 0.0f && ra >= -qmax_f && __fsub_rn(rb, ra) <= qmax_f;   // the group cannot clip
}

__device__ __forceinline__ void row_tail(const RowHead& h, const f32x2 (&sv)[8], const f32x2 (&rsv)[8], float tie_lim,
                                         float qmax_f, bool col_ok, const uint4* tile16, const uint16_t* s16,
                                         const float* rs16, uint4* dst) {
  if (!h.fast) {
    if (col_ok) delta16_general(tile16, s16, rs16, h.mn, h.step, h.inv, qmax_f, dst);
    return;
  }
  const f32x2 magic2 = pair_of(kMagic, kMagic);
  const f32x2 inv2 = pair_of(h.inv, h.inv), step2 = pair_of(h.step, h.step);
  uint32_t outw[8];
  float near = 0.0f;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const f32x2 q = pmul(pmul(sv[j], h.w[j]), inv2);
    const f32x2 rq = psub(padd(q, magic2), magic2);      // rint(q), which is q - z
    const float2 df = halves(psub(q, rq));
    near = max3(near, fabsf(df.x), fabsf(df.y));
    const float2 d = halves(psub(h.w[j], pmul(pmul(rq, step2), rsv[j])));
    outw[j] = pack_bf16x2(d.x, d.y);
  }
  if (near > tie_lim) {
    // some element of this thread is near a tie: find the pair(s) and redo them with the exact quotient
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const f32x2 pr = pmul(sv[j], h.w[j]);
      const f32x2 q = pmul(pr, inv2);
      const float2 df = halves(psub(q, psub(padd(q, magic2), magic2)));
      if (fmaxf(fabsf(df.x), fabsf(df.y)) > tie_lim) {
        const float2 pj = halves(pr);
        const f32x2 rq = pair_of(round_magic(__fdiv_rn(pj.x, h.step)), round_magic(__fdiv_rn(pj.y, h.step)));
        const float2 d = halves(psub(h.w[j], pmul(pmul(rq, step2), rsv[j])));
        outw[j] = pack_bf16x2(d.x, d.y);
      }
    }
  }
  if (col_ok) {
    dst[0] = make_uint4(outw[0], outw[1], outw[2], outw[3]);
    dst[1] = make_uint4(outw[4], outw[5], outw[6], outw[7]);
  }
}

__global__ void __launch_bounds__(kGqThreads, 2)
fakequant_delta_kernel(const uint16_t* __restrict__ W, const uint16_t* __restrict__ s_tab,
                       const float* __restrict__ rs_tab, int K, int k_per_cta, int64_t C2, int64_t C1, int group,
                       int qmax, float tie_eps, uint16_t* __restrict__ dW) {
  extern __shared__ uint4 tile_dyn[];
  uint4 (*tile)[kGqCols / 8] = reinterpret_cast<uint4 (*)[kGqCols / 8]>(tile_dyn);
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t col_blocks = (C1 + kGqCols - 1) / kGqCols;      // grid.x = column blocks x row tiles, columns fastest
  const int64_t c0 = (int64_t)(blockIdx.x % col_blocks) * kGqCols + lane * 16;
  const int64_t row0 = (int64_t)(blockIdx.x / col_blocks) * kHotRows;
  const bool col_ok = c0 < C1;
  const int lanes_per_group = group >> 4;
  const float qmax_f = (float)qmax;
  const float tie_lim = 0.5f - tie_eps;
  const int k_begin = blockIdx.y * k_per_cta;
  const int k_end = min(K, k_begin + k_per_cta);

#pragma unroll
  for (int p = 0; p < kHotRows / 8; ++p) {
    const int r = p * 8 + warp;
    uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
    if (col_ok && row0 + r < C2) {
      const uint16_t* src = W + (row0 + r) * C1 + c0;
      v0 = ld_nc_16(src);
      v1 = ld_nc_16(src + 8);
    }
    tile[r][lane * 2] = v0;
    tile[r][lane * 2 + 1] = v1;
  }
  __syncthreads();

  for (int k = k_begin; k < k_end; ++k) {
    f32x2 sv[8], rsv[8];
    if (!col_ok) {          // lanes past the last channel work on zeros and store nothing
#pragma unroll
      for (int j = 0; j < 8; ++j) sv[j] = rsv[j] = pair_of(1.0f, 1.0f);
    } else {
      const uint4* sp = reinterpret_cast<const uint4*>(s_tab + (int64_t)k * C1 + c0);
      unpack16_pairs(sp[0], sp[1], sv);
      load_pairs16(rs_tab + (int64_t)k * C1 + c0, rsv);
    }
#pragma unroll 1
    for (int p = 0; p < kHotRows / 8; ++p) {
      const int r = p * 8 + warp;
      if (row0 + r >= C2) break;                  // rows of a warp ascend with p; shuffles below stay warp-uniform
      RowHead h;
      row_head(tile[r][lane * 2], tile[r][lane * 2 + 1], sv, lanes_per_group, qmax_f, tie_lim, h);
      row_tail(h, sv, rsv, tie_lim, qmax_f, col_ok, &tile[r][lane * 2], s_tab + (int64_t)k * C1 + c0,
               rs_tab + (int64_t)k * C1 + c0, reinterpret_cast<uint4*>(dW + ((int64_t)k * C2 + row0 + r) * C1 + c0));
    }
  }
}

__global__ void __launch_bounds__(kGqThreads)
fakequant_group_kernel(const uint16_t* __restrict__ W, const uint16_t* __restrict__ s_tab,
                       const float* __restrict__ rs_tab, int K, int k_per_cta, int64_t C2, int64_t C1, int group,
                       int qmax, uint16_t* __restrict__ dW, uint8_t* __restrict__ codes, float* __restrict__ steps,
                       int32_t* __restrict__ zeros, const WorkspaceHeader* __restrict__ refine, int row_tiles_per_cta) {
  __shared__ uint4 tile[kGqRows][kGqCols / 8];
  // Residual mode (refine pass of the search): blockIdx.y names an entry of the refine set; the candidate's delta
  // weights d are formed as always and what is stored, in the slot the set assigns, is bf16(d - bf16(d)).
  if (refine != nullptr && (int)blockIdx.y >= refine->refine_count) return;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t col_blocks = (C1 + kGqCols - 1) / kGqCols;      // grid.x = column blocks x runs of row tiles
  const int64_t c0 = (int64_t)(blockIdx.x % col_blocks) * kGqCols + lane * 16;
  const int64_t row_tile0 = (int64_t)(blockIdx.x / col_blocks) * row_tiles_per_cta;
  const bool col_ok = c0 < C1;                    // C1 % 16 == 0 is guaranteed by the group sizes
  const int lanes_per_group = group >> 4;
  const float qmax_f = (float)qmax;
  const int64_t ngroups = C1 / group;
  const int k_begin = refine != nullptr ? refine->refine_cand[blockIdx.y] : blockIdx.y * k_per_cta;
  const int k_end = refine != nullptr ? k_begin + 1 : min(K, k_begin + k_per_cta);
  const int k_shift = refine != nullptr ? refine->refine_slot[blockIdx.y] - k_begin : 0;   // output slot - candidate

  for (int rt = 0; rt < row_tiles_per_cta; ++rt) {
    const int64_t row0 = (row_tile0 + rt) * kGqRows;
    if (row0 >= C2) break;
    if (rt > 0) __syncthreads();                  // the previous tile has been read by every warp
    // stage the W tile (zeros outside the matrix)
#pragma unroll
    for (int p = 0; p < kGqRows / 8; ++p) {
      const int r = p * 8 + warp;
      uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
      if (col_ok && row0 + r < C2) {
        const uint16_t* src = W + (row0 + r) * C1 + c0;
        v0 = ld_nc_16(src);
        v1 = ld_nc_16(src + 8);
      }
      tile[r][lane * 2] = v0;
      tile[r][lane * 2 + 1] = v1;
    }
    __syncthreads();

    for (int k = k_begin; k < k_end; ++k) {
      float sv[16], rsv[16];
      if (s_tab != nullptr && col_ok) {
        const uint16_t* sp = s_tab + (int64_t)k * C1 + c0;
        float a[8], b[8];
        unpack8(*reinterpret_cast<const uint4*>(sp), a);
        unpack8(*reinterpret_cast<const uint4*>(sp + 8), b);
#pragma unroll
        for (int j = 0; j < 8; ++j) { sv[j] = a[j]; sv[8 + j] = b[j]; }
        if (rs_tab != nullptr) {
          const float4* rp = reinterpret_cast<const float4*>(rs_tab + (int64_t)k * C1 + c0);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float4 r4 = rp[j];
            rsv[j * 4] = r4.x; rsv[j * 4 + 1] = r4.y; rsv[j * 4 + 2] = r4.z; rsv[j * 4 + 3] = r4.w;
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) rsv[j] = __fdiv_rn(1.0f, sv[j]);
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) { sv[j] = 1.0f; rsv[j] = 1.0f; }
      }
#pragma unroll 1
      for (int p = 0; p < kGqRows / 8; ++p) {
        const int r = p * 8 + warp;
        float w[16], pr[16];
        {
          float a[8], b[8];
          unpack8(tile[r][lane * 2], a);
          unpack8(tile[r][lane * 2 + 1], b);
#pragma unroll
          for (int j = 0; j < 8; ++j) { w[j] = a[j]; w[8 + j] = b[j]; }
        }
        float mx, mn;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          pr[j] = __fmul_rn(sv[j], w[j]);            // exact: 8-bit x 8-bit significands
          mx = (j == 0) ? pr[0] : fmaxf(mx, pr[j]);
          mn = (j == 0) ? pr[0] : fminf(mn, pr[j]);
        }
        for (int off = 1; off < lanes_per_group; off <<= 1) {
          mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
          mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, off));
        }
        const float range = fmaxf(__fsub_rn(mx, mn), TLQ_RANGE_FLOOR);
        const float step = __fdiv_rn(range, qmax_f);
        const float inv = rcp_fast(step);
        // zero-point z = clamp(-rint(mn / step), 0, qmax), kept as a float
        const float zf = -quotient_rint_clamped(mn, step, inv, -qmax_f, 0.0f);
        const float lo = -zf, hi = qmax_f - zf;          // bounds of q - z
        uint32_t outw[8];
        uint32_t qpack[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
          float d[2];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const float qz = quotient_rint_clamped(pr[j + h], step, inv, lo, hi);     // q - z
            const float dq = __fmul_rn(qz, step);
            const float w_hat = __fmul_rn(dq, rsv[j + h]);
            d[h] = __fsub_rn(w[j + h], w_hat);
            if (codes != nullptr)
              qpack[(j + h) >> 2] |= (__float_as_uint(__fadd_rn(__fadd_rn(qz, zf), kMagic)) & 0xFFu) << (((j + h) & 3) * 8);
          }
          outw[j >> 1] = pack_bf16x2(d[0], d[1]);
          if (refine != nullptr) {      // d - bf16(d) is exact in binary32; its own bf16 rounding leaves 2^-18 |d|
            const uint32_t hi = outw[j >> 1];
            outw[j >> 1] = pack_bf16x2(__fsub_rn(d[0], __uint_as_float(hi << 16)),
                                       __fsub_rn(d[1], __uint_as_float(hi & 0xFFFF0000u)));
          }
        }
        const int64_t row = row0 + r;
        if (col_ok && row < C2) {
          if (dW != nullptr) {
            uint4* dst = reinterpret_cast<uint4*>(dW + ((int64_t)(k + k_shift) * C2 + row) * C1 + c0);
            dst[0] = make_uint4(outw[0], outw[1], outw[2], outw[3]);
            dst[1] = make_uint4(outw[4], outw[5], outw[6], outw[7]);
          }
          if (codes != nullptr)
            *reinterpret_cast<uint4*>(codes + row * C1 + c0) = make_uint4(qpack[0], qpack[1], qpack[2], qpack[3]);
          if ((lane % lanes_per_group) == 0) {
            const int64_t g = c0 / group;
            if (steps != nullptr) steps[row * ngroups + g] = step;
            if (zeros != nullptr) zeros[row * ngroups + g] = (int)zf;
          }
        }
      }
    }
  }
}

int launch_fakequant_group(const uint16_t* W, const uint16_t* s, const float* rs, int K, int64_t C2, int64_t C1,
                           int group, int w_bits, uint16_t* dW, uint8_t* codes, float* steps, int32_t* zeros,
                           cudaStream_t st) {
  const bool hot = dW != nullptr && s != nullptr && rs != nullptr && codes == nullptr && steps == nullptr && zeros == nullptr;
  const int tile_rows = hot ? kHotRows : kGqRows;
  const int64_t ctas = ceil_div(C1, kGqCols) * ceil_div(C2, tile_rows);
  const int sms = device_sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  int64_t kchunks = ceil_div((int64_t)sms * 6, ctas);        // aim for several CTAs per SM
  if (kchunks > K) kchunks = K;
  if (kchunks < 1) kchunks = 1;
  const int k_per_cta = (int)ceil_div(K, kchunks);
  kchunks = ceil_div(K, k_per_cta);
  dim3 grid((unsigned)(ceil_div(C1, kGqCols) * ceil_div(C2, tile_rows)), (unsigned)kchunks);
  if (hot) {
    static OncePerDevice once;
    const int rc_cfg = once_per_device(once, [] {
      return cudaFuncSetAttribute(fakequant_delta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kHotSmem);
    });
    if (rc_cfg != TLQ_OK) return rc_cfg;
    // |quotient| <= qmax + 1 on the straight-line path; 4e-7 per unit covers the reciprocal (1 ulp), the product
    // and the exact quotient's own rounding (together < 2.4e-7 relative)
    const float tie_eps = 4.0e-7f * (float)(1 << w_bits);
    fakequant_delta_kernel<<<grid, kGqThreads, kHotSmem, st>>>(W, s, rs, K, k_per_cta, C2, C1, group, (1 << w_bits) - 1,
                                                        tie_eps, dW);
    return after_launch();
  }
  fakequant_group_kernel<<<grid, kGqThreads, 0, st>>>(W, s, rs, K, k_per_cta, C2, C1, group, (1 << w_bits) - 1, dW,
                                                     codes, steps, zeros, nullptr, 1);
  return after_launch();
}

int launch_fakequant_group_residual(const uint16_t* W, const uint16_t* s, const float* rs, int64_t C2, int64_t C1,
                                    int group, int w_bits, uint16_t* dW, const WorkspaceHeader* hdr, cudaStream_t st) {
  // launched whether or not there is a refine set: few CTAs, each walking a run of row tiles
  constexpr int kRun = 8;
  dim3 grid((unsigned)(ceil_div(C1, kGqCols) * ceil_div(ceil_div(C2, kGqRows), kRun)), (unsigned)kMaxRefine);
  fakequant_group_kernel<<<grid, kGqThreads, 0, st>>>(W, s, rs, 0, 1, C2, C1, group, (1 << w_bits) - 1, dW, nullptr,
                                                     nullptr, nullptr, hdr, kRun);
  return after_launch();
}

// ------------------------------------------------------------------------------------------------
// Symmetric quantization of whole rows into int8 containers: weights per output channel
// (value = scale * w, exact) or activations per token (value = fl32(x * (1/scale))), step =
// max|value| / qpos, code = rint(value / step) (Sec. 2.2, first two equations; qpos = 2^(n-1) - 1).
//
// A row's maximum couples all of its channels, so the work is split in two fully parallel passes
// over 512-channel tiles (32 rows in pass 1, 16 in pass 2).  A thread owns 16 channels of its rows and keeps them, unpacked
// to binary32 pairs, in registers for all of its candidates (read straight from global memory: a warp
// covers 1 KB of a row), so a candidate costs it one load of the 16 multipliers and the arithmetic:
//   pass 1  per (candidate, row) the maximum |value| over the tile's channels -> atomic max on the
//           float's bit pattern (non-negative floats order like integers, so the result does not
//           depend on arrival order); a one-line kernel then turns the maxima into steps in place;
//   pass 2  codes: straight-line packed arithmetic, rint(value * (1/step)) with the distance to the
//           nearest integer folded into one running maximum per thread; a thread that met a
//           near-tie redoes its 16 elements with the exact division.  No clamp is needed:
//           |value| <= max|value| keeps |code| <= qpos.
// `mult` below is the per-channel multiplier of one candidate: the bf16 scale for weights, the
// binary32 reciprocal for activations (from the table, or taken here from a bf16 scale), or 1.
// ------------------------------------------------------------------------------------------------
enum MultKind { kMultScale = 0, kMultRecipTable = 1, kMultRecipOfScale = 2 };
constexpr int kAmaxRowsPerThread = 4;      // pass 1: 32-row tiles (the multipliers of a candidate serve four rows)
constexpr int kCodeRowsPerThread = 2;      // pass 2: 16-row tiles (its temporaries leave room for two rows)

template <int kKind>
__device__ __forceinline__ void load_mult_pairs(const uint16_t* s_row, const float* rs_row, int64_t c0, bool col_ok,
                                                f32x2 (&m)[8]) {
  if (!col_ok || (kKind != kMultRecipTable && s_row == nullptr)) {
#pragma unroll
    for (int j = 0; j < 8; ++j) m[j] = pair_of(1.0f, 1.0f);
    return;
  }
  if (kKind == kMultRecipTable) {
    load_pairs16(rs_row + c0, m);
  } else {
    const uint4* sp = reinterpret_cast<const uint4*>(s_row + c0);
    unpack16_pairs(sp[0], sp[1], m);
    if (kKind == kMultRecipOfScale) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float2 v = halves(m[j]);
        m[j] = pair_of(__fdiv_rn(1.0f, v.x), __fdiv_rn(1.0f, v.y));
      }
    }
  }
}

// This thread's 16 channels of its rows (rows warp, warp + 8, ... of the tile), zeros outside the matrix.
template <int kRows>
__device__ __forceinline__ void load_rows_to_registers(const uint16_t* __restrict__ src, int64_t row0, int64_t R,
                                                       int64_t C1, int64_t c0, bool col_ok, int warp,
                                                       f32x2 (&w)[kRows][8]) {
  uint4 raw[kRows][2];
#pragma unroll
  for (int p = 0; p < kRows; ++p) {            // all loads first, then the unpacking
    const int64_t row = row0 + p * 8 + warp;
    raw[p][0] = raw[p][1] = make_uint4(0, 0, 0, 0);
    if (col_ok && row < R) {
      const uint16_t* sp = src + row * C1 + c0;
      raw[p][0] = ld_nc_16(sp);
      raw[p][1] = ld_nc_16(sp + 8);
    }
  }
#pragma unroll
  for (int p = 0; p < kRows; ++p) unpack16_pairs(raw[p][0], raw[p][1], w[p]);
}

template <int kKind>
__global__ void __launch_bounds__(kGqThreads, 2)
row_amax_kernel(const uint16_t* __restrict__ src, const uint16_t* __restrict__ s_tab, const float* __restrict__ rs_tab,
                int K, int k_per_cta, int64_t R_all, const int32_t* __restrict__ n_rows_dev, int64_t C1,
                int* __restrict__ amax_bits /*[K,R_all], zeroed*/) {
  constexpr int kRows = kAmaxRowsPerThread;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t col_blocks = (C1 + kGqCols - 1) / kGqCols;      // grid.x = column blocks x row tiles, columns fastest
  const int64_t c0 = (int64_t)(blockIdx.x % col_blocks) * kGqCols + lane * 16;
  const int64_t row0 = (int64_t)(blockIdx.x / col_blocks) * (kRows * 8);
  const int64_t R = (n_rows_dev != nullptr) ? (int64_t)*n_rows_dev : R_all;    // rows beyond are not live
  if (row0 >= R) return;                                                        // the whole CTA leaves together
  const bool col_ok = c0 < C1;
  f32x2 w[kRows][8];
  load_rows_to_registers<kRows>(src, row0, R, C1, c0, col_ok, warp, w);
  const int k_begin = blockIdx.y * k_per_cta;
  const int k_end = min(K, k_begin + k_per_cta);
  auto mult_of = [&](int k, f32x2 (&m)[8]) {
    load_mult_pairs<kKind>(s_tab ? s_tab + (int64_t)k * C1 : nullptr, rs_tab ? rs_tab + (int64_t)k * C1 : nullptr, c0,
                           col_ok, m);
  };
  // one candidate: the next candidate's multipliers are requested before this one's arithmetic starts
  auto candidate = [&](int k, const f32x2 (&m)[8], f32x2 (&m_next)[8]) {
    if (k + 1 < k_end) mult_of(k + 1, m_next);
    float a[kRows];
#pragma unroll
    for (int p = 0; p < kRows; ++p) {
      a[p] = 0.0f;                                    // rows and channels outside the matrix were loaded as zeros
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float2 v = halves(pmul(w[p][j], m[j]));
        a[p] = max3(a[p], fabsf(v.x), fabsf(v.y));
      }
    }
    // independent shuffle chains, one per row, instead of one after the other
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
      for (int p = 0; p < kRows; ++p) a[p] = fmaxf(a[p], __shfl_xor_sync(0xFFFFFFFFu, a[p], off));
    }
    float mine = a[0];
#pragma unroll
    for (int p = 1; p < kRows; ++p) mine = (lane == p) ? a[p] : mine;
    const int64_t my_row = row0 + lane * 8 + warp;
    if (lane < kRows && my_row < R) atomicMax(amax_bits + (int64_t)k * R_all + my_row, __float_as_int(mine));
  };
  f32x2 ma[8], mb[8];
  mult_of(k_begin, ma);
  for (int k = k_begin; k < k_end; k += 2) {
    candidate(k, ma, mb);
    if (k + 1 < k_end) candidate(k + 1, mb, ma);
  }
}

__global__ void amax_to_step_kernel(float* __restrict__ v, int64_t n, float qpos) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) v[i] = __fdiv_rn(fmaxf(v[i], TLQ_RANGE_FLOOR), qpos);
}

// One thread's 16 codes with the exact division (a near-tie was seen on the straight-line path).
struct Pairs8 {
  f32x2 v[8];
};
__device__ __noinline__ void codes16_exact(Pairs8 w, Pairs8 m, float st, float qpos, uint4* dst) {
  uint32_t pk[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float2 wv = halves(w.v[j]), mv = halves(m.v[j]);
    const float q0 = fminf(fmaxf(__fdiv_rn(__fmul_rn(wv.x, mv.x), st), -qpos - 1.0f), qpos);
    const float q1 = fminf(fmaxf(__fdiv_rn(__fmul_rn(wv.y, mv.y), st), -qpos - 1.0f), qpos);
    const int e = 2 * j;
    pk[e >> 2] |= (__float_as_uint(__fadd_rn(q0, kMagic)) & 0xFFu) << ((e & 3) * 8);
    pk[e >> 2] |= (__float_as_uint(__fadd_rn(q1, kMagic)) & 0xFFu) << (((e + 1) & 3) * 8);
  }
  *dst = make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

template <int kKind>
__global__ void __launch_bounds__(kGqThreads, 2)
row_codes_kernel(const uint16_t* __restrict__ src, const uint16_t* __restrict__ s_tab, const float* __restrict__ rs_tab,
                 const float* __restrict__ step /*[K,R_all]*/, int K, int k_per_cta, int64_t R_all,
                 const int32_t* __restrict__ n_rows_dev, int64_t C1, float qpos, float tie_eps,
                 int8_t* __restrict__ q /*[K,R_all,C1]*/) {
  constexpr int kRows = kCodeRowsPerThread;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t col_blocks = (C1 + kGqCols - 1) / kGqCols;      // grid.x = column blocks x row tiles, columns fastest
  const int64_t c0 = (int64_t)(blockIdx.x % col_blocks) * kGqCols + lane * 16;
  const int64_t row0 = (int64_t)(blockIdx.x / col_blocks) * (kRows * 8);
  const int64_t R = (n_rows_dev != nullptr) ? (int64_t)*n_rows_dev : R_all;
  if (row0 >= R || c0 >= C1) return;      // no warp-wide operation below
  f32x2 w[kRows][8];
  load_rows_to_registers<kRows>(src, row0, R, C1, c0, true, warp, w);
  const float tie_lim = 0.5f - tie_eps;
  const f32x2 magic2 = pair_of(kMagic, kMagic);
  const int k_begin = blockIdx.y * k_per_cta;
  const int k_end = min(K, k_begin + k_per_cta);
  // what a candidate needs from memory: its 16 multipliers and the steps of this thread's rows
  auto fetch = [&](int k, f32x2 (&m)[8], float (&st)[kRows]) {
    load_mult_pairs<kKind>(s_tab ? s_tab + (int64_t)k * C1 : nullptr, rs_tab ? rs_tab + (int64_t)k * C1 : nullptr, c0,
                           true, m);
#pragma unroll
    for (int p = 0; p < kRows; ++p) {
      const int64_t row = row0 + p * 8 + warp;
      st[p] = row < R ? step[(int64_t)k * R_all + row] : 1.0f;
    }
  };
  // one candidate: the next candidate's operands are requested before this one's arithmetic starts
  auto candidate = [&](int k, const f32x2 (&m)[8], const float (&st)[kRows], f32x2 (&m_next)[8], float (&st_next)[kRows]) {
    if (k + 1 < k_end) fetch(k + 1, m_next, st_next);
#pragma unroll
    for (int p = 0; p < kRows; ++p) {
      const int64_t row = row0 + p * 8 + warp;
      if (row < R) {
        const float inv = rcp_fast(st[p]);
        const f32x2 inv2 = pair_of(inv, inv);
        float near = 0.0f;
        uint32_t tb[16];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const f32x2 qv = pmul(pmul(w[p][j], m[j]), inv2);
          const f32x2 t = padd(qv, magic2);             // low mantissa byte = the code in two's complement
          const float2 df = halves(psub(qv, psub(t, magic2)));
          near = max3(near, fabsf(df.x), fabsf(df.y));
          const float2 th = halves(t);
          tb[2 * j] = __float_as_uint(th.x);
          tb[2 * j + 1] = __float_as_uint(th.y);
        }
        uint4* dst = reinterpret_cast<uint4*>(q + ((int64_t)k * R_all + row) * C1 + c0);
        if (near > tie_lim) {
          Pairs8 wp, mp;
#pragma unroll
          for (int j = 0; j < 8; ++j) { wp.v[j] = w[p][j]; mp.v[j] = m[j]; }
          codes16_exact(wp, mp, st[p], qpos, dst);
        } else {
          uint32_t pk[4];
#pragma unroll
          for (int g = 0; g < 4; ++g)
            pk[g] = __byte_perm(__byte_perm(tb[4 * g], tb[4 * g + 1], 0x0040), __byte_perm(tb[4 * g + 2], tb[4 * g + 3], 0x0040),
                                0x5410);
          *dst = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
    }
  };
  f32x2 ma[8], mb[8];
  float sta[kRows], stb[kRows];
  fetch(k_begin, ma, sta);
  for (int k = k_begin; k < k_end; k += 2) {
    candidate(k, ma, sta, mb, stb);
    if (k + 1 < k_end) candidate(k + 1, mb, stb, ma, sta);
  }
}

template <int kKind>
static int launch_rows(const uint16_t* src, const uint16_t* s, const float* rs, int K, int64_t R, int64_t C1, int bits,
                       int8_t* q, float* step, const int32_t* n_rows_dev, cudaStream_t st) {
  const int sms = device_sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  // candidates are split over grid.y only when the tiles alone would not fill the machine several times over
  auto shape = [&](int tile_rows, int& k_per_cta) {
    const int64_t tiles = ceil_div(C1, kGqCols) * ceil_div(R, tile_rows);
    int64_t kchunks = ceil_div((int64_t)sms * 6, tiles);
    if (kchunks > K) kchunks = K;
    if (kchunks < 1) kchunks = 1;
    k_per_cta = (int)ceil_div(K, kchunks);
    return dim3((unsigned)tiles, (unsigned)ceil_div(K, k_per_cta));
  };
  int kpc_amax = 1, kpc_codes = 1;
  const dim3 grid_amax = shape(kAmaxRowsPerThread * 8, kpc_amax);
  const dim3 grid_codes = shape(kCodeRowsPerThread * 8, kpc_codes);
  const float qpos = (float)((1 << (bits - 1)) - 1);
  const float tie_eps = 4.0e-7f * (qpos + 1.0f);
  const int64_t n = (int64_t)K * R;
  TLQ_CUDA_TRY(cudaMemsetAsync(step, 0, (size_t)n * sizeof(float), st));
  row_amax_kernel<kKind><<<grid_amax, kGqThreads, 0, st>>>(src, s, rs, K, kpc_amax, R, n_rows_dev, C1,
                                                     reinterpret_cast<int*>(step));
  int rc = after_launch();
  if (rc != TLQ_OK) return rc;
  amax_to_step_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(step, n, qpos);
  if ((rc = after_launch()) != TLQ_OK) return rc;
  row_codes_kernel<kKind><<<grid_codes, kGqThreads, 0, st>>>(src, s, rs, step, K, kpc_codes, R, n_rows_dev, C1, qpos, tie_eps, q);
  return after_launch();
}

int launch_fakequant_rows_i8(const uint16_t* W, const uint16_t* s, int K, int64_t C2, int64_t C1, int bits, int8_t* q,
                             float* u, cudaStream_t st) {
  return launch_rows<kMultScale>(W, s, nullptr, K, C2, C1, bits, q, u, nullptr, st);
}

int launch_actquant_i8(const uint16_t* X, const uint16_t* s, const float* rs, int K, int64_t N, int64_t C1, int bits,
                       int8_t* q, float* t, const int32_t* n_rows_dev, cudaStream_t st) {
  if (rs != nullptr) return launch_rows<kMultRecipTable>(X, nullptr, rs, K, N, C1, bits, q, t, n_rows_dev, st);
  return launch_rows<kMultRecipOfScale>(X, s, nullptr, K, N, C1, bits, q, t, n_rows_dev, st);
}

// ------------------------------------------------------------------------------------------------
// Storage format of 4-bit codes: two per byte, the even channel in the low nibble.  Works for the
// unsigned codes of the group mode (0..15) and for the symmetric mode's integers (-8..7, kept as
// two's-complement nibbles).  One thread packs 32 codes (two 128-bit loads, one 128-bit store).
// ------------------------------------------------------------------------------------------------
__global__ void pack_codes4_kernel(const uint8_t* __restrict__ codes, int64_t n_packets, uint8_t* __restrict__ packed) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;      // packet of 32 codes -> 16 bytes
  if (i >= n_packets) return;
  const uint4 a = ld_nc_16(codes + i * 32), b = ld_nc_16(codes + i * 32 + 16);
  auto pack8 = [](uint32_t lo, uint32_t hi) {     // 8 codes (one per byte in lo, hi) -> 4 bytes
    const uint32_t l = lo & 0x0F0F0F0Fu, h = hi & 0x0F0F0F0Fu;
    const uint32_t pl = (l | (l >> 4)) & 0x00FF00FFu;        // bytes 0 and 2 hold the pairs (c0,c1) and (c2,c3)
    const uint32_t ph = (h | (h >> 4)) & 0x00FF00FFu;
    return (pl & 0xFFu) | ((pl >> 8) & 0xFF00u) | ((ph & 0xFFu) << 16) | ((ph >> 8) & 0xFF00u) << 16;
  };
  const uint4 out = make_uint4(pack8(a.x, a.y), pack8(a.z, a.w), pack8(b.x, b.y), pack8(b.z, b.w));
  *reinterpret_cast<uint4*>(packed + i * 16) = out;
}

int launch_pack_codes4(const uint8_t* codes, int64_t n_codes, uint8_t* packed, cudaStream_t st) {
  const int64_t packets = n_codes / 32;
  pack_codes4_kernel<<<(unsigned)ceil_div(packets, 256), 256, 0, st>>>(codes, packets, packed);
  return after_launch();
}

}  // namespace tlq
