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

// ---- packed binary32 pairs: one instruction carries two independent IEEE round-to-nearest operations
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
  float2 r;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return r;
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
  float2 r;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return r;
}
__device__ __forceinline__ float2 sub2(float2 a, float2 b) {
  float2 r;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "sub.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return r;
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
// two bf16 values packed in a 32-bit word -> their binary32 values (low half first)
__device__ __forceinline__ float2 unpack2(uint32_t v) {
  return make_float2(__uint_as_float(v << 16), __uint_as_float(v & 0xFFFF0000u));
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
constexpr int kRowRows = 32;     // row quantizers: 32 KB tiles leave the L1 to the per-candidate reciprocal tables (64-row tiles measured slower)
constexpr size_t kRowSmem = (size_t)kRowRows * kGqCols * 2;

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

  const float2 magic2 = make_float2(kMagic, kMagic);
  for (int k = k_begin; k < k_end; ++k) {
    float2 sv[8], rsv[8];
    if (!col_ok) {          // lanes past the last channel work on zeros and store nothing
#pragma unroll
      for (int j = 0; j < 8; ++j) sv[j] = rsv[j] = make_float2(1.0f, 1.0f);
    } else {
      const uint4* sp = reinterpret_cast<const uint4*>(s_tab + (int64_t)k * C1 + c0);
      const uint4 a = sp[0], b = sp[1];
      sv[0] = unpack2(a.x); sv[1] = unpack2(a.y); sv[2] = unpack2(a.z); sv[3] = unpack2(a.w);
      sv[4] = unpack2(b.x); sv[5] = unpack2(b.y); sv[6] = unpack2(b.z); sv[7] = unpack2(b.w);
      const float4* rp = reinterpret_cast<const float4*>(rs_tab + (int64_t)k * C1 + c0);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 r4 = rp[j];
        rsv[2 * j] = make_float2(r4.x, r4.y);
        rsv[2 * j + 1] = make_float2(r4.z, r4.w);
      }
    }
#pragma unroll 1
    for (int p = 0; p < kHotRows / 8; ++p) {
      const int r = p * 8 + warp;
      const int64_t row = row0 + r;
      if (row >= C2) break;                       // rows of a warp ascend with p; shuffles below stay warp-uniform
      const uint4 t0 = tile[r][lane * 2], t1 = tile[r][lane * 2 + 1];
      float2 w[8];
      w[0] = unpack2(t0.x); w[1] = unpack2(t0.y); w[2] = unpack2(t0.z); w[3] = unpack2(t0.w);
      w[4] = unpack2(t1.x); w[5] = unpack2(t1.y); w[6] = unpack2(t1.z); w[7] = unpack2(t1.w);
      float mx, mn;
      {
        const float2 p0 = mul2(sv[0], w[0]);       // exact: 8-bit x 8-bit significands
        mx = fmaxf(p0.x, p0.y);
        mn = fminf(p0.x, p0.y);
#pragma unroll
        for (int j = 1; j < 8; ++j) {
          const float2 pj = mul2(sv[j], w[j]);
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
      const bool fast = ra <= 0.0f && ra >= -qmax_f && __fsub_rn(rb, ra) <= qmax_f;   // the group cannot clip
      uint32_t outw[8];
      if (fast) {
        const float2 inv2 = make_float2(inv, inv), step2 = make_float2(step, step);
        float near = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float2 pj = mul2(sv[j], w[j]);
          const float2 q = mul2(pj, inv2);
          const float2 rq = sub2(add2(q, magic2), magic2);      // rint(q), which is q - z
          const float2 df = sub2(q, rq);
          near = max3(near, fabsf(df.x), fabsf(df.y));
          const float2 w_hat = mul2(mul2(rq, step2), rsv[j]);
          const float2 d = sub2(w[j], w_hat);
          outw[j] = pack_bf16x2(d.x, d.y);
        }
        if (near > tie_lim) {
          // some element of this thread is near a tie: find the pair(s) and redo them with the exact quotient
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float2 pj = mul2(sv[j], w[j]);
            const float2 q = mul2(pj, inv2);
            const float2 df = sub2(q, sub2(add2(q, magic2), magic2));
            if (fmaxf(fabsf(df.x), fabsf(df.y)) > tie_lim) {
              const float2 rq = make_float2(round_magic(__fdiv_rn(pj.x, step)), round_magic(__fdiv_rn(pj.y, step)));
              const float2 d = sub2(w[j], mul2(mul2(rq, step2), rsv[j]));
              outw[j] = pack_bf16x2(d.x, d.y);
            }
          }
        }
      }
      uint4* dst = reinterpret_cast<uint4*>(dW + ((int64_t)k * C2 + row) * C1 + c0);
      if (!fast) {
        if (col_ok)
          delta16_general(&tile[r][lane * 2], s_tab + (int64_t)k * C1 + c0, rs_tab + (int64_t)k * C1 + c0, mn, step, inv,
                          qmax_f, dst);
      } else if (col_ok) {
        dst[0] = make_uint4(outw[0], outw[1], outw[2], outw[3]);
        dst[1] = make_uint4(outw[4], outw[5], outw[6], outw[7]);
      }
    }
  }
}

__global__ void __launch_bounds__(kGqThreads)
fakequant_group_kernel(const uint16_t* __restrict__ W, const uint16_t* __restrict__ s_tab,
                       const float* __restrict__ rs_tab, int K, int k_per_cta, int64_t C2, int64_t C1, int group,
                       int qmax, uint16_t* __restrict__ dW, uint8_t* __restrict__ codes, float* __restrict__ steps,
                       int32_t* __restrict__ zeros) {
  __shared__ uint4 tile[kGqRows][kGqCols / 8];
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t col_blocks = (C1 + kGqCols - 1) / kGqCols;      // grid.x = column blocks x row tiles, columns fastest
  const int64_t c0 = (int64_t)(blockIdx.x % col_blocks) * kGqCols + lane * 16;
  const int64_t row0 = (int64_t)(blockIdx.x / col_blocks) * kGqRows;
  const bool col_ok = c0 < C1;                    // C1 % 16 == 0 is guaranteed by the group sizes
  const int lanes_per_group = group >> 4;
  const float qmax_f = (float)qmax;
  const int64_t ngroups = C1 / group;
  const int k_begin = blockIdx.y * k_per_cta;
  const int k_end = min(K, k_begin + k_per_cta);

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
      }
      const int64_t row = row0 + r;
      if (col_ok && row < C2) {
        if (dW != nullptr) {
          uint4* dst = reinterpret_cast<uint4*>(dW + ((int64_t)k * C2 + row) * C1 + c0);
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
                                                     codes, steps, zeros);
  return after_launch();
}

// ------------------------------------------------------------------------------------------------
// Symmetric quantization of whole rows into int8 containers: weights per output channel
// (value = scale * w, exact) or activations per token (value = fl32(x * (1/scale))), step =
// max|value| / qpos, code = rint(value / step) (Sec. 2.2, first two equations; qpos = 2^(n-1) - 1).
//
// A row's maximum couples all of its channels, so the work is split in two fully parallel passes
// over the same 32-row x 512-channel tiles as the group kernels, each tile staged once in shared
// memory and re-used for every candidate:
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

template <int kKind>
__device__ __forceinline__ void load_mult16(const uint16_t* s_row, const float* rs_row, int64_t c0, bool col_ok,
                                            float2 (&m)[8]) {
  if (!col_ok || (kKind != kMultRecipTable && s_row == nullptr)) {
#pragma unroll
    for (int j = 0; j < 8; ++j) m[j] = make_float2(1.0f, 1.0f);
    return;
  }
  if (kKind == kMultRecipTable) {
    const float4* rp = reinterpret_cast<const float4*>(rs_row + c0);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 r4 = rp[j];
      m[2 * j] = make_float2(r4.x, r4.y);
      m[2 * j + 1] = make_float2(r4.z, r4.w);
    }
  } else {
    const uint4* sp = reinterpret_cast<const uint4*>(s_row + c0);
    const uint4 a = sp[0], b = sp[1];
    m[0] = unpack2(a.x); m[1] = unpack2(a.y); m[2] = unpack2(a.z); m[3] = unpack2(a.w);
    m[4] = unpack2(b.x); m[5] = unpack2(b.y); m[6] = unpack2(b.z); m[7] = unpack2(b.w);
    if (kKind == kMultRecipOfScale) {
#pragma unroll
      for (int j = 0; j < 8; ++j) m[j] = make_float2(__fdiv_rn(1.0f, m[j].x), __fdiv_rn(1.0f, m[j].y));
    }
  }
}

__device__ __forceinline__ void stage_tile(uint4 (*tile)[kGqCols / 8], const uint16_t* __restrict__ src, int64_t row0,
                                           int64_t R, int64_t C1, int64_t c0, bool col_ok, int warp, int lane) {
#pragma unroll
  for (int p = 0; p < kRowRows / 8; ++p) {
    const int r = p * 8 + warp;
    uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
    if (col_ok && row0 + r < R) {
      const uint16_t* sp = src + (row0 + r) * C1 + c0;
      v0 = ld_nc_16(sp);
      v1 = ld_nc_16(sp + 8);
    }
    tile[r][lane * 2] = v0;
    tile[r][lane * 2 + 1] = v1;
  }
  __syncthreads();
}

__device__ __forceinline__ void unpack16(const uint4& t0, const uint4& t1, float2 (&w)[8]) {
  w[0] = unpack2(t0.x); w[1] = unpack2(t0.y); w[2] = unpack2(t0.z); w[3] = unpack2(t0.w);
  w[4] = unpack2(t1.x); w[5] = unpack2(t1.y); w[6] = unpack2(t1.z); w[7] = unpack2(t1.w);
}

template <int kKind>
__global__ void __launch_bounds__(kGqThreads, 3)
row_amax_kernel(const uint16_t* __restrict__ src, const uint16_t* __restrict__ s_tab, const float* __restrict__ rs_tab,
                int K, int k_per_cta, int64_t R_all, const int32_t* __restrict__ n_rows_dev, int64_t C1,
                int* __restrict__ amax_bits /*[K,R_all], zeroed*/) {
  extern __shared__ uint4 tile_dyn[];
  uint4 (*tile)[kGqCols / 8] = reinterpret_cast<uint4 (*)[kGqCols / 8]>(tile_dyn);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t col_blocks = (C1 + kGqCols - 1) / kGqCols;      // grid.x = column blocks x row tiles, columns fastest
  const int64_t c0 = (int64_t)(blockIdx.x % col_blocks) * kGqCols + lane * 16;
  const int64_t row0 = (int64_t)(blockIdx.x / col_blocks) * kRowRows;
  const int64_t R = (n_rows_dev != nullptr) ? (int64_t)*n_rows_dev : R_all;    // rows beyond are not live
  if (row0 >= R) return;                                                        // the whole CTA leaves together
  const bool col_ok = c0 < C1;
  stage_tile(tile, src, row0, R, C1, c0, col_ok, warp, lane);
  const int k_begin = blockIdx.y * k_per_cta;
  const int k_end = min(K, k_begin + k_per_cta);
  for (int k = k_begin; k < k_end; ++k) {
    float2 m[8];
    load_mult16<kKind>(s_tab ? s_tab + (int64_t)k * C1 : nullptr, rs_tab ? rs_tab + (int64_t)k * C1 : nullptr, c0,
                       col_ok, m);
    // four of the warp's rows at a time: four independent shuffle chains instead of one after the other
#pragma unroll 1
    for (int h = 0; h < kRowRows / 32; ++h) {
      float a[4];
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        const int r = (h * 4 + p) * 8 + warp;          // rows past the end were staged as zeros
        float2 w[8];
        unpack16(tile[r][lane * 2], tile[r][lane * 2 + 1], w);
        a[p] = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float2 v = mul2(w[j], m[j]);
          a[p] = max3(a[p], fabsf(v.x), fabsf(v.y));
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
        for (int p = 0; p < 4; ++p) a[p] = fmaxf(a[p], __shfl_xor_sync(0xFFFFFFFFu, a[p], off));
      }
      float mine = a[0];
#pragma unroll
      for (int p = 1; p < 4; ++p) mine = (lane == p) ? a[p] : mine;
      const int64_t my_row = row0 + (h * 4 + lane) * 8 + warp;
      if (lane < 4 && my_row < R) atomicMax(amax_bits + (int64_t)k * R_all + my_row, __float_as_int(mine));
    }
  }
}

__global__ void amax_to_step_kernel(float* __restrict__ v, int64_t n, float qpos) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) v[i] = __fdiv_rn(fmaxf(v[i], TLQ_RANGE_FLOOR), qpos);
}

// One thread's 16 codes with the exact division (a near-tie was seen on the straight-line path).
__device__ __noinline__ void codes16_exact(const uint4* tile16, const float* mult16, float st, float qpos, uint4* dst) {
  uint32_t pk[4] = {0u, 0u, 0u, 0u};
#pragma unroll 1
  for (int h = 0; h < 2; ++h) {
    float w[8];
    unpack8(tile16[h], w);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float v = __fmul_rn(w[j], mult16[h * 8 + j]);
      const float q = fminf(fmaxf(__fdiv_rn(v, st), -qpos - 1.0f), qpos);
      const int e = h * 8 + j;
      pk[e >> 2] |= (__float_as_uint(__fadd_rn(q, kMagic)) & 0xFFu) << ((e & 3) * 8);
    }
  }
  *dst = make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

template <int kKind>
__global__ void __launch_bounds__(kGqThreads, 3)
row_codes_kernel(const uint16_t* __restrict__ src, const uint16_t* __restrict__ s_tab, const float* __restrict__ rs_tab,
                 const float* __restrict__ step /*[K,R_all]*/, int K, int k_per_cta, int64_t R_all,
                 const int32_t* __restrict__ n_rows_dev, int64_t C1, float qpos, float tie_eps,
                 int8_t* __restrict__ q /*[K,R_all,C1]*/) {
  extern __shared__ uint4 tile_dyn[];
  uint4 (*tile)[kGqCols / 8] = reinterpret_cast<uint4 (*)[kGqCols / 8]>(tile_dyn);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t col_blocks = (C1 + kGqCols - 1) / kGqCols;      // grid.x = column blocks x row tiles, columns fastest
  const int64_t c0 = (int64_t)(blockIdx.x % col_blocks) * kGqCols + lane * 16;
  const int64_t row0 = (int64_t)(blockIdx.x / col_blocks) * kRowRows;
  const int64_t R = (n_rows_dev != nullptr) ? (int64_t)*n_rows_dev : R_all;
  if (row0 >= R) return;
  const bool col_ok = c0 < C1;
  stage_tile(tile, src, row0, R, C1, c0, col_ok, warp, lane);
  if (!col_ok) return;                    // no warp-wide operation below
  const float tie_lim = 0.5f - tie_eps;
  const float2 magic2 = make_float2(kMagic, kMagic);
  const int k_begin = blockIdx.y * k_per_cta;
  const int k_end = min(K, k_begin + k_per_cta);
  for (int k = k_begin; k < k_end; ++k) {
    float2 m[8];
    load_mult16<kKind>(s_tab ? s_tab + (int64_t)k * C1 : nullptr, rs_tab ? rs_tab + (int64_t)k * C1 : nullptr, c0,
                       true, m);
#pragma unroll 1
    for (int p = 0; p < kRowRows / 8; ++p) {
      const int r = p * 8 + warp;
      const int64_t row = row0 + r;
      if (row >= R) break;
      const float st = step[(int64_t)k * R_all + row];
      const float inv = rcp_fast(st);
      const float2 inv2 = make_float2(inv, inv);
      float2 w[8];
      unpack16(tile[r][lane * 2], tile[r][lane * 2 + 1], w);
      float near = 0.0f;
      uint32_t tb[16];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float2 qv = mul2(mul2(w[j], m[j]), inv2);
        const float2 t = add2(qv, magic2);           // low mantissa byte = the code in two's complement
        const float2 df = sub2(qv, sub2(t, magic2));
        near = max3(near, fabsf(df.x), fabsf(df.y));
        tb[2 * j] = __float_as_uint(t.x);
        tb[2 * j + 1] = __float_as_uint(t.y);
      }
      uint4* dst = reinterpret_cast<uint4*>(q + ((int64_t)k * R_all + row) * C1 + c0);
      if (near > tie_lim) {
        float mf[16];
#pragma unroll
        for (int j = 0; j < 8; ++j) { mf[2 * j] = m[j].x; mf[2 * j + 1] = m[j].y; }
        codes16_exact(&tile[r][lane * 2], mf, st, qpos, dst);
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
}

template <int kKind>
static int launch_rows_two_pass(const uint16_t* src, const uint16_t* s, const float* rs, int K, int64_t R, int64_t C1, int bits,
                       int8_t* q, float* step, const int32_t* n_rows_dev, cudaStream_t st) {
  static OncePerDevice once;      // one per instantiation of this template
  int rc = once_per_device(once, [] {
    const cudaError_t e = cudaFuncSetAttribute(row_amax_kernel<kKind>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRowSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(row_codes_kernel<kKind>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRowSmem);
  });
  if (rc != TLQ_OK) return rc;
  const int sms = device_sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  const int64_t ctas = ceil_div(C1, kGqCols) * ceil_div(R, kRowRows);
  int64_t kchunks = ceil_div((int64_t)sms * 6, ctas);
  if (kchunks > K) kchunks = K;
  if (kchunks < 1) kchunks = 1;
  const int k_per_cta = (int)ceil_div(K, kchunks);
  kchunks = ceil_div(K, k_per_cta);
  const dim3 grid((unsigned)(ceil_div(C1, kGqCols) * ceil_div(R, kRowRows)), (unsigned)kchunks);
  const float qpos = (float)((1 << (bits - 1)) - 1);
  const float tie_eps = 4.0e-7f * (qpos + 1.0f);
  const int64_t n = (int64_t)K * R;
  TLQ_CUDA_TRY(cudaMemsetAsync(step, 0, (size_t)n * sizeof(float), st));
  row_amax_kernel<kKind><<<grid, kGqThreads, kRowSmem, st>>>(src, s, rs, K, k_per_cta, R, n_rows_dev, C1,
                                                      reinterpret_cast<int*>(step));
  rc = after_launch();
  if (rc != TLQ_OK) return rc;
  amax_to_step_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(step, n, qpos);
  if ((rc = after_launch()) != TLQ_OK) return rc;
  row_codes_kernel<kKind><<<grid, kGqThreads, kRowSmem, st>>>(src, s, rs, step, K, k_per_cta, R, n_rows_dev, C1, qpos, tie_eps, q);
  return after_launch();
}

// ------------------------------------------------------------------------------------------------
// The same quantizer with whole rows resident in one CTA: one launch instead of four, the source read
// from HBM once, and per element about half the instructions of the two tiled passes above.
//
// A CTA stages RB complete rows in shared memory (RB x C1 bf16, at most ~100 KB so that two CTAs share
// an SM) and walks its candidates in order.  A thread owns fixed 16-channel columns, so the candidate's
// per-channel multipliers are loaded once per column and serve all RB rows.  While the codes of
// candidate k are formed, the same unpacked values are multiplied by candidate k+1's multipliers and
// folded into running row maxima; the maxima are combined across the CTA (shuffles, then one warp per
// row), which yields step and 1/step of candidate k+1 for the next round.  Only the first candidate of
// a CTA needs a maximum pass of its own.  Per (row, candidate) the result is what the tiled passes
// give: max over channels of |value| is taken over the same binary32 products, the step is the same
// IEEE division, the codes come from the same straight-line arithmetic with the exact-division fix-up.
// ------------------------------------------------------------------------------------------------
constexpr int kFusedThreads = 256;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr size_t kFusedSmemBudget = 100 << 10;     // two CTAs per SM
constexpr size_t kFusedSmemLimit = 220 << 10;      // one CTA per SM: the widest row this kernel takes

template <int kKind, int RB>
__global__ void __launch_bounds__(kFusedThreads, 2)
row_quant_fused_kernel(const uint16_t* __restrict__ src, const uint16_t* __restrict__ s_tab,
                       const float* __restrict__ rs_tab, int K, int k_per_cta, int64_t R_all,
                       const int32_t* __restrict__ n_rows_dev, int64_t C1, float qpos, float tie_eps,
                       int8_t* __restrict__ q /*[K,R_all,C1]*/, float* __restrict__ step /*[K,R_all]*/) {
  extern __shared__ uint4 tile_dyn[];                 // [RB][C1 / 8]
  __shared__ float red[2][kFusedWarps][RB];           // per-warp row maxima of the candidate being prepared
  __shared__ float2 step_inv[2][RB];                  // (step, ~1/step) per row, double-buffered over candidates
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int64_t R = (n_rows_dev != nullptr) ? (int64_t)*n_rows_dev : R_all;    // rows beyond are not live
  const int64_t row0 = (int64_t)blockIdx.x * RB;
  if (row0 >= R) return;                              // the whole CTA leaves together
  const int nchunks = (int)(C1 >> 4);                 // 16-channel columns of a row
  const int row_u4 = nchunks * 2;                     // uint4 per staged row
  const int k_begin = blockIdx.y * k_per_cta;
  const int k_end = min(K, k_begin + k_per_cta);

  for (int i = t; i < RB * row_u4; i += kFusedThreads) {
    const int r = i / row_u4, c = i - r * row_u4;
    uint4 v = make_uint4(0, 0, 0, 0);                 // rows past the end count as zeros and store nothing
    if (row0 + r < R) v = ld_nc_16(src + (row0 + r) * C1 + (int64_t)c * 8);
    tile_dyn[i] = v;
  }
  // Narrow rows leave threads over: they are dealt out over row groups, thread (rg, column) taking rows rg, rg + groups, ...
  const int col_threads = nchunks < kFusedThreads ? nchunks : kFusedThreads;
  const int groups = kFusedThreads / col_threads;
  const int rg = t / col_threads;
  const int col0 = t - rg * col_threads;
  uint32_t row_mask = 0;
  if (rg < groups)
    for (int r = rg; r < RB; r += groups) row_mask |= 1u << r;
  __syncthreads();

  const float tie_lim = 0.5f - tie_eps;
  const float2 magic2 = make_float2(kMagic, kMagic);
  auto mult_rows = [&](int k, const uint16_t*& s_row, const float*& rs_row) {
    s_row = s_tab ? s_tab + (int64_t)k * C1 : nullptr;
    rs_row = rs_tab ? rs_tab + (int64_t)k * C1 : nullptr;
  };
  // Combine the threads' running maxima of candidate k into (step, 1/step) per row; buffer `par`.
  auto publish = [&](float (&am)[RB], int par, int k) {
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      float v = am[r];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
      if (lane == 0) red[par][warp][r] = v;
    }
    __syncthreads();
    if (warp < RB) {                                  // warp w finishes row w
      float v = lane < kFusedWarps ? red[par][lane][warp] : 0.0f;
#pragma unroll
      for (int off = kFusedWarps / 2; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
      if (lane == 0) {
        const float st = __fdiv_rn(fmaxf(v, TLQ_RANGE_FLOOR), qpos);
        step_inv[par][warp] = make_float2(st, rcp_fast(st));
        if (row0 + warp < R) step[(int64_t)k * R_all + row0 + warp] = st;
      }
    }
    __syncthreads();
  };

  float am[RB];
#pragma unroll
  for (int r = 0; r < RB; ++r) am[r] = 0.0f;
  if (row_mask != 0) {                                // the first candidate's maxima: a pass of its own
    const uint16_t* s_row; const float* rs_row;
    mult_rows(k_begin, s_row, rs_row);
    for (int ch = col0; ch < nchunks; ch += col_threads) {
      float2 m[8];
      load_mult16<kKind>(s_row, rs_row, (int64_t)ch * 16, true, m);
#pragma unroll
      for (int r = 0; r < RB; ++r) {
        if (!((row_mask >> r) & 1u)) continue;
        float2 w[8];
        unpack16(tile_dyn[r * row_u4 + ch * 2], tile_dyn[r * row_u4 + ch * 2 + 1], w);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float2 v = mul2(w[j], m[j]);
          am[r] = max3(am[r], fabsf(v.x), fabsf(v.y));
        }
      }
    }
  }
  publish(am, 0, k_begin);

  for (int k = k_begin; k < k_end; ++k) {
    const int par = (k - k_begin) & 1;
    const bool has_next = k + 1 < k_end;
    float st[RB], inv[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const float2 si = step_inv[par][r];
      st[r] = si.x; inv[r] = si.y;
      am[r] = 0.0f;
    }
    if (row_mask != 0) {
      const uint16_t* s_row; const float* rs_row;
      const uint16_t* s_next = nullptr; const float* rs_next = nullptr;
      mult_rows(k, s_row, rs_row);
      if (has_next) mult_rows(k + 1, s_next, rs_next);
      for (int ch = col0; ch < nchunks; ch += col_threads) {
        float2 m[8], m2[8];
        load_mult16<kKind>(s_row, rs_row, (int64_t)ch * 16, true, m);
        if (has_next) load_mult16<kKind>(s_next, rs_next, (int64_t)ch * 16, true, m2);
#pragma unroll
        for (int r = 0; r < RB; ++r) {
          if (!((row_mask >> r) & 1u)) continue;
          const uint4* tile16 = &tile_dyn[r * row_u4 + ch * 2];
          float2 w[8];
          unpack16(tile16[0], tile16[1], w);
          if (has_next) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float2 v = mul2(w[j], m2[j]);
              am[r] = max3(am[r], fabsf(v.x), fabsf(v.y));
            }
          }
          const int64_t row = row0 + r;
          if (row >= R) continue;
          const float2 inv2 = make_float2(inv[r], inv[r]);
          float near = 0.0f;
          uint32_t tb[16];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float2 qv = mul2(mul2(w[j], m[j]), inv2);
            const float2 tt = add2(qv, magic2);          // low mantissa byte = the code in two's complement
            const float2 df = sub2(qv, sub2(tt, magic2));
            near = max3(near, fabsf(df.x), fabsf(df.y));
            tb[2 * j] = __float_as_uint(tt.x);
            tb[2 * j + 1] = __float_as_uint(tt.y);
          }
          uint4* dst = reinterpret_cast<uint4*>(q + ((int64_t)k * R_all + row) * C1 + (int64_t)ch * 16);
          if (near > tie_lim) {
            float mf[16];
#pragma unroll
            for (int j = 0; j < 8; ++j) { mf[2 * j] = m[j].x; mf[2 * j + 1] = m[j].y; }
            codes16_exact(tile16, mf, st[r], qpos, dst);
          } else {
            uint32_t pk[4];
#pragma unroll
            for (int g = 0; g < 4; ++g)
              pk[g] = __byte_perm(__byte_perm(tb[4 * g], tb[4 * g + 1], 0x0040),
                                  __byte_perm(tb[4 * g + 2], tb[4 * g + 3], 0x0040), 0x5410);
            *dst = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
    }
    if (has_next) publish(am, par ^ 1, k + 1);
  }
}

template <int kKind, int RB>
static int launch_rows_fused(const uint16_t* src, const uint16_t* s, const float* rs, int K, int64_t R, int64_t C1,
                             int bits, int8_t* q, float* step, const int32_t* n_rows_dev, cudaStream_t st) {
  static OncePerDevice once;
  int rc = once_per_device(once, [] {
    return cudaFuncSetAttribute(row_quant_fused_kernel<kKind, RB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)kFusedSmemLimit);
  });
  if (rc != TLQ_OK) return rc;
  const int sms = device_sm_count();
  if (sms <= 0) return TLQ_ERR_CUDA;
  const int64_t row_blocks = ceil_div(R, RB);
  int64_t kchunks = ceil_div((int64_t)sms * 12, row_blocks);     // several work units per resident CTA
  if (kchunks > K) kchunks = K;
  if (kchunks < 1) kchunks = 1;
  const int k_per_cta = (int)ceil_div(K, kchunks);
  kchunks = ceil_div(K, k_per_cta);
  const dim3 grid((unsigned)row_blocks, (unsigned)kchunks);
  const float qpos = (float)((1 << (bits - 1)) - 1);
  const float tie_eps = 4.0e-7f * (qpos + 1.0f);
  const size_t smem = (size_t)RB * (size_t)C1 * 2;
  row_quant_fused_kernel<kKind, RB><<<grid, kFusedThreads, smem, st>>>(src, s, rs, K, k_per_cta, R, n_rows_dev, C1, qpos,
                                                                  tie_eps, q, step);
  return after_launch();
}

// Rows per CTA of the whole-row kernel: the largest of 8, 4, 2, 1 whose rows fit the shared-memory budget; rows too
// wide even for one per CTA go through the two tiled passes.
template <int kKind>
static int launch_rows(const uint16_t* src, const uint16_t* s, const float* rs, int K, int64_t R, int64_t C1, int bits,
                       int8_t* q, float* step, const int32_t* n_rows_dev, cudaStream_t st) {
  const size_t row_bytes = (size_t)C1 * 2;
  if ((C1 & 15) != 0 || row_bytes > kFusedSmemLimit)
    return launch_rows_two_pass<kKind>(src, s, rs, K, R, C1, bits, q, step, n_rows_dev, st);
  if (8 * row_bytes <= kFusedSmemBudget) return launch_rows_fused<kKind, 8>(src, s, rs, K, R, C1, bits, q, step, n_rows_dev, st);
  if (4 * row_bytes <= kFusedSmemBudget) return launch_rows_fused<kKind, 4>(src, s, rs, K, R, C1, bits, q, step, n_rows_dev, st);
  if (2 * row_bytes <= kFusedSmemBudget) return launch_rows_fused<kKind, 2>(src, s, rs, K, R, C1, bits, q, step, n_rows_dev, st);
  return launch_rows_fused<kKind, 1>(src, s, rs, K, R, C1, bits, q, step, n_rows_dev, st);
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
