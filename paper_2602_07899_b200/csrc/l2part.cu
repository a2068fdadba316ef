// Measuring which L2 partition each SM sits next to (see l2part.cuh for why).
//
// Method: one CTA per SM, the CTAs take turns.  The first one writes and reads back a set of lines for every CTA, which
// leaves each line in its home L2 slice and in the first CTA's own partition.  Every CTA then times one load of each of ITS lines,
// which nobody but the first CTA has touched.  For a CTA in the first CTA's partition all of them are ordinary
// L2 hits (250-350 cycles).  For a CTA in the other partition about half are (the lines whose home slice is on its
// own side) and the other half come across from the far partition (about 650 cycles).  So the number of slow loads
// separates the SMs into two groups with a wide margin, or the measurement is declared unusable.
// Every wait is bounded; nothing here can hang or fault: all accesses lie inside the scratch buffer.
#include "l2part.cuh"

namespace tlq {

namespace {

constexpr int kLines = 32;                    // timed lines per CTA
constexpr int kLineStride = 4096 + 128;       // bytes between lines: spreads them over the slices
constexpr long long kTurnLimitCycles = 400000000LL;   // ~0.2 s: a whole probe takes about a millisecond

static __device__ __align__(256) L2PartMap g_l2_part_map;

struct ProbeScratch {          // layout of the caller's scratch memory
  int32_t turn;
  int32_t timeouts;
  int32_t pad[62];
  int32_t smid[kMaxSmIds];
  uint32_t lat[kMaxSmIds * kLines];
};
constexpr size_t kLinesOffset = (sizeof(ProbeScratch) + 4095) / 4096 * 4096;

__global__ void l2_probe_kernel(ProbeScratch* ps, uint32_t* lines) {
  extern __shared__ uint8_t occupy_the_sm[];      // sized so that one CTA fills an SM
  if (threadIdx.x != 0) return;
  const int r = (int)blockIdx.x;
  unsigned smid;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
  ps->smid[r] = (int)smid;
  volatile int32_t* turn = &ps->turn;
  const long long t0 = clock64();
  while (*turn != r) {
    if (clock64() - t0 > kTurnLimitCycles) {
      atomicAdd(&ps->timeouts, 1);
      return;
    }
  }
  constexpr int kWordsPerLine = kLineStride / 4;
  uint32_t acc = 0;
  if (r == 0) {
    // The first CTA prepares every CTA's lines: a store leaves no stale copy in either partition, the load after it
    // brings the line next to this SM as well as into its home slice.
    for (int j = 0; j < kLines * (int)gridDim.x; ++j)
      asm volatile("st.global.cg.u32 [%0], %1;" ::"l"(lines + (size_t)j * kWordsPerLine), "r"(j) : "memory");
    __threadfence();
    for (int j = 0; j < kLines * (int)gridDim.x; ++j) {
      uint32_t v;
      asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(v) : "l"(lines + (size_t)j * kWordsPerLine) : "memory");
      acc += v;
    }
  }
  for (int j = 0; j < kLines; ++j) {
    const uint32_t* p = lines + (size_t)(r * kLines + j) * kWordsPerLine;
    unsigned long long a, b;
    uint32_t v;
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(a)::"memory");
    // the xor needs the loaded value, and instructions issue in order: the second clock is read after the load returned
    asm volatile("{\n\t.reg .u32 t;\n\tld.global.cg.u32 t, [%2];\n\txor.b32 %1, t, %3;\n\tmov.u64 %0, %%clock64;\n\t}"
                 : "=l"(b), "=r"(v) : "l"(p), "r"(r + j) : "memory");
    acc += v;
    ps->lat[r * kLines + j] = (uint32_t)(b - a);
  }
  if (acc == 0xDEADBEEFu) ps->pad[0] = 1;         // keeps the loads alive
  __threadfence();
  *turn = r + 1;
}

// One thread: turn the latencies into the table, or leave it invalid.
__global__ void l2_classify_kernel(const ProbeScratch* ps, int n_sms, L2PartMap* map) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  map->valid = 0;
  map->n_sms = n_sms;
  map->count[0] = map->count[1] = 0;
  for (int i = 0; i < kMaxSmIds; ++i) map->part[i] = 0;
  if (ps->timeouts != 0 || ps->turn != n_sms || n_sms > kMaxSmIds) return;
  // reference: the first CTA's own loads are all near hits; take their median
  uint32_t ref[kLines];
  for (int j = 0; j < kLines; ++j) ref[j] = ps->lat[j];
  for (int i = 1; i < kLines; ++i)
    for (int j = i; j > 0 && ref[j - 1] > ref[j]; --j) { const uint32_t t = ref[j]; ref[j] = ref[j - 1]; ref[j - 1] = t; }
  const uint32_t slow = ref[kLines / 2] + ref[kLines / 2] / 2;      // 1.5 x a near hit
  bool clear = true;
  for (int r = 0; r < n_sms; ++r) {
    int n_slow = 0;
    for (int j = 0; j < kLines; ++j) n_slow += ps->lat[r * kLines + j] > slow;
    const int smid = ps->smid[r];
    if (smid < 0 || smid >= kMaxSmIds) { clear = false; break; }
    int p;
    if (n_slow <= 1) p = 0;
    else if (n_slow >= kLines / 4) p = 1;
    else { clear = false; break; }                                  // neither group: do not trust the measurement
    map->part[smid] = (uint8_t)p;
    map->count[p] += 1;
  }
  // two groups of comparable size, every SM seen once
  if (clear && map->count[0] + map->count[1] == n_sms && map->count[0] * 4 >= n_sms && map->count[1] * 4 >= n_sms)
    map->valid = 1;
}

}  // namespace

size_t l2_partition_scratch_bytes() { return kLinesOffset + (size_t)kMaxSmIds * kLines * kLineStride; }

const L2PartMap* l2_partition_map(void* scratch, size_t scratch_bytes, cudaStream_t st) {
  static L2PartMap* address[kMaxDevices] = {};
  static bool measured[kMaxDevices] = {};
  const int dev = current_device_index();
  if (dev < 0) return nullptr;
  if (address[dev] == nullptr) {      // in host code the array's name stands for the symbol, not for an address
    L2PartMap* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_l2_part_map) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return nullptr;
    }
    address[dev] = p;
  }
  if (!measured[dev] && scratch != nullptr && scratch_bytes >= l2_partition_scratch_bytes() &&
      (reinterpret_cast<uintptr_t>(scratch) & 255u) == 0) {
    const int sms = device_sm_count();
    constexpr int kSmem = 200 << 10;      // more than half of an SM's shared memory: one CTA per SM
    if (sms > 0 && sms <= kMaxSmIds &&
        cudaFuncSetAttribute(l2_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) == cudaSuccess &&
        cudaMemsetAsync(scratch, 0, sizeof(ProbeScratch), st) == cudaSuccess) {
      ProbeScratch* ps = reinterpret_cast<ProbeScratch*>(scratch);
      uint32_t* lines = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(scratch) + kLinesOffset);
      l2_probe_kernel<<<sms, 32, kSmem, st>>>(ps, lines);
      if (after_launch() == TLQ_OK) {
        l2_classify_kernel<<<1, 32, 0, st>>>(ps, sms, address[dev]);
        if (after_launch() == TLQ_OK) measured[dev] = true;
      }
    } else {
      cudaGetLastError();
    }
  }
  return address[dev];
}

// Host copy of the current device's table (synchronises the device); TLQ_ERR_CUDA on failure.
int l2_partition_read(L2PartMap* out) {
  if (cudaDeviceSynchronize() != cudaSuccess) return TLQ_ERR_CUDA;
  if (cudaMemcpyFromSymbol(out, g_l2_part_map, sizeof(L2PartMap)) != cudaSuccess) {
    cudaGetLastError();
    return TLQ_ERR_CUDA;
  }
  return TLQ_OK;
}

}  // namespace tlq
