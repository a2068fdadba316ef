// Which half of the L2 each SM sits next to, and a tile walk that uses it.
//
// The L2 of this GPU is two partitions (one per die).  A line read by SMs of both partitions ends up in both, so
// data shared by every SM (the activation tiles of the search GEMM, which all CTAs of a wave re-read) only has half
// of the nominal capacity.  Measured with the fused bf16 GEMM of a 7B-class gate projection: the 59 MB of
// activations should stay resident beside the streamed weights, but 40 % of them were fetched from HBM again in
// every wave.  The remedy is to give each partition's CTAs their own token tiles, so that a partition only ever
// holds its own share of the activations.
//
// The assignment of SMs to partitions is not documented; it is measured once per device (l2part.cu) and kept in a
// small table in device memory.  Correctness never depends on it: CTAs claim numbered slots, every slot is claimed
// exactly once wherever the CTA happens to run, and a table that could not be measured just means the plain walk.
#pragma once

#include "common.cuh"

namespace tlq {

constexpr int kMaxSmIds = 256;

struct L2PartMap {
  int32_t valid;            // 1 once the measurement succeeded and split the SMs into two clear groups
  int32_t n_sms;            // SMs measured (= CTAs of a one-CTA-per-SM grid)
  int32_t count[2];         // SMs per partition
  uint8_t part[kMaxSmIds];  // partition of each %smid
};

// Device address of this device's table, measuring it first if that has not happened yet and `scratch` (device
// memory nobody else uses until the stream reaches the caller's next kernel) is large enough; nullptr on error.
// A table that has not been measured yet has valid == 0.
size_t l2_partition_scratch_bytes();
const L2PartMap* l2_partition_map(void* scratch, size_t scratch_bytes, cudaStream_t st);

// This CTA's share of a (candidate, output tile, token tile) space.
struct TileWalk {
  int first, stride;        // work items first, first + stride, ... below `count`
  int m_first, m_count;     // token tiles [m_first, m_first + m_count) of this CTA's partition
  int64_t count;            // K * otiles * m_count
  int64_t tiles_per_k;      // otiles * m_count
  TileRaster raster;        // over (m_count, otiles)
  __device__ void decode(int64_t item, int& k, int& mt, int& ot) const {
    k = (int)(item / tiles_per_k);
    int ml;
    raster.decode(item - (int64_t)k * tiles_per_k, ml, ot);
    mt = m_first + ml;
  }
};

// Called by ONE thread of every CTA of the grid, exactly once per launch.  `mtiles` token tiles, `otiles` output
// tiles, K candidates; `blocked` says whether the walk inside a partition goes by blocks of `block_a` token tiles.
// `hdr->slot_count` must have been zeroed before the launch.
__device__ inline void make_tile_walk(const L2PartMap* map, WorkspaceHeader* hdr, int mtiles, int otiles, int K,
                                      bool blocked, int block_a, TileWalk& w) {
  const int grid = (int)gridDim.x;
  int part = -1, rank = (int)blockIdx.x, n_part = grid;
  if (map != nullptr && map->valid != 0 && map->n_sms == grid && mtiles >= 4) {
    unsigned smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    int p = smid < (unsigned)kMaxSmIds ? (int)map->part[smid] : 0;
    int r = atomicAdd(&hdr->slot_count[p], 1);
    if (r >= map->count[p]) {       // more CTAs landed in this partition than it has SMs: take a slot of the other one
      p ^= 1;
      r = atomicAdd(&hdr->slot_count[p], 1);
    }
    if (r < map->count[p]) {
      part = p; rank = r; n_part = map->count[p];
    } else {                        // cannot happen while slots == CTAs; results would have holes, so say so
      hdr->where = 41;
      hdr->status = TLQ_ERR_TIMEOUT;
    }
  }
  w.first = rank;
  w.stride = n_part;
  if (part < 0) {
    w.m_first = 0;
    w.m_count = mtiles;
  } else {
    int m0 = (int)(((int64_t)mtiles * map->count[0] + grid / 2) / grid);     // token tiles in proportion to the SMs
    m0 = m0 < 1 ? 1 : (m0 > mtiles - 1 ? mtiles - 1 : m0);
    w.m_first = part == 0 ? 0 : m0;
    w.m_count = part == 0 ? m0 : mtiles - m0;
  }
  w.tiles_per_k = (int64_t)otiles * w.m_count;
  w.count = (int64_t)K * w.tiles_per_k;
  w.raster.mtiles = w.m_count;
  w.raster.otiles = otiles;
  if (blocked) {
    w.raster.a = block_a;
    w.raster.b = n_part / block_a > 0 ? n_part / block_a : 1;
  } else {
    w.raster.a = w.m_count > 0 ? w.m_count : 1;
    w.raster.b = 1;
  }
}

}  // namespace tlq
