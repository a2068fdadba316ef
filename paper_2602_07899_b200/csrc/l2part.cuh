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
int l2_partition_read(L2PartMap* out);      // host copy of the current device's table (synchronises the device)

// This CTA's share of a (candidate, output tile, token tile) space.
//
// Whole grid (part < 0): items are (candidate, position in the raster over all token and output tiles).
// One L2 partition (part 0 or 1): the token tiles are cut between the partitions in proportion to their SM counts.
// The exact proportion is rarely a whole number of tiles (72 of 148 SMs want 15.57 of 32 tiles), and rounding it
// would leave one partition several percent more rounds than the other, so the cut moves from candidate to
// candidate: after k candidates partition 0 has had floor(k * mtiles * n0 / n) token tiles in total, i.e. 15 or 16
// per candidate in the right mix.  Inside a candidate the partition walks its token tiles fastest, then the output
// tiles.
struct TileWalk {
  int first, stride;        // work items first, first + stride, ... below `count`
  int part;                 // -1: the whole grid shares one walk
  int mtiles, otiles;
  int n0, n;                // SMs of partition 0, SMs in total
  int64_t count;            // items of this walk
  TileRaster raster;        // whole-grid walk only: over (mtiles, otiles)

  __host__ __device__ int64_t tiles0_before(int k) const { return ((int64_t)k * mtiles * n0) / n; }   // partition 0's token tiles
  __host__ __device__ int64_t base(int k) const {            // items before candidate k
    if (part < 0) return (int64_t)k * otiles * mtiles;
    const int64_t t0 = tiles0_before(k);
    return (int64_t)otiles * (part == 0 ? t0 : (int64_t)k * mtiles - t0);
  }
  // `k` is the caller's running candidate: items only ever increase, so it is advanced, never searched
  __host__ __device__ void decode(int64_t item, int& k, int& mt, int& ot) const {
    while (item >= base(k + 1)) ++k;
    const int64_t r = item - base(k);
    if (part < 0) {
      raster.decode(r, mt, ot);
    } else {
      const int cut = (int)(tiles0_before(k + 1) - tiles0_before(k));
      const int mc = part == 0 ? cut : mtiles - cut;
      ot = (int)(r / mc);
      mt = (part == 0 ? 0 : cut) + (int)(r - (int64_t)ot * mc);
    }
  }
};

// The walk of slot `rank` of `n_part` in partition `part` (-1: slot `rank` of a whole grid of `grid` CTAs).  Pure
// integer arithmetic, shared by the kernels and by the host-side coverage check (tlq_debug_tile_walk).
__host__ __device__ inline void fill_tile_walk(TileWalk& w, int part, int rank, int n_part, int mtiles, int otiles,
                                               int K, bool blocked, int block_a, int n0, int grid) {
  w.first = rank;
  w.stride = n_part;
  w.part = part;
  w.mtiles = mtiles;
  w.otiles = otiles;
  w.n0 = part < 0 ? 1 : n0;
  w.n = part < 0 ? 1 : grid;
  w.raster.mtiles = mtiles;
  w.raster.otiles = otiles;
  if (blocked) {
    w.raster.a = block_a;
    w.raster.b = grid / block_a > 0 ? grid / block_a : 1;
  } else {
    w.raster.a = mtiles > 0 ? mtiles : 1;
    w.raster.b = 1;
  }
  w.count = w.base(K);
}

// Called by ONE thread of every CTA of the grid, exactly once per launch.  `mtiles` token tiles, `otiles` output
// tiles, K candidates; `blocked` says whether the whole-grid walk goes by blocks of `block_a` token tiles (then the
// partitions are not used: see the launcher).  `hdr->slot_count` must have been zeroed before the launch.
__device__ inline void make_tile_walk(const L2PartMap* map, WorkspaceHeader* hdr, int mtiles, int otiles, int K,
                                      bool blocked, int block_a, TileWalk& w) {
  const int grid = (int)gridDim.x;
  int part = -1, rank = (int)blockIdx.x, n_part = grid;
  if (map != nullptr && map->valid != 0 && map->n_sms == grid && mtiles >= 4 && !blocked) {
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
  fill_tile_walk(w, part, rank, n_part, mtiles, otiles, K, blocked, block_a, part < 0 ? 1 : map->count[0], grid);
}

}  // namespace tlq
