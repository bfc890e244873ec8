// Eq. 4 (mixed-radix packing) and Eq. 5 (the set V of valid IDs) on the GPU.
//
// V is an open-addressing hash set of 64-bit packed keys.  Slots are grouped in buckets of 4 (32 bytes = one
// DRAM sector); a key hashes to a bucket and probes linearly over buckets.  Insertion takes the first empty
// slot of the first non-full bucket on its probe path, so a lookup can stop at the first bucket that still
// has an empty slot.  Stand-alone lookups are warp-cooperative: a tile of 4 lanes reads one bucket with one
// 8-byte load per lane and votes.  All walks are bounded by kMaxProbeBuckets.
#include "common.cuh"

namespace nz {

__global__ void hs_clear_kernel(unsigned long long* slots, unsigned long long n_slots) {
  unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
  unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  for (; i < n_slots; i += stride) slots[i] = kEmptyKey;
}

__global__ void hs_pack_kernel(LevelInfo li, const int* __restrict__ codes, unsigned long long n,
                               unsigned long long* __restrict__ keys, int* status) {
  unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
  if (i >= n) return;
  int c[kMaxLevels];
  bool bad = false;
  for (int l = 0; l < li.L; ++l) {
    c[l] = codes[i * li.L + l];
    bad |= (c[l] < 0 || c[l] >= li.T[l]);
  }
  if (bad) { atomicOr(status, kStBadCode); keys[i] = kEmptyKey; return; }
  keys[i] = pack_key(li, c);
}

__global__ void hs_insert_kernel(LevelInfo li, HashSetView hs, const int* __restrict__ codes, unsigned long long n,
                                 unsigned long long* n_unique, int* status) {
  unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
  bool inserted = false;
  if (i < n) {
    int c[kMaxLevels];
    bool bad = false;
    for (int l = 0; l < li.L; ++l) {
      c[l] = codes[i * li.L + l];
      bad |= (c[l] < 0 || c[l] >= li.T[l]);
    }
    if (bad) {
      atomicOr(status, kStBadCode);
    } else {
      const unsigned long long key = pack_key(li, c);
      unsigned long long b = hs_bucket(key, hs.n_buckets);
      bool done = false;
      for (int step = 0; step < kMaxProbeBuckets && !done; ++step) {
        unsigned long long* bucket = hs.slots + b * kBucketSlots;
        for (int s = 0; s < kBucketSlots && !done; ++s) {
          unsigned long long cur = *reinterpret_cast<volatile unsigned long long*>(bucket + s);
          if (cur == kEmptyKey) cur = atomicCAS(bucket + s, kEmptyKey, key), inserted = (cur == kEmptyKey);
          if (inserted || cur == key) done = true;     // placed now, or already present (duplicate tuple)
        }
        if (++b == hs.n_buckets) b = 0;
      }
      if (!done) atomicOr(status, kStHashFull);
    }
  }
  unsigned m = __ballot_sync(0xffffffffu, inserted);
  if ((threadIdx.x & 31) == 0 && m) atomicAdd(n_unique, (unsigned long long)__popc(m));
}

// 4 lanes per key; every lane of the warp stays in the loop until all 8 tiles of the warp have finished.
__global__ void hs_probe_kernel(HashSetView hs, const unsigned long long* __restrict__ keys, unsigned long long n,
                                uint8_t* __restrict__ found) {
  const unsigned long long gid = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
  const unsigned long long ki = gid / kBucketSlots;
  const int sub = threadIdx.x & (kBucketSlots - 1);
  const int tile_shift = (threadIdx.x & 31) & ~(kBucketSlots - 1);
  const bool in_range = ki < n;
  const unsigned long long key = in_range ? __ldg(keys + ki) : 0ull;
  unsigned long long b = hs_bucket(key, hs.n_buckets);
  bool active = in_range, hit = false;
  for (int step = 0; step < kMaxProbeBuckets; ++step) {
    if (!__any_sync(0xffffffffu, active)) break;
    unsigned long long v = active ? __ldg(hs.slots + b * kBucketSlots + sub) : kEmptyKey;
    unsigned match = (__ballot_sync(0xffffffffu, active && v == key) >> tile_shift) & 0xFu;
    unsigned empty = (__ballot_sync(0xffffffffu, active && v == kEmptyKey) >> tile_shift) & 0xFu;
    if (active) {
      if (match) { hit = true; active = false; }
      else if (empty) active = false;
      else if (++b == hs.n_buckets) b = 0;
    }
  }
  if (in_range && sub == 0) found[ki] = hit ? 1 : 0;
}

void launch_hs_clear(HashSetView hs, cudaStream_t st) {
  LaunchScope ls(kcHash, st);
  hs_clear_kernel<<<148 * 8, 512, 0, st>>>(hs.slots, hs.n_buckets * kBucketSlots);
}
void launch_hs_pack(const LevelInfo& li, const int* codes, unsigned long long n, unsigned long long* keys, int* status,
                    cudaStream_t st) {
  if (!n) return;
  LaunchScope ls(kcHash, st);
  hs_pack_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(li, codes, n, keys, status);
}
void launch_hs_insert(const LevelInfo& li, HashSetView hs, const int* codes, unsigned long long n,
                      unsigned long long* n_unique, int* status, cudaStream_t st) {
  if (!n) return;
  LaunchScope ls(kcHash, st);
  hs_insert_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(li, hs, codes, n, n_unique, status);
}
void launch_hs_probe(HashSetView hs, const unsigned long long* keys, unsigned long long n, uint8_t* found,
                     cudaStream_t st) {
  if (!n) return;
  unsigned long long threads = n * kBucketSlots;
  LaunchScope ls(kcHash, st);
  hs_probe_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(hs, keys, n, found);
}

}  // namespace nz
