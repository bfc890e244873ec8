// Eq. 4 (mixed-radix packing) and Eq. 5 (the set V of valid IDs) on the GPU.
//
// V is an open-addressing hash set of 64-bit packed keys.  Slots are grouped in buckets of 4 (32 bytes = one
// DRAM sector); a key hashes to a bucket and probes linearly over buckets.  Insertion takes the first empty
// slot of the first non-full bucket on its probe path, so a lookup can stop at the first bucket that still
// has an empty slot.  A lookup is one thread reading whole buckets (two 16-byte loads of one sector); stand-alone
// lookups take two keys per thread so that both sectors are in flight together.  All walks are bounded by
// kMaxProbeBuckets.
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

// A thread answers kProbeKeysPerThread keys: it loads them (coalesced: thread t of the block takes keys t, t + 256, ...),
// asks for all their home buckets at once -- one 32-byte sector each, the only traffic that is not streaming -- and only
// then compares.  The kernel is bound by the number of random sectors in flight.  Measured on 2^26 keys, half of them
// hits: 1, 2, 4, 8 keys per thread give 106, 108, 85, 55 G probes/s on a table that fits L2 and 77, 77, 61, 37 on one
// that does not (four lanes per key, each loading one slot: 43 and 34).
constexpr int kProbeKeysPerThread = 2;
__global__ void __launch_bounds__(256) hs_probe_kernel(HashSetView hs, const unsigned long long* __restrict__ keys,
                                                       unsigned long long n, uint8_t* __restrict__ found) {
  const unsigned long long base = (unsigned long long)blockIdx.x * (256u * kProbeKeysPerThread) + threadIdx.x;
  unsigned long long k[kProbeKeysPerThread];
  bool want[kProbeKeysPerThread], hit[kProbeKeysPerThread];
#pragma unroll
  for (int j = 0; j < kProbeKeysPerThread; ++j) {
    const unsigned long long i = base + 256ull * j;
    want[j] = i < n;
    k[j] = want[j] ? __ldg(keys + i) : 0ull;
    hit[j] = false;
  }
  hs_contains_many<kProbeKeysPerThread>(hs, k, want, hit);
#pragma unroll
  for (int j = 0; j < kProbeKeysPerThread; ++j) {
    const unsigned long long i = base + 256ull * j;
    if (want[j]) found[i] = hit[j] ? 1 : 0;
  }
}

// One thread per item: for every n in [0, L) it claims (or finds) the slot of the item's n-code prefix in region n and sets
// the bit of the item's next code.  The bit is tested first: the few prefixes at the top of the tree are shared by
// millions of items, whose atomics on the same word would otherwise serialise.
__global__ void pm_insert_kernel(LevelInfo li, PrefixMapView pm, const int* __restrict__ codes, unsigned long long n, int* status) {
  const unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
  if (i >= n) return;
  int c[kMaxLevels];
  for (int l = 0; l < li.L; ++l) {
    c[l] = codes[i * li.L + l];
    if (c[l] < 0 || c[l] >= li.T[l]) return;        // hs_insert_kernel has reported it
  }
  unsigned long long p = 0;
  for (int lv = 0; lv < li.L; ++lv) {               // prefix of lv codes, next code c[lv]
    if (lv > 0) p += (unsigned long long)c[lv - 1] * li.mult[lv - 1];
    const int t = c[lv];
    const unsigned long long ns = pm.level_slots[lv];
    unsigned long long* region = pm.slots + pm.level_off[lv] * pm.stride;
    unsigned long long s = __umul64hi(hs_mix(p), ns);
    bool done = false;
    for (int step = 0; step < kMaxProbeBuckets && !done; ++step) {
      unsigned long long* slot = region + s * pm.stride;
      unsigned long long cur = *reinterpret_cast<volatile unsigned long long*>(slot);
      if (cur == 0ull) cur = atomicCAS(slot, 0ull, p + 1);
      if (cur == 0ull || cur == p + 1) {
        unsigned long long* word = slot + 1 + (t >> 6);
        const unsigned long long bit = 1ull << (t & 63);
        if (!(*reinterpret_cast<volatile unsigned long long*>(word) & bit)) atomicOr(word, bit);
        done = true;
      }
      if (++s == ns) s = 0;
    }
    if (!done) { atomicOr(status, kStHashFull); return; }
  }
}

void launch_pm_build(const LevelInfo& li, PrefixMapView pm, const int* codes, unsigned long long n, int* status, cudaStream_t st) {
  if (!pm.slots) return;
  cudaMemsetAsync(pm.slots, 0, (size_t)pm.n_slots * pm.stride * sizeof(unsigned long long), st);
  if (!n) return;
  LaunchScope ls(kcHash, st);
  pm_insert_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(li, pm, codes, n, status);
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
  const unsigned long long per_block = 256ull * kProbeKeysPerThread;
  LaunchScope ls(kcHash, st);
  hs_probe_kernel<<<(unsigned)((n + per_block - 1) / per_block), 256, 0, st>>>(hs, keys, n, found);
}

}  // namespace nz
