// TMA / mbarrier device helpers and the host-side tensor-map cache shared by the tensor-core kernels.
// No cluster multicast is used anywhere: every copy is CTA-local.
#pragma once

#include <cuda.h>

#include <map>
#include <mutex>
#include <tuple>

#include "common.cuh"

namespace nz {

constexpr long long kWaitCycles = 2000000000ll;     // about one second of SM clock: bound of every barrier wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait; false = gave up.  The clock is read only once the first try has failed: a wait that is already
// satisfied costs one instruction, which matters to the single threads that issue every copy and every MMA.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > kWaitCycles) return false;
  }
}
// The same, giving up early when another role of the CTA has raised the abort flag (so one expired wait does not
// make every other role sit out its own full bound).
__device__ __forceinline__ bool mbar_wait_or_abort(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag || clock64() - t0 > kWaitCycles) return false;
  }
}
// One lane waits for the barrier and tells the rest of the warp (which sleeps at the shuffle instead of polling): 32
// polling lanes are 32 times the instructions, taken from the warps of the SM that have arithmetic to issue.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, int lane) {
  int ok = 1;
  if (lane == 0) ok = mbar_wait_or_abort(bar, parity, abort_flag) ? 1 : 0;
  __syncwarp();                                    // orders the other lanes' later accesses after lane 0's acquire
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// Fetches a tensor map into the descriptor cache ahead of its first copy (the map is a kernel parameter: this reads
// nothing an earlier kernel wrote, so it may run before the dependency wait).
__device__ __forceinline__ void tma_prefetch_map(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// x = innermost coordinate (elements; x * element size must be a multiple of 16 bytes), y = row coordinate.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tma_encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    cudaGetLastError();
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Index of the current device, clamped to the tables below.
constexpr int kMaxDevices = 64;
inline int current_device() {
  int d = 0;
  if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDevices) d = 0;
  cudaGetLastError();
  return d;
}

// One-time set-up per device (a function attribute belongs to the device's context, not to the process): run(f) calls f
// the first time it is reached with a given device current, under a lock, so that no other host thread launches before
// the set-up has been made.
struct PerDeviceOnce {
  std::mutex mu;
  bool done[kMaxDevices] = {};
  template <typename F> void run(F&& f) {
    std::lock_guard<std::mutex> g(mu);
    const int d = current_device();
    if (!done[d]) { f(); done[d] = true; }
  }
};

// 2-D bf16 row-major [rows, cols] with row pitch ld (elements); box = 64 columns x box_rows rows, 128-byte swizzle.
// The map is returned by value (it is a kernel parameter anyway); encoded maps are kept in a process-wide table behind a
// lock, keyed by everything that goes into them, and the table is emptied when it has grown past a few thousand entries.
inline bool tma_map_bf16(const void* ptr, long long rows, long long cols, long long ld, int box_rows, CUtensorMap* out) {
  using Key = std::tuple<const void*, long long, long long, long long, int>;
  static std::map<Key, CUtensorMap> cache;
  static std::mutex mu;
  if (!tma_encode_fn()) return false;
  const Key key{ptr, rows, cols, ld, box_rows};
  std::lock_guard<std::mutex> g(mu);
  auto it = cache.find(key);
  if (it != cache.end()) { *out = it->second; return true; }
  CUtensorMap tm;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  if (tma_encode_fn()(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  if (cache.size() > 8192) cache.clear();
  cache.emplace(key, tm);
  *out = tm;
  return true;
}

}  // namespace nz
