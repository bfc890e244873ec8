// Shared declarations of the decode library's translation units (device helpers, argument structs,
// kernel launchers).  Everything here is internal; the public surface is include/nezha.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "nezha.h"

namespace nz {

constexpr int kMaxLevels = NEZHA_MAX_LEVELS;
constexpr int kBucketSlots = 4;                  // 4 x 8 B = one 32-byte sector per bucket
constexpr unsigned long long kEmptyKey = ~0ull;  // never a packed key: prod(T) < 2^64 - 1
constexpr int kMaxProbeBuckets = 4096;           // bound of every probe / insert walk

// bits of the device status word
enum : int { kStHashFull = 1, kStBadCode = 2, kStInternal = 4 };

// Kernel classes for the launch counter and the optional CUDA-event timing (see nezha_profile_*).
enum KernelClass : int {
  kcGemm = 0, kcAttention, kcSelect, kcNorm, kcRope, kcEmbed, kcSwiglu, kcDraftGlue, kcNodes, kcAccept, kcHash, kcMisc,
  kcCount
};
static_assert(kcCount <= NEZHA_PROFILE_CLASSES, "profile classes");
// Wrap the launch(es) of one kernel class: counts them and, when profiling is on, brackets them with events.
struct LaunchScope {
  LaunchScope(int cls, cudaStream_t st, int n_launches = 1);
  ~LaunchScope();
  int cls; cudaStream_t st; int slot;
};

// --------------------------------------------------------------------------------------------------
// programmatic dependent launch: the kernels of the decode path are launched so that a kernel may be scheduled, and
// run the part of its prologue that touches no global memory, while its predecessor in the stream is still finishing
// --------------------------------------------------------------------------------------------------
// EVERY thread block of a kernel launched with launch_pdl must execute pdl_wait() before its first global memory
// access and before it exits (a block that exits without waiting lets the grid "complete" while its predecessor is
// still running, and the grid after it would then start too early).  pdl_wait() returns once the preceding grid has
// completed and its writes are visible; pdl_launch() lets the following grid start being scheduled.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

bool pdl_enabled();     // false when NEZHA_NO_PDL is set: plain stream-ordered launches

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// --------------------------------------------------------------------------------------------------
// small device helpers
// --------------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// --------------------------------------------------------------------------------------------------
// hash set (Eq. 5): open addressing over 4-slot buckets, linear probing over buckets
// --------------------------------------------------------------------------------------------------
struct HashSetView {
  unsigned long long* slots;       // [n_buckets * kBucketSlots]
  unsigned long long n_buckets;
};

// 64-bit finalizer (the published murmur3 fmix64 constants), then multiply-shift range reduction so that
// any bucket count works (no power-of-two requirement).
__device__ __forceinline__ unsigned long long hs_mix(unsigned long long k) {
  k ^= k >> 33; k *= 0xff51afd7ed558ccdull; k ^= k >> 33; k *= 0xc4ceb9fe1a85ec53ull; k ^= k >> 33;
  return k;
}
__device__ __forceinline__ unsigned long long hs_bucket(unsigned long long key, unsigned long long n_buckets) {
  return __umul64hi(hs_mix(key), n_buckets);
}

// One thread walks the probe sequence alone, a whole bucket (one sector) per step.  The empty-slot sentinel is not a
// packed key (Eq. 4 maps onto [0, prod T) and prod T < 2^64 - 1): it is never a member, although it equals every free slot.
__device__ __forceinline__ bool hs_contains_thread(const HashSetView& hs, unsigned long long key) {
  if (key == kEmptyKey) return false;
  unsigned long long b = hs_bucket(key, hs.n_buckets);
  for (int step = 0; step < kMaxProbeBuckets; ++step) {
    const ulonglong2* p = reinterpret_cast<const ulonglong2*>(hs.slots + b * kBucketSlots);
    ulonglong2 lo = __ldg(p), hi = __ldg(p + 1);
    if (lo.x == key || lo.y == key || hi.x == key || hi.y == key) return true;
    if (lo.x == kEmptyKey || lo.y == kEmptyKey || hi.x == kEmptyKey || hi.y == kEmptyKey) return false;
    if (++b == hs.n_buckets) b = 0;
  }
  return false;
}

// Membership of N keys per thread with the memory round trips overlapped: the home buckets of all keys are loaded
// first (independent loads), and only a key whose home bucket is full without holding it walks on alone.
template <int N>
__device__ __forceinline__ void hs_contains_many(const HashSetView& hs, const unsigned long long* keys, const bool* want,
                                                 bool* found) {
  ulonglong2 lo[N], hi[N];
#pragma unroll
  for (int j = 0; j < N; ++j) {
    if (want[j]) {
      const ulonglong2* p = reinterpret_cast<const ulonglong2*>(hs.slots + hs_bucket(keys[j], hs.n_buckets) * kBucketSlots);
      lo[j] = __ldg(p); hi[j] = __ldg(p + 1);
    }
  }
#pragma unroll
  for (int j = 0; j < N; ++j) {
    found[j] = false;
    if (!want[j]) continue;
    const unsigned long long k = keys[j];
    if (k == kEmptyKey) continue;                      // the sentinel matches every free slot and is no key
    if (lo[j].x == k || lo[j].y == k || hi[j].x == k || hi[j].y == k) found[j] = true;
    else if (lo[j].x == kEmptyKey || lo[j].y == kEmptyKey || hi[j].x == kEmptyKey || hi[j].y == kEmptyKey) found[j] = false;
    else found[j] = hs_contains_thread(hs, k);        // home bucket full: rare at the load factors in use
  }
}

// --------------------------------------------------------------------------------------------------
// prefix map: the same set V, regrouped as (prefix of n codes) -> bit set of the codes that may follow it
// --------------------------------------------------------------------------------------------------
// For every n in [0, L): the distinct n-code prefixes of the valid IDs, each with the bit set of the level-(n+1) codes t
// such that some valid ID begins with (prefix, t).  For n = L - 1 that is Eq. 5 itself for all T_L extensions of a beam in
// one look-up -- the same answers as T_L hash probes, bit for bit; for n < L - 1 it answers "does any valid ID begin with
// these codes?", the validity filter at the earlier levels.  One table region per n (so a key needs no level tag), open
// addressing with linear probing over slots of `stride` words inside the region: word 0 = prefix key + 1 (0 = empty),
// words 1.. = the bit set.
struct PrefixMapView {
  unsigned long long* slots;       // [n_slots * stride]; null = not in use
  unsigned long long n_slots;      // all regions together
  int stride;                      // words per slot: a power of two >= 1 + ceil(max T / 64)
  unsigned long long level_off[kMaxLevels];     // first slot of the region of prefixes with n codes
  unsigned long long level_slots[kMaxLevels];   // its slot count
};
// The bit set of a prefix of n codes, or null if no valid ID begins with it.  Every lane of a warp may call this with the
// same key (the loads are then broadcasts).
__device__ __forceinline__ const unsigned long long* pm_find(const PrefixMapView& pm, int n, unsigned long long prefix_key) {
  const unsigned long long ns = pm.level_slots[n];
  const unsigned long long* region = pm.slots + pm.level_off[n] * pm.stride;
  unsigned long long s = __umul64hi(hs_mix(prefix_key), ns);
  for (int step = 0; step < kMaxProbeBuckets; ++step) {
    const unsigned long long* slot = region + s * pm.stride;
    const unsigned long long k = __ldg(slot);
    if (k == prefix_key + 1) return slot + 1;
    if (k == 0ull) return nullptr;
    if (++s == ns) s = 0;
  }
  return nullptr;
}
__device__ __forceinline__ bool pm_test(const unsigned long long* bits, int t) {
  return bits != nullptr && ((__ldg(bits + (t >> 6)) >> (t & 63)) & 1ull);
}

// --------------------------------------------------------------------------------------------------
// model / engine description shared by the host code and the kernels
// --------------------------------------------------------------------------------------------------
struct LevelInfo {
  int L;
  int T[kMaxLevels];
  int off[kMaxLevels];             // vocabulary offset of each level's codes
  unsigned long long mult[kMaxLevels];   // Eq. 4 positional multipliers
  int vocab_codes;                 // sum(T)
};

// Eq. 4 on a code tuple held in registers / local memory.
__device__ __forceinline__ unsigned long long pack_key(const LevelInfo& li, const int* codes) {
  unsigned long long k = 0;
  for (int l = 0; l < li.L; ++l) k += (unsigned long long)codes[l] * li.mult[l];
  return k;
}

// --------------------------------------------------------------------------------------------------
// GEMM:  C[M,N] (op)= A[M,K] * W[N,K]^T   (both operands K-major)
// --------------------------------------------------------------------------------------------------
enum GemmEpilogue : int {
  kEpiStoreAct = 0,     // C (activation type) = acc
  kEpiStoreF32 = 1,     // C (float) = acc
  kEpiAddF32 = 2,       // C (float) += acc                    (residual stream)
  kEpiBiasTanhF32 = 3,  // C (float) = tanh(acc + bias[n])     (Eq. 3)
  // ---- fused epilogues of the tensor-core kernel only -------------------------------------------------------
  kEpiSwiGLU = 4,       // weight rows interleaved (gate, gate, up, up per 4 columns): C (act)[m, n/2] = silu(gate) * up
  kEpiAddNorm = 5,      // C (float) += acc; xg (act)[m, n] = C * gain[n]; ss_out[n / 32][m] = sum of C^2 over the 32 columns
  kEpiRopeKV = 6        // fused QKV projection: rotary embedding on q and k, q to C, k and v to the KV cache
};

// Extras of the fused epilogues.  RMSNorm is split around the GEMMs: the producer of the residual stream
// (kEpiAddNorm) leaves x * gain as the next GEMM's A operand and partial sums of x^2 per 32 columns; the consumer GEMM
// multiplies its accumulator rows by rsqrt(mean(x^2) + eps), summing the partials in a fixed order.
struct GemmFuse {
  const float* ss_in; int ss_in_parts; long long ss_ld; float inv_dim, eps;   // row scale of the A operand (or null)
  float* ss_out;                     // [N / 32][ss_ld]
  void* xg; const void* gain;        // kEpiAddNorm: next A operand [M, N] (activation type) and its norm gain [N]
  // kEpiRopeKV: weight rows of every q / k head permuted so that every 4 consecutive columns hold two rotary pairs
  const int* tok_pos; const long long* kv_dst; long long kv_head_stride;
  void* k_cache; void* v_cache; const float* cos_tab; const float* sin_tab;
  int Hq, Hkv, hd;
};

constexpr int kSkinnyRows = 128;    // most rows a launch of the weight-streaming GEMM kernel takes

struct GemmArgs {
  const void* A; long long lda;
  const void* W; long long ldw;
  void* C; long long ldc;
  int M;                 // upper bound of rows (grid is sized for it)
  const int* M_dev;      // optional: actual row count on the device (<= M); rows beyond are skipped
  int N, K;
  int epilogue;
  const float* bias;
  int* status;           // device status word (bounded waits report here)
  GemmFuse f;            // zero-initialised unless a fused epilogue is asked for
  int M_expected;        // 0, or the row count the caller expects on the device (<= M): only shapes the tiling
  // 0: the K range is accumulated in order.  2: products with N <= 1024 accumulate it in two interleaved partial sums
  // (k-step k goes to sum k mod 2), added at the end, so that two MMA issuers can run the k-loop.  The two orders round
  // differently: a caller that needs the same bits from launches of different sizes asks for the same value in all of
  // them (the tiling itself never changes the result).
  int chains;
  // Non-zero: a launch of at most kSkinnyRows rows may run as the weight-streaming kernel (weights as the 128-row MMA
  // operand, the rows as its N, the K range split over the CTAs of a cluster).  Its summation order differs from the
  // other kernels' and depends on (N, K) and the device only: a caller that needs the same bits from two launches sets
  // the flag in both or in neither.  W must be constant data (it is read before the launch's dependency on its
  // predecessor is resolved).
  int skinny;
};

void launch_gemm_simt(const GemmArgs& a, bool bf16, cudaStream_t st);

// --------------------------------------------------------------------------------------------------
// element-wise / glue kernels
// --------------------------------------------------------------------------------------------------
void launch_embed(const void* table, bool bf16, const int* tokens, int M, const int* M_dev, int d, float* resid,
                  cudaStream_t st);
void launch_embed_norm(const void* table, const int* tokens, int M, const int* M_dev, int d, float* resid,
                       const void* gain, void* xg, float* ss, cudaStream_t st);
void launch_permute_rotary_rows(const void* src, void* dst, int rows, int hd, int cols, cudaStream_t st);
void launch_interleave_gate_up(const void* gate, const void* up, void* dst, int F, int cols, cudaStream_t st);
void launch_rmsnorm(const float* x, long long x_stride, const int* row_index, const void* gain, bool bf16, void* out,
                    float* out_f32, int M, const int* M_dev, int d, float eps, cudaStream_t st);

struct RopeAppendArgs {
  void* qkv;                       // [M, (Hq + 2 Hkv) * hd], activation type; q and k rotated in place
  const int* tok_pos;              // [M] rotary position
  const long long* kv_dst;         // [M] element offset of the token's K (and V) row group in the layer's cache:
                                   //     token's head h row starts at kv_dst[i] + h * kv_head_stride
  long long kv_head_stride;
  void* k_cache; void* v_cache;    // layer base pointers
  const float* cos_tab; const float* sin_tab;   // [positions, hd/2]
  int M; const int* M_dev;
  int Hq, Hkv, hd;
};
void launch_rope_append(const RopeAppendArgs& a, bool bf16, cudaStream_t st);
void launch_swiglu(const void* gu, void* act, int M, const int* M_dev, int F, bool bf16, cudaStream_t st);

// --------------------------------------------------------------------------------------------------
// attention over (context KV prefix) + (a few extra KV rows per token)
// --------------------------------------------------------------------------------------------------
struct AttnArgs {
  const void* q; long long q_stride;        // token i, head h at q + i*q_stride + h*hd
  void* out; long long out_stride;          // [M, Hq*hd]
  const void* k_ctx; const void* v_ctx;     // layer base of the context cache [rows][Hkv][S][hd]
  long long ctx_row_stride, ctx_head_stride;// element strides (row = request, head = kv head)
  const void* k_ext; const void* v_ext;     // layer base of the draft-token cache
  long long ext_head_stride;                // element stride between kv heads inside one extra entry
  const int* tok_row;                       // [M] request (cache row) of the token
  const int* tok_ctx_len;                   // [M] number of context positions visible
  const long long* tok_ext;                 // [M, n_ext_max] element offsets of extra KV entries, -1 = unused
  int n_ext_max;
  int M; const int* M_dev;
  int Hq, Hkv, hd;
  float scale;
  // grouping of the token list by request (tokens of a request are contiguous), for the tensor-core kernel
  const int* row_start; const int* row_count;   // [n_rows] first token / token count of each request in this pass
  const int4* req_info;                         // [n_rows] {first token, token count, cache row, context length visible to
                                                //  every token of the request, or -1: token j of the request sees j + 1}
  int n_rows, max_tokens_per_row;
  int rows_expected;                            // 0, or the query rows per (request, kv head) the caller expects: tiling only
  long long ctx_rows_total;                     // requests * kv heads * positions of the layer's context cache
  // the draft-token cache seen as positions: a request owns ext_positions consecutive positions (level-major, then beam
  // slot), ext_pos_stride elements apart (all KV heads of a position are adjacent), ext_req_stride elements per request
  int ext_positions; long long ext_pos_stride, ext_req_stride, ext_rows_total;
  int* status;
};
void launch_attention_simt(const AttnArgs& a, bool bf16, cudaStream_t st);

}  // namespace nz
