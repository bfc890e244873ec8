// Beam-search kernels: fused log-softmax + validity mask + beam top-k (one level of Algorithm 1 / Algorithm 3),
// the draft head's glue (Eq. 1-3 inputs), the verify pass's token list, and accept / roll-back (Algorithm 2's
// rejection and update steps).  Every kernel here runs one thread block per request; requests never interact.
#include <math.h>

#include "engine_state.cuh"

namespace nz {

// ====================================================================================================
// fused log-softmax + mask + top-k
// ====================================================================================================
// Per request: each warp takes beams r = warp, warp + n_warps, ...  For a beam it loads the T logits of the
// level's codebook (VPL per lane), computes log-softmax with warp shuffles, and extracts the beam's best
// candidates in order (repeated warp arg-max; ties to the smaller code):
//   per_beam <  T : the per_beam most probable codes, THEN the hash-set filter on those       (Algorithm 3: top-K, then verification)
//   per_beam >= T : the filter on all T codes, THEN the K best by cumulative log-probability  (top-k restricted to V)
// The sorted per-beam lists go to shared memory and warp 0 merges them into the K best of the request
// (ties to the smaller parent rank, then the smaller code).
namespace {

struct Cand { float s; int r; int t; };

__device__ __forceinline__ bool cand_better(float s, int r, int t, float s2, int r2, int t2) {
  if (s != s2) return s > s2;
  if (r != r2) return r < r2;
  return t < t2;
}

// Monotone map float -> unsigned (larger float, larger integer), so that a warp maximum is one redux instruction.
__device__ __forceinline__ unsigned ordered_bits(float f) {
  const unsigned u = __float_as_uint(f + 0.f);           // + 0: minus zero and plus zero rank alike
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(unsigned o) {
  return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}
constexpr unsigned kOrderedNegInf = 0x007fffffu;          // ordered_bits(-inf)

// Sorts v in descending order with Batcher's odd-even merge network (N a power of two; every index is a compile-time
// constant once unrolled, so v stays in registers).
template <int N>
__device__ __forceinline__ void sort_desc(unsigned long long (&v)[N]) {
#pragma unroll
  for (int p = 1; p < N; p <<= 1) {
#pragma unroll
    for (int k = p; k >= 1; k >>= 1) {
#pragma unroll
      for (int j = k % p; j + k < N; j += 2 * k) {
#pragma unroll
        for (int i = 0; i < k; ++i) {
          if (i + j + k < N && (i + j) / (2 * p) == (i + j + k) / (2 * p)) {
            const unsigned long long x = v[i + j], y = v[i + j + k];
            v[i + j] = x > y ? x : y;
            v[i + j + k] = x > y ? y : x;
          }
        }
      }
    }
  }
}

// One block per request.  Stage 1, a warp per input beam: log-softmax of the beam's logits row (+ Eq. 5 on every
// extension at the last level), then its `want` best codes in order into shared memory.  Stage 2: the K best of those
// lists (score, then parent rank, then code).  Stage 3, all threads: the output beams.  The kernel is a chain of
// dependent steps on a few warps, so its time is the sum of their latencies: loads whose address needs no other load
// go out together at the top; each lane keeps its keys sorted, so one survivor costs two redux and a shift; small
// merges are a rank count with no serial loop at all.
// Codebooks of more than 512 codes keep 32 keys per lane in registers besides the scores: that variant runs with at most
// 8 warps so that a thread may use up to 255 registers.
__host__ __device__ constexpr int select_max_threads(int vpl) { return vpl >= 32 ? 256 : 512; }
inline int select_warps(const SelectArgs& a) {
  const int cap = a.T > 512 ? 8 : 16;
  return a.in_stride < 8 ? 8 : a.in_stride > cap ? cap : a.in_stride;
}

template <int VPL>
__device__ __forceinline__ void select_body(const SelectArgs& a) {
  const int b = blockIdx.x;
  extern __shared__ unsigned char smem_raw[];
  const int nb_cap = a.in_stride;
  float* l_score = reinterpret_cast<float*>(smem_raw);              // [nb_cap][K]
  int* l_tok = reinterpret_cast<int*>(l_score + (size_t)nb_cap * a.K);   // [nb_cap][K]
  int* l_cnt = l_tok + (size_t)nb_cap * a.K;                         // [nb_cap]
  float* sel_s = reinterpret_cast<float*>(l_cnt + nb_cap);           // [K] the selected (score, parent, code)
  int* sel_r = reinterpret_cast<int*>(sel_s + a.K);
  int* sel_t = sel_r + a.K;
  int* s_nout = sel_t + a.K;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;

  // ---- first wave of loads (none of these addresses depends on a loaded value)
  const int gate_v = a.gate_mode ? a.gate[b] : 0;
  const int nb_raw = a.in_count[b];
  const bool has0 = warp < nb_cap;                                   // this warp's first beam slot exists in the arrays
  const long long slot0 = (long long)b * a.in_stride + warp;
  const bool direct0 = has0 && !a.src_row && warp < a.src_mul;       // its logits row is known without a look-up
  long long row0 = 0;
  if (has0) row0 = a.src_row ? (long long)a.src_row[slot0] : (long long)b * a.src_mul + warp;
  const float base0 = has0 ? a.in_score[slot0] : 0.f;
  unsigned long long pk0 = 0;
  if (has0)
    for (int l = 0; l < a.n; ++l) pk0 += (unsigned long long)a.in_codes[slot0 * a.tuple_len + l] * a.li.mult[l];
  float bias[VPL], z0[VPL];
#pragma unroll
  for (int j = 0; j < VPL; ++j) {
    const int t = lane + 32 * j;
    bias[j] = (a.logit_bias && t < a.T) ? a.logit_bias[(long long)b * a.bias_stride + t] : 0.f;
    z0[j] = (direct0 && t < a.T) ? a.logits[row0 * a.row_stride + a.col_off + t] : 0.f;
  }
  if (a.gate_mode == 1 && gate_v != a.gate_value) return;
  if (a.gate_mode == 2 && !(gate_v < a.gate_value)) return;
  const int nb = min(nb_raw, nb_cap);
  const bool all_codes = a.per_beam >= a.T;
  const int want = all_codes ? min(a.K, a.T) : min(a.per_beam, a.K);
  const unsigned long long mult_n = a.li.mult[a.n];

  for (int r = warp; r < nb; r += n_warps) {
    const bool first = r == warp;
    const long long slot = (long long)b * a.in_stride + r;
    const long long row = first ? row0 : (a.src_row ? (long long)a.src_row[slot] : (long long)b * a.src_mul + r);
    const float* z = a.logits + row * a.row_stride + a.col_off;
    float key[VPL];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int t = lane + 32 * j;
      key[j] = (t < a.T) ? ((first && direct0) ? z0[j] : z[t]) + bias[j] : -INFINITY;
      mx = fmaxf(mx, key[j]);
    }
    const float base = first ? base0 : a.in_score[slot];
    unsigned long long prefix_key = pk0;
    if (!first) {
      prefix_key = 0;
      for (int l = 0; l < a.n; ++l) prefix_key += (unsigned long long)a.in_codes[slot * a.tuple_len + l] * a.li.mult[l];
    }
    mx = warp_max(mx);
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < VPL; ++j) sum += (lane + 32 * j < a.T) ? expf(key[j] - mx) : 0.f;
    sum = warp_sum(sum);
    const float lse = mx + logf(sum);
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      if (lane + 32 * j < a.T) {
        key[j] -= lse;                                   // log-probability
        if (all_codes) key[j] += base;                   // rank by cumulative log-probability
      }
    }
    // The bit set of the codes that may follow this beam: Eq. 5 for all T_L extensions at the last level, "some valid ID
    // begins with it" at an earlier level.
    const bool use_bits = a.prefix_filter || (all_codes && a.filter && a.final_mask_from_map);
    const unsigned long long* bits = use_bits ? pm_find(a.pm, a.n, prefix_key) : nullptr;
    if (all_codes && use_bits) {
#pragma unroll
      for (int j = 0; j < VPL; ++j) {
        const int t = lane + 32 * j;
        if (t < a.T && !pm_test(bits, t)) key[j] = -INFINITY;
      }
    } else if (all_codes && a.filter) {                  // Eq. 5 on every extension of the beam, 8 probes in flight
      constexpr int PB = VPL < 8 ? VPL : 8;
#pragma unroll
      for (int j0 = 0; j0 < VPL; j0 += PB) {
        unsigned long long pk[PB]; bool want_probe[PB], ok[PB];
#pragma unroll
        for (int j = 0; j < PB; ++j) {
          want_probe[j] = lane + 32 * (j0 + j) < a.T;
          pk[j] = prefix_key + (unsigned long long)(lane + 32 * (j0 + j)) * mult_n;
        }
        hs_contains_many<PB>(a.hs, pk, want_probe, ok);
#pragma unroll
        for (int j = 0; j < PB; ++j)
          if (want_probe[j] && !ok[j]) key[j0 + j] = -INFINITY;
      }
    }
    int cnt = 0;
    if constexpr (VPL >= 16) {
      // Wide codebooks: no per-lane sort.  A sorting network of 16 or 32 keys is kilobytes of straight-line code that a
      // warp runs once, and fetching it costs more than it saves (12.6 us per beam at T = 512 against 3.2 at T = 256;
      // 6 us with this loop).  With many survivors per beam (K = 50) the sorted lists below are the cheaper form.
      // Each round every lane finds its best remaining key (four independent scans, so the chain is VPL / 4 long), the
      // warp picks the best of those (ties go to the smaller code), and the owner retires it: a short loop body.
      unsigned ob[VPL];                                  // ordered score bits; 0 = used up
#pragma unroll
      for (int j = 0; j < VPL; ++j) ob[j] = ordered_bits(key[j]);
#pragma unroll 1
      for (int it = 0; it < want; ++it) {
        unsigned qo[4]; int qj[4];
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          qo[q4] = 0u; qj[q4] = q4 * (VPL / 4);
#pragma unroll
          for (int j = q4 * (VPL / 4); j < (q4 + 1) * (VPL / 4); ++j)
            if (ob[j] > qo[q4]) { qo[q4] = ob[j]; qj[q4] = j; }
        }
        unsigned ho = qo[0]; int hj = qj[0];
#pragma unroll
        for (int q4 = 1; q4 < 4; ++q4)
          if (qo[q4] > ho) { ho = qo[q4]; hj = qj[q4]; }     // strict: the smaller code wins a tie
        const int ht = lane + 32 * hj;
        const unsigned mo = __reduce_max_sync(0xffffffffu, ho);
        if (mo <= kOrderedNegInf) break;
        const int bt = (int)__reduce_min_sync(0xffffffffu, ho == mo ? (unsigned)ht : 0x7fffffffu);
        if ((bt & 31) == lane) {
#pragma unroll
          for (int j = 0; j < VPL; ++j)
            if (j == (bt >> 5)) ob[j] = 0u;
        }
        if (lane == 0) {
          const float bv = from_ordered_bits(mo);
          l_score[(size_t)r * a.K + cnt] = all_codes ? bv : base + bv;
          l_tok[(size_t)r * a.K + cnt] = bt;
        }
        ++cnt;
      }
    } else {
      // this lane's keys in descending order: (ordered score bits, then the smaller code first); 0 = used up
      unsigned long long sk[VPL];
#pragma unroll
      for (int j = 0; j < VPL; ++j) sk[j] = ((unsigned long long)ordered_bits(key[j]) << 32) | (unsigned)(VPL - 1 - j);
      sort_desc<VPL>(sk);
      // ordered extraction: the warp's best head (ties go to the smaller code), whose lane then shifts its list
      for (int it = 0; it < want; ++it) {
        const unsigned ho = (unsigned)(sk[0] >> 32);
        const int ht = lane + 32 * (VPL - 1 - (int)(unsigned)sk[0]);
        const unsigned mo = __reduce_max_sync(0xffffffffu, ho);
        if (mo <= kOrderedNegInf) break;
        const int bt = (int)__reduce_min_sync(0xffffffffu, ho == mo ? (unsigned)ht : 0x7fffffffu);
        if ((bt & 31) == lane) {
#pragma unroll
          for (int j = 0; j + 1 < VPL; ++j) sk[j] = sk[j + 1];
          sk[VPL - 1] = 0ull;
        }
        if (lane == 0) {
          const float bv = from_ordered_bits(mo);
          l_score[(size_t)r * a.K + cnt] = all_codes ? bv : base + bv;
          l_tok[(size_t)r * a.K + cnt] = bt;
        }
        ++cnt;
      }
    }
    __syncwarp();
    if (!all_codes && (a.filter || a.prefix_filter)) {   // filter the chosen codes, keep their order
      int kept = 0;
      for (int c0 = 0; c0 < cnt; c0 += 32) {
        const int c = c0 + lane;
        bool ok = false; float sv = 0.f; int t = 0;
        if (c < cnt) {
          sv = l_score[(size_t)r * a.K + c]; t = l_tok[(size_t)r * a.K + c];
          ok = a.prefix_filter ? pm_test(bits, t) : hs_contains_thread(a.hs, prefix_key + (unsigned long long)t * mult_n);
        }
        const unsigned m = __ballot_sync(0xffffffffu, ok);
        __syncwarp();
        if (ok) {
          const int dst = kept + __popc(m & ((1u << lane) - 1u));
          l_score[(size_t)r * a.K + dst] = sv; l_tok[(size_t)r * a.K + dst] = t;
        }
        kept += __popc(m);
        __syncwarp();
      }
      cnt = kept;
    }
    if (lane == 0) l_cnt[r] = cnt;
  }
  __syncthreads();

  // ---- stage 2: the K best candidates of the nb lists into sel_*[0 .. n_out)
  if (nb * a.K <= 1024) {
    // few candidates: a candidate's output position is the number of candidates that beat it (the order is strict)
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int r = 0; r < nb; ++r) tot += l_cnt[r];
      *s_nout = min(tot, a.K);
    }
    for (int i = threadIdx.x; i < nb * a.K; i += blockDim.x) {
      const int r = i / a.K, c = i - r * a.K;
      if (c >= l_cnt[r]) continue;
      const float sv = l_score[i];
      const int t = l_tok[i];
      // Its own list is sorted: c of its entries come before it.  In another list the entries that beat it are a prefix
      // (the list is sorted and the parent rank breaks ties), so the scan of a list stops at the first entry that does
      // not, and the whole count stops once the candidate is known to miss the best K.
      int rank = c;
      for (int r2 = 0; r2 < nb && rank < a.K; ++r2) {
        if (r2 == r) continue;
        const int n2 = l_cnt[r2];
        int c2 = 0;
        while (c2 < n2 && cand_better(l_score[(size_t)r2 * a.K + c2], r2, l_tok[(size_t)r2 * a.K + c2], sv, r, t)) ++c2;
        rank += c2;
      }
      if (rank < a.K) { sel_s[rank] = sv; sel_r[rank] = r; sel_t[rank] = t; }
    }
  } else if (warp == 0) {
    constexpr int RPL = 4;                                 // lists per lane: in_stride <= 128
    int ptr[RPL];
#pragma unroll
    for (int q = 0; q < RPL; ++q) ptr[q] = 0;
    int n_out = 0;
    for (int k = 0; k < a.K; ++k) {
      float bs = -INFINITY; int br = 0x7fffffff, bt = 0x7fffffff;
#pragma unroll
      for (int q = 0; q < RPL; ++q) {
        const int r = lane + 32 * q;
        if (r < nb && ptr[q] < l_cnt[r]) {
          const float sv = l_score[(size_t)r * a.K + ptr[q]];
          const int t = l_tok[(size_t)r * a.K + ptr[q]];
          if (br == 0x7fffffff || cand_better(sv, r, t, bs, br, bt)) { bs = sv; br = r; bt = t; }
        }
      }
      // warp arg-best: maximum score, then the smallest (parent rank, code) among the lanes that hold it
      const unsigned bo = br == 0x7fffffff ? 0u : ordered_bits(bs);
      const unsigned mo = __reduce_max_sync(0xffffffffu, bo);
      if (mo == 0u) break;                                   // every list is exhausted
      const unsigned pick = __reduce_min_sync(0xffffffffu, bo == mo ? ((unsigned)br << 16 | (unsigned)bt) : 0xffffffffu);
      br = (int)(pick >> 16); bt = (int)(pick & 0xffffu);
#pragma unroll
      for (int q = 0; q < RPL; ++q)
        if (lane + 32 * q == br) ++ptr[q];
      if (lane == 0) { sel_s[k] = from_ordered_bits(mo); sel_r[k] = br; sel_t[k] = bt; }
      ++n_out;
    }
    if (lane == 0) *s_nout = n_out;
  }
  __syncthreads();

  // ---- stage 3: the output beams, all threads
  const int n_out = *s_nout;
  for (int k = threadIdx.x; k < a.K; k += blockDim.x) {
    const long long o = (long long)b * a.out_stride + k;
    const bool live = k < n_out;
    a.out_score[o] = live ? sel_s[k] : -INFINITY;
    if (a.out_parent) a.out_parent[o] = live ? sel_r[k] : -1;
    if (a.out_token) a.out_token[o] = live ? sel_t[k] : -1;
  }
  if (a.out_codes) {
    for (int i = threadIdx.x; i < a.K * a.tuple_len; i += blockDim.x) {
      const int k = i / a.tuple_len, l = i - k * a.tuple_len;
      int c = -1;
      if (k < n_out) {
        if (l < a.n) c = a.in_codes[((long long)b * a.in_stride + sel_r[k]) * a.tuple_len + l];
        else if (l == a.n) c = sel_t[k];
      }
      a.out_codes[((long long)b * a.out_stride + k) * a.tuple_len + l] = c;
    }
  }
  if (threadIdx.x == 0) a.out_count[b] = n_out;
}

template <int VPL>
__global__ void __launch_bounds__(select_max_threads(VPL)) select_kernel(SelectArgs a) {
  pdl_wait();
  pdl_launch();
  select_body<VPL>(a);
}

}  // namespace

cudaError_t select_step_configure(int bytes);

size_t select_smem_bytes(int in_stride, int K) {
  return (size_t)in_stride * K * (sizeof(float) + sizeof(int)) + (size_t)in_stride * sizeof(int) +
         (size_t)K * (sizeof(float) + 2 * sizeof(int)) + sizeof(int);
}

// The attribute belongs to the device, and several contexts may share one: it is only ever raised.
cudaError_t select_configure(int max_beam) {
  static int configured_bytes[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  int bytes = (int)select_smem_bytes(max_beam, max_beam);
  if (bytes <= configured_bytes[dev]) return cudaSuccess;
  configured_bytes[dev] = bytes;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(select_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  return select_step_configure(bytes);
}

void launch_select(const SelectArgs& a, cudaStream_t st) {
  if (a.batch <= 0) return;
  const size_t smem = select_smem_bytes(a.in_stride, a.K);
  LaunchScope ls(kcSelect, st);
  const int warps = select_warps(a);   // a warp per beam where that fits
  const dim3 block(32 * warps);
  if (a.T <= 32) launch_pdl(select_kernel<1>, dim3(a.batch), block, smem, st, a);
  else if (a.T <= 256) launch_pdl(select_kernel<8>, dim3(a.batch), block, smem, st, a);
  else if (a.T <= 512) launch_pdl(select_kernel<16>, dim3(a.batch), block, smem, st, a);
  else launch_pdl(select_kernel<32>, dim3(a.batch), block, smem, st, a);
}

// ====================================================================================================
// small state kernels
// ====================================================================================================
namespace {

__global__ void fill_i32_kernel(int* p, long long n, int v) {
  pdl_wait();
  pdl_launch();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    p[i] = v;
}
__global__ void fill_f32_kernel(float* p, long long n, float v) {
  pdl_wait();
  pdl_launch();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    p[i] = v;
}

// B_0 = { empty beam, score 0 } for every request; nothing settled.
__global__ void init_decode_kernel(EngineState e, int batch) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b == 0) {
    for (int i = 0; i < 8; ++i) e.counters[i] = 0;
    *e.draft_rows = batch * e.Kmax;
  }
  if (b >= batch) return;
  e.tb_count[0 * e.Bmax + b] = 1;
  e.tb_score[lvl_bk(e, 0, b, 0)] = 0.f;
  e.tb_parent[lvl_bk(e, 0, b, 0)] = -1;
  e.tb_src[lvl_bk(e, 0, b, 0)] = -1;
  e.row_m[b] = 0;
  e.row_cur[b] = -1;
  e.row_spec[b] = 1;
  e.row_m_start[b] = 0;
  e.d_m[b] = e.L;
  for (int l = 0; l <= e.L; ++l) e.dw_count[(long long)l * e.Bmax + b] = 0;     // no draft tree yet
}

// Start of a round's drafting (Algorithm 2's drafting step): the draft head continues from the true beams B_m, or from
// the empty beam in the first round (Algorithm 3's initialisation).
// Also clears the round's counters (this is the first kernel of a drafting round) and, when s_act is given, starts
// every beam slot's draft state at s_1 = h_0 (Eq. 1).
__global__ void draft_init_kernel(EngineState e, int batch, int from_scratch, __nv_bfloat16* s_act) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  if (b == 0 && threadIdx.x < 8) e.counters[threadIdx.x] = 0;
  if (b >= batch) return;
  if (s_act) {
    const float* h0 = e.h_f32 + (long long)b * (e.L + 1) * e.d;
    __nv_bfloat16* dst = s_act + (long long)b * e.Kmax * e.d;
    for (int c = threadIdx.x; c < e.d; c += blockDim.x) {
      const __nv_bfloat16 v = __float2bfloat16_rn(h0[c]);
      for (int k = 0; k < e.Kmax; ++k) dst[(long long)k * e.d + c] = v;
    }
  }
  const int m = e.row_m[b];
  if (m >= e.L || !e.row_spec[b]) {              // finished, or its drafting is switched off: an empty tree this round
    if (threadIdx.x == 0) e.d_m[b] = e.L;
    if ((int)threadIdx.x <= e.L) e.dw_count[(long long)threadIdx.x * e.Bmax + b] = 0;
    return;
  }
  const int mm = from_scratch ? 0 : m;
  const int cnt = e.tb_count[mm * e.Bmax + b];
  for (int k = threadIdx.x; k < e.Kmax; k += blockDim.x) {
    const long long s = lvl_bk(e, mm, b, k);
    const bool live = k < cnt;
    e.dw_score[s] = live ? e.tb_score[s] : -INFINITY;
    e.dw_parent[s] = live ? k : -1;
    for (int l = 0; l < e.L; ++l) e.dw_codes[s * e.L + l] = live ? e.tb_codes[s * e.L + l] : -1;
  }
  if (threadIdx.x == 0) { e.dw_count[mm * e.Bmax + b] = cnt; e.d_m[b] = mm; }
}

// Caller-supplied drafted tuples for the round (or none: n_draft == nullptr and drafts == nullptr -> an empty tree).
// The tree of the tuples is built level by level: level j holds their distinct j-prefixes in order of first appearance
// (tuples that share a prefix share its node), each with the slot of its parent.  One block of >= Kmax threads per request.
__global__ void draft_set_kernel(EngineState e, int batch, int K, const int* drafts, const int* n_draft) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  if (b == 0 && threadIdx.x < 8) e.counters[threadIdx.x] = 0;      // first kernel of the round: clear its counters
  if (b >= batch) return;
  const int L = e.L, k = threadIdx.x;
  __shared__ int s_slot[2][128];                 // slot of tuple k's prefix in the previous / the current level
  __shared__ int s_new[128], s_ok[128], s_cnt;
  const int cnt = (drafts && e.row_m[b] < L) ? max(0, min(n_draft[b], K)) : 0;
  int code[kMaxLevels];
  bool ok = k < cnt;
  for (int l = 0; l < L; ++l) {
    code[l] = ok ? drafts[((long long)b * K + k) * L + l] : -1;
    if (k < cnt && (code[l] < 0 || code[l] >= e.li.T[l])) { atomicOr(e.status, kStBadCode); ok = false; }
  }
  s_slot[0][k] = 0;                              // level 0: the empty prefix, slot 0
  s_ok[k] = ok ? 1 : 0;                          // a tuple with an out-of-range code is dropped as a whole
  __syncthreads();
  for (int j = 1; j <= L; ++j) {
    const int cur = j & 1, prev = cur ^ 1;
    int first = -1;                              // the first tuple with the same j-prefix
    if (ok) {
      for (int k2 = 0; k2 <= k && first < 0; ++k2) {
        if (!s_ok[k2]) continue;
        bool eq = true;
        for (int l = 0; l < j; ++l) eq &= (drafts[((long long)b * K + k2) * L + l] == code[l]);
        if (eq) first = k2;
      }
    }
    s_new[k] = (ok && first == k) ? 1 : 0;
    __syncthreads();
    if (k == 0) {                                // exclusive scan of the "new node" flags -> slots
      int c = 0;
      for (int i = 0; i < cnt; ++i) { const int f = s_new[i]; s_new[i] = c; c += f; }
      s_cnt = c;
    }
    __syncthreads();
    if (ok) {
      const int slot = s_new[first];
      s_slot[cur][k] = slot;
      if (first == k) {
        const long long s = lvl_bk(e, j, b, slot);
        for (int l = 0; l < L; ++l) e.dw_codes[s * L + l] = l < j ? code[l] : -1;
        e.dw_score[s] = 0.f;
        e.dw_parent[s] = s_slot[prev][k];
      }
    }
    if (k == 0) e.dw_count[(long long)j * e.Bmax + b] = s_cnt;
    __syncthreads();
  }
  if (k == 0) e.d_m[b] = L;
}

// Caller-supplied draft tree (test hook): level j's nodes are taken as listed; a node's parent is the node of level j - 1
// that equals its first j - 1 codes (-1 if there is none: the node is then dead).  One block of >= Kmax threads per request.
__global__ void draft_tree_set_kernel(EngineState e, int batch, int K, const int* tree_codes, const int* tree_count) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  if (b == 0 && threadIdx.x < 8) e.counters[threadIdx.x] = 0;
  if (b >= batch) return;
  const int L = e.L, k = threadIdx.x;
  const bool row_live = e.row_m[b] < L;
  for (int j = 1; j <= L; ++j) {
    const int cnt = row_live ? max(0, min(tree_count[(long long)(j - 1) * batch + b], K)) : 0;
    const int cnt_prev = j > 1 && row_live ? max(0, min(tree_count[(long long)(j - 2) * batch + b], K)) : 0;
    if (k < cnt) {
      const int* src = tree_codes + (((long long)(j - 1) * batch + b) * K + k) * L;
      const long long s = lvl_bk(e, j, b, k);
      bool ok = true;
      for (int l = 0; l < L; ++l) {
        int c = l < j ? src[l] : -1;
        if (l < j && (c < 0 || c >= e.li.T[l])) { atomicOr(e.status, kStBadCode); ok = false; c = 0; }
        e.dw_codes[s * L + l] = c;
      }
      int parent = j == 1 ? 0 : -1;
      if (ok && j > 1) {
        const int* prv = tree_codes + (((long long)(j - 2) * batch + b) * K) * L;
        for (int k2 = 0; k2 < cnt_prev && parent < 0; ++k2) {
          bool eq = true;
          for (int l = 0; l < j - 1; ++l) eq &= (prv[(long long)k2 * L + l] == src[l]);
          if (eq) parent = k2;
        }
      }
      e.dw_score[s] = 0.f;
      e.dw_parent[s] = ok ? parent : -1;
    }
    if (k == 0) e.dw_count[(long long)j * e.Bmax + b] = cnt;
  }
  if (k == 0) e.d_m[b] = L;
}

// Eq. 2 input: x = h_l + s_l for every (request, beam); s_1 = h_0 (Eq. 1).
template <typename T>
__global__ void draft_x_kernel(EngineState e, int batch, int l, T* x) {
  pdl_wait();
  pdl_launch();
  const int bk = blockIdx.x;                       // b * Kmax + k
  const int b = bk / e.Kmax;
  if (b >= batch) return;
  const float* h = e.h_f32 + ((long long)b * (e.L + 1) + l) * e.d;
  const float* s = (l == 1) ? e.h_f32 + (long long)b * (e.L + 1) * e.d
                            : e.state_lv + ((long long)l * e.Bmax * e.Kmax + bk) * e.d;
  const float uh = e.draft_use_h ? 1.f : 0.f, us = e.draft_use_s ? 1.f : 0.f;     // ablations: drop h_l or s_l
  for (int c = threadIdx.x; c < e.d; c += blockDim.x) x[(long long)bk * e.d + c] = from_f32<T>(uh * h[c] + us * s[c]);
}

// Eq. 3 input rows [s_l ; e_l] for the step s_l -> s_{l+1}.
//   requests still teacher-forcing (d_m >= l): beam k of the start set, its own state, its l-th code;
//   requests drafting (d_m < l): survivor k of level l, its parent's state, the code just chosen.
//   ADD = true (ablation: Transition replaced by addition): writes s_{l+1} = s_l + e_l (fp32) itself, no GEMM follows.
template <typename T, bool ADD>
__global__ void trans_gather_kernel(EngineState e, int batch, int l, const T* embed, T* A) {
  pdl_wait();
  pdl_launch();
  const int bk = blockIdx.x;
  const int b = bk / e.Kmax, k = bk - b * e.Kmax;
  if (b >= batch) return;
  T* dst = A + (long long)bk * 2 * e.d;
  float* nxt = e.state_lv + ((long long)(l + 1) * e.Bmax * e.Kmax + bk) * e.d;
  const int dm = e.d_m[b];
  int src_level, parent;
  bool live = dm < e.L || e.row_m[b] < e.L;
  if (dm >= l) { src_level = min(dm, e.L); parent = k; }
  else { src_level = l; parent = -2; }
  const long long s_idx = lvl_bk(e, src_level, b, k);
  live = live && k < e.dw_count[src_level * e.Bmax + b];
  if (live && parent == -2) parent = e.dw_parent[s_idx];
  const int code = live ? e.dw_codes[s_idx * e.L + (l - 1)] : -1;
  live = live && code >= 0 && parent >= 0;
  if (!live) {
    if (ADD) { for (int c = threadIdx.x; c < e.d; c += blockDim.x) nxt[c] = 0.f; }
    else { for (int c = threadIdx.x; c < 2 * e.d; c += blockDim.x) dst[c] = from_f32<T>(0.f); }
    return;
  }
  const float* s = (l == 1) ? e.h_f32 + (long long)b * (e.L + 1) * e.d
                            : e.state_lv + ((long long)l * e.Bmax * e.Kmax + (long long)b * e.Kmax + parent) * e.d;
  const T* emb = embed + (long long)(e.li.off[l - 1] + code) * e.d;
  for (int c = threadIdx.x; c < e.d; c += blockDim.x) {
    if (ADD) { nxt[c] = s[c] + to_f32(emb[c]); }
    else { dst[c] = from_f32<T>(s[c]); dst[e.d + c] = emb[c]; }
  }
}

// ---- the draft head with merged products ---------------------------------------------------------------------
// s_1 = h_0 (Eq. 1) for every beam slot of every request, as the bf16 A operand of the level's product.
__global__ void draft_state_init_kernel(EngineState e, int batch, __nv_bfloat16* s_act) {
  pdl_wait();
  pdl_launch();
  const int bk = blockIdx.x, b = bk / e.Kmax;
  if (b >= batch) return;
  const float* h0 = e.h_f32 + (long long)b * (e.L + 1) * e.d;
  for (int c = threadIdx.x; c < e.d; c += blockDim.x) s_act[(long long)bk * e.d + c] = __float2bfloat16_rn(h0[c]);
}

// Eq. 3 after the product: s_{l+1}[k] = tanh((W_s s_l)[parent] + (W_e E)[code] + b).  G holds [logits | W_s s_l] of
// every beam slot of level l (W_s s_l from column t_cols on), U = W_e E for every code token.  Which (parent, code) a
// slot takes is decided exactly as in trans_gather_kernel.
__device__ __forceinline__ void draft_step_slot(const EngineState& e, int b, int k, int l, const float* __restrict__ G,
                                                long long g_stride, int t_cols, const float* __restrict__ U,
                                                const float* __restrict__ bias, __nv_bfloat16* s_act, int tid, int n_thr) {
  __nv_bfloat16* dst = s_act + ((long long)b * e.Kmax + k) * e.d;
  const int dm = e.d_m[b];
  int src_level, parent;
  bool live = dm < e.L || e.row_m[b] < e.L;
  if (dm >= l) { src_level = min(dm, e.L); parent = k; }
  else { src_level = l; parent = -2; }
  const long long s_idx = lvl_bk(e, src_level, b, k);
  live = live && k < e.dw_count[src_level * e.Bmax + b];
  if (live && parent == -2) parent = e.dw_parent[s_idx];
  const int code = live ? e.dw_codes[s_idx * e.L + (l - 1)] : -1;
  live = live && code >= 0 && parent >= 0;
  if (!live) {
    for (int c = tid; c < e.d; c += n_thr) dst[c] = __float2bfloat16_rn(0.f);
    return;
  }
  const float* z = G + ((long long)b * e.Kmax + parent) * g_stride + t_cols;
  const float* u = U + (long long)(e.li.off[l - 1] + code) * e.d;
  for (int c = tid; c < e.d; c += n_thr) dst[c] = __float2bfloat16_rn(tanhf(z[c] + u[c] + bias[c]));
}
__global__ void draft_step_kernel(EngineState e, int batch, int l, const float* __restrict__ G, long long g_stride, int t_cols,
                                  const float* __restrict__ U, const float* __restrict__ bias, __nv_bfloat16* s_act) {
  pdl_wait();
  pdl_launch();
  const int bk = blockIdx.x;
  const int b = bk / e.Kmax, k = bk - b * e.Kmax;
  if (b >= batch) return;
  draft_step_slot(e, b, k, l, G, g_stride, t_cols, U, bias, s_act, threadIdx.x, blockDim.x);
}
// The selection of draft level l and the state update that follows it, in one launch: a block selects its request's
// beams (or skips that when the request's level is already settled) and then advances the states of its own slots.
template <int VPL>
__global__ void __launch_bounds__(select_max_threads(VPL)) select_step_kernel(SelectArgs a, EngineState e, int l, const float* __restrict__ G,
                                                          long long g_stride, int t_cols, const float* __restrict__ U,
                                                          const float* __restrict__ bias, __nv_bfloat16* s_act) {
  pdl_wait();
  pdl_launch();
  select_body<VPL>(a);
  __syncthreads();                                 // the block's own selection (global writes) is visible to all its threads
  for (int k = threadIdx.x >> 5; k < e.Kmax; k += blockDim.x >> 5)          // a warp per beam slot
    draft_step_slot(e, blockIdx.x, k, l, G, g_stride, t_cols, U, bias, s_act, threadIdx.x & 31, 32);
}

// dst[b, r, :] = src[(b * row_mul + r), 0 : T] + bias[b, :]
__global__ void copy_logits_bias_kernel(const float* src, long long row_stride, int row_mul, int n_beams, int T,
                                        const float* bias, long long bias_stride, float* dst) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x / n_beams, r = blockIdx.x % n_beams;
  const float* z = src + ((long long)b * row_mul + r) * row_stride;
  for (int t = threadIdx.x; t < T; t += blockDim.x) dst[(long long)blockIdx.x * T + t] = z[t] + bias[(long long)b * bias_stride + t];
}

// ----------------------------------------------------------------------------------------------------
// verify-pass token list (the nodes M_p runs on this round)
// ----------------------------------------------------------------------------------------------------
// Request with m levels settled: nodes = the level-m code of every beam of B_m (slot = beam rank) and, for the levels
// m+1..L-1, the last code of every alive node of the round's draft tree (slot = the node's slot in its level): one token
// per distinct drafted prefix.  A level-m node of the tree is alive if its codes are a beam of B_m; a higher node if its
// parent is alive.  Tokens of a request are contiguous; requests are laid out in order (each block sums the counts of the
// requests before it).
__global__ void nodes_count_kernel(EngineState e, int batch) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  const int m = e.row_m[b];
  const int L = e.L;
  __shared__ int n_alive;
  if (threadIdx.x == 0) n_alive = 0;
  if (b == 0 && threadIdx.x == 0) *e.draft_rows = 0;     // this round's drafting is over; round_end raises it again if needed
  __syncthreads();
  if (m >= L) {
    if (threadIdx.x == 0) { e.row_tok_count[b] = 0; e.row_cur[b] = -1; e.req_info[b] = make_int4(0, 0, b, 0); }
    return;
  }
  const int nb = e.tb_count[m * e.Bmax + b];
  for (int j = m; j < L; ++j) {
    const int cnt = min(e.dw_count[(long long)j * e.Bmax + b], e.Kmax);
    for (int k = threadIdx.x; k < e.Kmax; k += blockDim.x) {
      int beta = -1;
      if (k < cnt) {
        if (j == m) {
          const int* dc = e.dw_codes + lvl_bk(e, m, b, k) * L;
          for (int r = 0; r < nb && beta < 0; ++r) {
            const int* bc = e.tb_codes + lvl_bk(e, m, b, r) * L;
            bool eq = true;
            for (int l = 0; l < m; ++l) eq &= (dc[l] == bc[l]);
            if (eq) beta = r;
          }
        } else {
          const int p = e.dw_parent[lvl_bk(e, j, b, k)];
          if (p >= 0 && p < e.Kmax) beta = e.d_beam[lvl_bk(e, j - 1, b, p)];
          if (beta >= 0) atomicAdd(&n_alive, 1);
        }
      }
      e.d_beam[lvl_bk(e, j, b, k)] = beta;
    }
    __syncthreads();                               // level j's answers (global, this block's own) before level j + 1 reads them
  }
  if (threadIdx.x == 0) {
    e.row_tok_count[b] = nb + n_alive;
    e.row_cur[b] = m;
    e.row_m_start[b] = m;
  }
}

__global__ void __launch_bounds__(128) nodes_fill_kernel(EngineState e, int batch) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  const int L = e.L, Kmax = e.Kmax;
  __shared__ int s_off, s_rank[kMaxLevels][128], s_level_start[kMaxLevels + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  const int m = e.row_m[b];
  if (threadIdx.x == 0) {
    int off = 0;
    for (int i = 0; i < b; ++i) off += e.row_tok_count[i];
    s_off = off;
    e.row_tok_start[b] = off;
    if (e.row_tok_count[b] > 0) e.req_info[b] = make_int4(off, e.row_tok_count[b], b, e.row_P[b]);
    if (b == batch - 1) *e.n_tokens = off + e.row_tok_count[b];
  }
  for (int i = threadIdx.x; i < L * Kmax; i += blockDim.x) e.node_index[(long long)b * L * Kmax + i] = -1;
  // rank of every alive node within its level (a warp per level: ballots over its <= 128 slots)
  for (int j = m + 1 + warp; j < L; j += n_warps) {
    int base = 0;
    for (int k0 = 0; k0 < Kmax; k0 += 32) {
      const int k = k0 + lane;
      const bool alive = k < Kmax && k < e.dw_count[(long long)j * e.Bmax + b] && e.d_beam[lvl_bk(e, j, b, k)] >= 0;
      const unsigned mask = __ballot_sync(0xffffffffu, alive);
      if (k < 128) s_rank[j][k] = alive ? base + __popc(mask & ((1u << lane) - 1u)) : -1;
      base += __popc(mask);
    }
    if (lane == 0) s_level_start[j] = base;        // the level's count for now; turned into a start below
  }
  __syncthreads();
  if (m >= L) return;
  const int nb = e.tb_count[m * e.Bmax + b];
  if (threadIdx.x == 0) {
    int start = nb;
    for (int j = m + 1; j < L; ++j) { const int c = s_level_start[j]; s_level_start[j] = start; start += c; }
  }
  __syncthreads();
  const int P = e.row_P[b];
  const long long slab_elems = (long long)Kmax * e.Hkv * e.hd;       // one level slab of one request
  const long long row_elems = (long long)(L - 1) * slab_elems;
  auto kv_off = [&](int level, int slot) {                             // level 1..L-1
    return (long long)b * row_elems + (long long)(level - 1) * slab_elems + (long long)slot * e.Hkv * e.hd;
  };
  // level-m nodes: the true beams
  for (int r = threadIdx.x; r < nb; r += blockDim.x) {
    const int t = s_off + r;
    const long long bi = lvl_bk(e, m, b, r);
    e.tok_row[t] = b; e.tok_pos[t] = P + m - 1; e.tok_ctx_len[t] = P;
    e.tok_id[t] = e.li.off[m - 1] + e.tb_codes[bi * L + (m - 1)];
    e.tok_kv_dst[t] = kv_off(m, r);
    for (int i = 1; i <= L; ++i) {
      long long o = -1;
      if (i < m) o = kv_off(i, e.tb_anc[bi * L + (i - 1)]);
      else if (i == m) o = kv_off(m, r);
      e.tok_ext[(long long)t * L + (i - 1)] = o;
    }
    e.tb_src[bi] = t;
    e.tb_self[bi] = r;
    e.node_index[((long long)b * L + m) * Kmax + r] = t;
  }
  // levels m+1 .. L-1: the alive nodes of the draft tree
  const int n_lv = L - 1 - m;
  for (int idx = threadIdx.x; idx < n_lv * Kmax; idx += blockDim.x) {
    const int j = m + 1 + idx / Kmax, k = idx % Kmax;
    const int rank = s_rank[j][k];
    if (rank < 0) continue;
    const int t = s_off + s_level_start[j] + rank;
    const int beta = e.d_beam[lvl_bk(e, j, b, k)];
    const long long bi = lvl_bk(e, m, b, beta);
    const long long di = lvl_bk(e, j, b, k);
    e.tok_row[t] = b; e.tok_pos[t] = P + j - 1; e.tok_ctx_len[t] = P;
    e.tok_id[t] = e.li.off[j - 1] + e.dw_codes[di * L + (j - 1)];
    e.tok_kv_dst[t] = kv_off(j, k);
    int anc[kMaxLevels + 1];                       // anc[i] = slot of the node's ancestor of level i in the tree
    anc[j] = k;
    for (int i = j; i > m + 1; --i) anc[i - 1] = e.dw_parent[lvl_bk(e, i, b, anc[i])];
    for (int i = 1; i <= L; ++i) {
      long long o = -1;
      if (i < m) o = kv_off(i, e.tb_anc[bi * L + (i - 1)]);
      else if (i == m) o = kv_off(m, beta);
      else if (i <= j) o = kv_off(i, anc[i]);
      e.tok_ext[(long long)t * L + (i - 1)] = o;
    }
    e.node_index[((long long)b * L + j) * Kmax + k] = t;
  }
}

// Teacher-forced nodes: beams given by the caller, every beam processes all of its `level` codes.
__global__ void nodes_from_prefixes_kernel(EngineState e, int batch, int n_beams, int level, const int* prefixes) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  const int L = e.L, Kmax = e.Kmax;
  const int per_row = n_beams * level;
  const int P = e.row_P[b];
  const long long slab_elems = (long long)Kmax * e.Hkv * e.hd;
  const long long row_elems = (long long)(L - 1) * slab_elems;
  if (b == 0 && threadIdx.x == 0) *e.n_tokens = batch * per_row;
  if (threadIdx.x == 0) {
    e.row_tok_start[b] = b * per_row; e.row_tok_count[b] = per_row;
    e.req_info[b] = make_int4(b * per_row, per_row, b, P);
  }
  for (int i = threadIdx.x; i < L * Kmax; i += blockDim.x) e.node_index[(long long)b * L * Kmax + i] = -1;
  __syncthreads();
  for (int idx = threadIdx.x; idx < per_row; idx += blockDim.x) {
    const int j = 1 + idx / n_beams, r = idx % n_beams;
    const int t = b * per_row + idx;
    int code = prefixes[((long long)b * n_beams + r) * level + (j - 1)];
    if (code < 0 || code >= e.li.T[j - 1]) { atomicOr(e.status, kStBadCode); code = 0; }
    e.tok_row[t] = b; e.tok_pos[t] = P + j - 1; e.tok_ctx_len[t] = P;
    e.tok_id[t] = e.li.off[j - 1] + code;
    const long long self = (long long)b * row_elems + (long long)(j - 1) * slab_elems + (long long)r * e.Hkv * e.hd;
    e.tok_kv_dst[t] = self;
    for (int i = 1; i <= L; ++i)
      e.tok_ext[(long long)t * L + (i - 1)] =
          (i <= j) ? (long long)b * row_elems + (long long)(i - 1) * slab_elems + (long long)r * e.Hkv * e.hd : -1;
    e.node_index[((long long)b * L + j) * Kmax + r] = t;
  }
}

// ----------------------------------------------------------------------------------------------------
// accept / roll back (Algorithm 2's rejection and update steps)
// ----------------------------------------------------------------------------------------------------
// After B_{n+1} has been selected for a request whose beams B_n had logits in this pass:
//   n + 1 == L : the request is finished; B_L is the result.
//   otherwise  : every beam of B_{n+1} inherits its parent's KV slots (a slot-table rewrite: rejected drafts'
//                KV rows simply become unreachable) and is matched against the alive nodes of level n+1 of the draft
//                tree.  If every beam is such a node, its hidden state is already in the pass and selection goes on;
//                else level n+1 is the rejection level and the request waits for the next round.
__device__ __forceinline__ void advance_body(const EngineState& e, int n, int K, int* out_codes, float* out_score, int* out_count) {
  const int b = blockIdx.x;
  if (e.row_cur[b] != n) return;
  const int L = e.L, Kmax = e.Kmax;
  const int n1 = n + 1;
  const int cnt = e.tb_count[n1 * e.Bmax + b];
  if (n1 == L) {
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
      const long long s = lvl_bk(e, L, b, k);
      out_score[(long long)b * K + k] = k < cnt ? e.tb_score[s] : -INFINITY;
      for (int l = 0; l < L; ++l) out_codes[((long long)b * K + k) * L + l] = k < cnt ? e.tb_codes[s * L + l] : -1;
    }
    if (threadIdx.x == 0) { out_count[b] = cnt; e.row_m[b] = L; e.row_cur[b] = -1; }
    return;
  }
  __shared__ int all_matched;
  if (threadIdx.x == 0) all_matched = 1;
  __syncthreads();
  const int nd = min(e.dw_count[(long long)n1 * e.Bmax + b], Kmax);
  for (int r = threadIdx.x; r < cnt; r += blockDim.x) {
    const long long bi = lvl_bk(e, n1, b, r);
    const int parent = e.tb_parent[bi];
    const long long pi = lvl_bk(e, n, b, parent);
    for (int i = 0; i + 1 < n; ++i) e.tb_anc[bi * L + i] = e.tb_anc[pi * L + i];
    if (n >= 1) e.tb_anc[bi * L + (n - 1)] = e.tb_self[pi];
    const int* bc = e.tb_codes + bi * L;
    int match = -1;
    for (int k = 0; k < nd && match < 0; ++k) {
      if (e.d_beam[lvl_bk(e, n1, b, k)] < 0) continue;
      const int* dc = e.dw_codes + lvl_bk(e, n1, b, k) * L;
      bool eq = true;
      for (int l = 0; l < n1; ++l) eq &= (dc[l] == bc[l]);
      if (eq) match = k;
    }
    if (match >= 0) {
      e.tb_src[bi] = e.node_index[((long long)b * L + n1) * Kmax + match];
      e.tb_self[bi] = match;
    } else {
      e.tb_src[bi] = -1;
      e.tb_self[bi] = -1;
      all_matched = 0;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    e.row_m[b] = n1;
    e.row_cur[b] = (all_matched && cnt > 0) ? n1 : -1;
    if (cnt == 0) {               // no beam survived (possible only with an empty codebook): finish empty
      e.row_m[b] = L;
      out_count[b] = 0;
    }
  }
}
__global__ void advance_kernel(EngineState e, int batch, int n, int K, int* out_codes, float* out_score, int* out_count) {
  pdl_wait();
  pdl_launch();
  advance_body(e, n, K, out_codes, out_score, out_count);
}
// The selection of B_{n+1} and the step above in one launch (both act on the requests whose current level is n).
template <int VPL>
__global__ void __launch_bounds__(select_max_threads(VPL)) select_advance_kernel(SelectArgs a, EngineState e, int n, int K, int* out_codes,
                                                             float* out_score, int* out_count) {
  pdl_wait();
  pdl_launch();
  select_body<VPL>(a);
  __syncthreads();                                 // the block's own selection (global writes) is visible to all its threads
  advance_body(e, n, K, out_codes, out_score, out_count);
}

// End of a round: accepted length of every draft = the largest i <= (level reached) with D[k][0..i) in B_i;
// trace outputs; counters for the host (unfinished requests, primary tokens, accepted levels).
// adaptive: a request whose round settled only the one level that the pass settles anyway gained nothing from its drafts
// and stops drafting (its remaining rounds are plain autoregressive steps).
__global__ void round_end_kernel(EngineState e, int batch, int K, int round, nezha_trace tr, int adaptive) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  const int L = e.L, Kmax = e.Kmax;
  const int took_part = e.row_tok_count[b] > 0;
  const int m_now = e.row_m[b];
  const int nd = took_part ? e.dw_count[(long long)L * e.Bmax + b] : 0;
  const long long tro = ((long long)(round - 1) * batch + b);
  __shared__ int acc_sum;
  if (threadIdx.x == 0) acc_sum = 0;
  __syncthreads();
  for (int k = threadIdx.x; k < K; k += blockDim.x) {
    int acc = -1;
    if (k < nd) {
      const int* dc = e.dw_codes + lvl_bk(e, L, b, k) * L;
      acc = 0;
      for (int i = 1; i <= m_now; ++i) {
        const int nbi = e.tb_count[i * e.Bmax + b];
        bool in = false;
        for (int r = 0; r < nbi && !in; ++r) {
          const int* bc = e.tb_codes + lvl_bk(e, i, b, r) * L;
          bool eq = true;
          for (int l = 0; l < i; ++l) eq &= (dc[l] == bc[l]);
          in = eq;
        }
        if (in) acc = i; else break;
      }
      atomicAdd(&acc_sum, acc);
    }
    if (tr.accepted_len) tr.accepted_len[tro * K + k] = acc;
    if (tr.drafts)
      for (int l = 0; l < L; ++l)
        tr.drafts[(tro * K + k) * L + l] = (k < nd) ? e.dw_codes[lvl_bk(e, L, b, k) * L + l] : -1;
    if (tr.tree_codes)
      for (int j = 1; j <= L; ++j) {
        const int nj = took_part ? min(e.dw_count[(long long)j * e.Bmax + b], Kmax) : 0;
        const long long o = ((((long long)(round - 1) * L + (j - 1)) * batch + b) * K + k) * L;
        for (int l = 0; l < L; ++l) tr.tree_codes[o + l] = (k < nj && l < j) ? e.dw_codes[lvl_bk(e, j, b, k) * L + l] : -1;
      }
  }
  if (tr.tree_count && threadIdx.x < L)
    tr.tree_count[((long long)(round - 1) * L + threadIdx.x) * batch + b] =
        took_part ? min(min(e.dw_count[(long long)(threadIdx.x + 1) * e.Bmax + b], Kmax), K) : -1;
  __syncthreads();
  if (threadIdx.x == 0) {
    if (tr.n_draft) tr.n_draft[tro] = took_part ? nd : -1;
    if (tr.level_reached) tr.level_reached[tro] = took_part ? m_now : -1;
    if (took_part && adaptive) e.row_spec[b] = (m_now - e.row_m_start[b] >= 2) ? 1 : 0;
    if (m_now < L && e.row_spec[b]) atomicMax(e.draft_rows, batch * Kmax);   // somebody drafts next round
    if (m_now < L) atomicAdd(&e.counters[0], 1);
    atomicAdd(&e.counters[1], e.row_tok_count[b]);
    atomicAdd(&e.counters[2], acc_sum);
    if (round == 1) atomicAdd(&e.counters[3], nd);
  }
}

__global__ void write_out_kernel(const int* codes, const float* score, const int* count, int stride, int L, int K,
                                 int* out_codes, float* out_score, int* out_count) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  const int cnt = min(count[b], K);
  for (int k = threadIdx.x; k < K; k += blockDim.x) {
    const long long s = (long long)b * stride + k;
    out_score[(long long)b * K + k] = k < cnt ? score[s] : -INFINITY;
    for (int l = 0; l < L; ++l) out_codes[((long long)b * K + k) * L + l] = k < cnt ? codes[s * L + l] : -1;
  }
  if (threadIdx.x == 0) out_count[b] = cnt;
}

// dst[b, r, :] = src[row(b, r), col_off : col_off + T],
// row = row_index ? row_index[b*idx_stride + r] : b*row_mul + r*beam_mul
__global__ void copy_logits_kernel(const float* src, long long row_stride, int col_off, const int* row_index, int row_mul,
                                   int beam_mul, int n_beams, int idx_stride, int T, float* dst) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x / n_beams, r = blockIdx.x % n_beams;
  const long long row = row_index ? row_index[(long long)b * idx_stride + r] : (long long)b * row_mul + (long long)r * beam_mul;
  if (row < 0) return;
  for (int t = threadIdx.x; t < T; t += blockDim.x)
    dst[(long long)blockIdx.x * T + t] = src[row * row_stride + col_off + t];
}

__global__ void trace_beams_kernel(EngineState e, int batch, int K, nezha_trace tr) {
  pdl_wait();
  pdl_launch();
  const int b = blockIdx.x;
  const int L = e.L;
  for (int n = 1; n <= L; ++n) {
    const int cnt = e.tb_count[n * e.Bmax + b];
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
      const long long s = lvl_bk(e, n, b, k);
      const long long o = ((long long)(n - 1) * batch + b) * K + k;
      if (tr.beam_scores) tr.beam_scores[o] = k < cnt ? e.tb_score[s] : -INFINITY;
      if (tr.beams)
        for (int l = 0; l < L; ++l) tr.beams[o * L + l] = (k < cnt && l < n) ? e.tb_codes[s * L + l] : -1;
    }
  }
}

}  // namespace

void launch_fill_i32(int* p, long long n, int v, cudaStream_t st) {
  if (n <= 0) return;
  LaunchScope ls(kcMisc, st);
  launch_pdl(fill_i32_kernel, dim3((unsigned)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184)), dim3(256), 0, st, p, n, v);
}
void launch_fill_f32(float* p, long long n, float v, cudaStream_t st) {
  if (n <= 0) return;
  LaunchScope ls(kcMisc, st);
  launch_pdl(fill_f32_kernel, dim3((unsigned)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184)), dim3(256), 0, st, p, n, v);
}
void launch_init_decode(const EngineState& e, int batch, cudaStream_t st) {
  LaunchScope ls(kcMisc, st);
  launch_pdl(init_decode_kernel, dim3((batch + 127) / 128), dim3(128), 0, st, e, batch);
}
void launch_draft_init(const EngineState& e, int batch, int from_scratch, void* s_act, cudaStream_t st) {
  LaunchScope ls(kcDraftGlue, st);
  launch_pdl(draft_init_kernel, dim3(batch), dim3(128), 0, st, e, batch, from_scratch, (__nv_bfloat16*)s_act);
}
void launch_draft_set(const EngineState& e, int batch, int K, const int* drafts, const int* n_draft, cudaStream_t st) {
  LaunchScope ls(kcDraftGlue, st);
  launch_pdl(draft_set_kernel, dim3(batch), dim3(128), 0, st, e, batch, K, drafts, n_draft);
}
void launch_draft_tree_set(const EngineState& e, int batch, int K, const int* tree_codes, const int* tree_count, cudaStream_t st) {
  LaunchScope ls(kcDraftGlue, st);
  launch_pdl(draft_tree_set_kernel, dim3(batch), dim3(128), 0, st, e, batch, K, tree_codes, tree_count);
}
void launch_draft_x(const EngineState& e, int batch, int l, void* x, bool bf16, cudaStream_t st) {
  LaunchScope ls(kcDraftGlue, st);
  if (bf16) launch_pdl(draft_x_kernel<__nv_bfloat16>, dim3(batch * e.Kmax), dim3(128), 0, st, e, batch, l, (__nv_bfloat16*)x);
  else launch_pdl(draft_x_kernel<float>, dim3(batch * e.Kmax), dim3(128), 0, st, e, batch, l, (float*)x);
}
void launch_trans_gather(const EngineState& e, int batch, int l, const void* embed, void* A, bool bf16,
                         cudaStream_t st) {
  LaunchScope ls(kcDraftGlue, st);
  if (bf16)
    launch_pdl(trans_gather_kernel<__nv_bfloat16, false>, dim3(batch * e.Kmax), dim3(128), 0, st, e, batch, l, (const __nv_bfloat16*)embed,
                                                                      (__nv_bfloat16*)A);
  else launch_pdl(trans_gather_kernel<float, false>, dim3(batch * e.Kmax), dim3(128), 0, st, e, batch, l, (const float*)embed, (float*)A);
}
void launch_trans_add(const EngineState& e, int batch, int l, const void* embed, bool bf16, cudaStream_t st) {
  LaunchScope ls(kcDraftGlue, st);
  if (bf16)
    launch_pdl(trans_gather_kernel<__nv_bfloat16, true>, dim3(batch * e.Kmax), dim3(128), 0, st, e, batch, l,
               (const __nv_bfloat16*)embed, (__nv_bfloat16*)nullptr);
  else
    launch_pdl(trans_gather_kernel<float, true>, dim3(batch * e.Kmax), dim3(128), 0, st, e, batch, l, (const float*)embed,
               (float*)nullptr);
}
void launch_draft_state_init(const EngineState& e, int batch, void* s_act, cudaStream_t st) {
  LaunchScope ls(kcDraftGlue, st);
  launch_pdl(draft_state_init_kernel, dim3(batch * e.Kmax), dim3(128), 0, st, e, batch, (__nv_bfloat16*)s_act);
}
void launch_draft_step(const EngineState& e, int batch, int l, const float* G, long long g_stride, int t_cols, const float* U,
                       const float* bias, void* s_act, cudaStream_t st) {
  LaunchScope ls(kcDraftGlue, st);
  launch_pdl(draft_step_kernel, dim3(batch * e.Kmax), dim3(128), 0, st, e, batch, l, G, g_stride, t_cols, U, bias,
             (__nv_bfloat16*)s_act);
}
cudaError_t select_step_configure(int bytes) {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(select_advance_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_advance_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_advance_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_advance_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_step_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_step_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  if ((e = cudaFuncSetAttribute(select_step_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return e;
  return cudaFuncSetAttribute(select_step_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}
void launch_select_step(const SelectArgs& a, const EngineState& e, int l, const float* G, long long g_stride, int t_cols,
                        const float* U, const float* bias, void* s_act, cudaStream_t st) {
  if (a.batch <= 0) return;
  const size_t smem = select_smem_bytes(a.in_stride, a.K);
  LaunchScope ls(kcSelect, st);
  const int warps = select_warps(a);
  const dim3 block(32 * warps), grid(a.batch);
  __nv_bfloat16* s = (__nv_bfloat16*)s_act;
  if (a.T <= 32) launch_pdl(select_step_kernel<1>, grid, block, smem, st, a, e, l, G, g_stride, t_cols, U, bias, s);
  else if (a.T <= 256) launch_pdl(select_step_kernel<8>, grid, block, smem, st, a, e, l, G, g_stride, t_cols, U, bias, s);
  else if (a.T <= 512) launch_pdl(select_step_kernel<16>, grid, block, smem, st, a, e, l, G, g_stride, t_cols, U, bias, s);
  else launch_pdl(select_step_kernel<32>, grid, block, smem, st, a, e, l, G, g_stride, t_cols, U, bias, s);
}
void launch_copy_logits_bias(const float* src, long long row_stride, int row_mul, int batch, int n_beams, int T,
                             const float* bias, long long bias_stride, float* dst, cudaStream_t st) {
  LaunchScope ls(kcMisc, st);
  launch_pdl(copy_logits_bias_kernel, dim3(batch * n_beams), dim3(128), 0, st, src, row_stride, row_mul, n_beams, T, bias,
             bias_stride, dst);
}
void launch_build_nodes(const EngineState& e, int batch, cudaStream_t st) {
  LaunchScope ls(kcNodes, st, 2);
  launch_pdl(nodes_count_kernel, dim3(batch), dim3(64), 0, st, e, batch);
  launch_pdl(nodes_fill_kernel, dim3(batch), dim3(128), 0, st, e, batch);
}
void launch_nodes_from_prefixes(const EngineState& e, int batch, int n_beams, int level, const int* prefixes,
                                cudaStream_t st) {
  LaunchScope ls(kcNodes, st);
  launch_pdl(nodes_from_prefixes_kernel, dim3(batch), dim3(128), 0, st, e, batch, n_beams, level, prefixes);
}
void launch_advance(const EngineState& e, int batch, int n, int K, int* out_codes, float* out_score, int* out_count,
                    cudaStream_t st) {
  LaunchScope ls(kcAccept, st);
  launch_pdl(advance_kernel, dim3(batch), dim3(64), 0, st, e, batch, n, K, out_codes, out_score, out_count);
}
void launch_select_advance(const SelectArgs& a, const EngineState& e, int n, int K, int* out_codes, float* out_score,
                           int* out_count, cudaStream_t st) {
  if (a.batch <= 0) return;
  const size_t smem = select_smem_bytes(a.in_stride, a.K);
  LaunchScope ls(kcSelect, st);
  const int warps = select_warps(a);
  const dim3 block(32 * warps), grid(a.batch);
  if (a.T <= 32) launch_pdl(select_advance_kernel<1>, grid, block, smem, st, a, e, n, K, out_codes, out_score, out_count);
  else if (a.T <= 256) launch_pdl(select_advance_kernel<8>, grid, block, smem, st, a, e, n, K, out_codes, out_score, out_count);
  else if (a.T <= 512) launch_pdl(select_advance_kernel<16>, grid, block, smem, st, a, e, n, K, out_codes, out_score, out_count);
  else launch_pdl(select_advance_kernel<32>, grid, block, smem, st, a, e, n, K, out_codes, out_score, out_count);
}
void launch_round_end(const EngineState& e, int batch, int K, int round, const nezha_trace& tr, int adaptive, cudaStream_t st) {
  LaunchScope ls(kcAccept, st);
  launch_pdl(round_end_kernel, dim3(batch), dim3(64), 0, st, e, batch, K, round, tr, adaptive);
}
void launch_write_out(const int* codes, const float* score, const int* count, int stride, int L, int batch, int K,
                      int* out_codes, float* out_score, int* out_count, cudaStream_t st) {
  LaunchScope ls(kcMisc, st);
  launch_pdl(write_out_kernel, dim3(batch), dim3(64), 0, st, codes, score, count, stride, L, K, out_codes, out_score, out_count);
}
void launch_copy_logits(const float* src, long long row_stride, int col_off, const int* row_index, int row_mul,
                        int beam_mul, int batch, int n_beams, int idx_stride, int T, float* dst, cudaStream_t st) {
  LaunchScope ls(kcMisc, st);
  launch_pdl(copy_logits_kernel, dim3(batch * n_beams), dim3(128), 0, st, src, row_stride, col_off, row_index, row_mul, beam_mul, n_beams,
                                                      idx_stride, T, dst);
}

// Prompt tokens of a chunk of requests: [BOS, history codes item by item, SP_1..SP_L], padded with BOS up to
// S_call positions (padding sits after the real tokens, so causal attention never shows it to them).
__global__ void prefill_tokens_kernel(EngineState e, const int* hist, const int* n_hist, int b0, int rows, int max_n,
                                      int S_call, int S_cap, int* h_rows) {
  pdl_wait();
  pdl_launch();
  const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (idx >= (long long)rows * S_call) return;
  const int lb = (int)(idx / S_call), p = (int)(idx % S_call), b = b0 + lb;
  const int L = e.L;
  int nh = n_hist[b];
  if (nh < 0 || nh > max_n) { atomicOr(e.status, kStBadCode); nh = nh < 0 ? 0 : max_n; }
  const int P = 1 + nh * L;
  const int bos = e.li.vocab_codes + L;
  int tok = bos;
  if (p > 0 && p < P) {
    const int item = (p - 1) / L, lv = (p - 1) % L;
    int code = hist[((long long)b * max_n + item) * L + lv];
    if (code < 0 || code >= e.li.T[lv]) { atomicOr(e.status, kStBadCode); code = 0; }
    tok = e.li.off[lv] + code;
  } else if (p >= P && p < P + L) {
    tok = e.li.vocab_codes + (p - P);
  }
  e.tok_id[idx] = tok; e.tok_pos[idx] = p; e.tok_row[idx] = b; e.tok_ctx_len[idx] = p + 1;
  e.tok_kv_dst[idx] = ((long long)b * e.Hkv * S_cap + p) * e.hd;
  if (p == 0) {
    e.row_P[b] = P; e.pf_row_start[lb] = lb * S_call; e.pf_row_count[lb] = S_call;
    e.pf_req_info[lb] = make_int4(lb * S_call, S_call, b, -1);
  }
  if (p >= P - 1 && p <= P - 1 + L) h_rows[lb * (L + 1) + (p - (P - 1))] = (int)idx;
}

void launch_prefill_tokens(const EngineState& e, const int* hist, const int* n_hist, int b0, int rows, int max_n,
                           int S_call, int S_cap, int* h_rows, cudaStream_t st) {
  const long long n = (long long)rows * S_call;
  LaunchScope ls(kcNodes, st);
  launch_pdl(prefill_tokens_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, st, e, hist, n_hist, b0, rows, max_n, S_call, S_cap, h_rows);
}
void launch_trace_beams(const EngineState& e, int batch, int K, const nezha_trace& tr, cudaStream_t st) {
  LaunchScope ls(kcMisc, st);
  launch_pdl(trace_beams_kernel, dim3(batch), dim3(64), 0, st, e, batch, K, tr);
}

}  // namespace nz
