// C ABI and host-side engine: arena layout, weight re-layout, prefill, the draft / verify / accept round loop.
// No model arithmetic happens on the host; it only orders kernel launches.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <array>
#include <map>
#include <string>
#include <vector>

#include "common.cuh"
#include "engine_state.cuh"

namespace nz {
void launch_hs_clear(HashSetView hs, cudaStream_t st);
void launch_hs_pack(const LevelInfo& li, const int* codes, unsigned long long n, unsigned long long* keys, int* status,
                    cudaStream_t st);
void launch_hs_insert(const LevelInfo& li, HashSetView hs, const int* codes, unsigned long long n,
                      unsigned long long* n_unique, int* status, cudaStream_t st);
void launch_pm_build(const LevelInfo& li, PrefixMapView pm, const int* codes, unsigned long long n, int* status, cudaStream_t st);
void launch_hs_probe(HashSetView hs, const unsigned long long* keys, unsigned long long n, uint8_t* found,
                     cudaStream_t st);
void launch_prefill_tokens(const EngineState& e, const int* hist, const int* n_hist, int b0, int rows, int max_n,
                           int S_call, int S_cap, int* h_rows, cudaStream_t st);
unsigned long long profile_total_launches();
void profile_enable(bool on);
bool profile_is_on();
void profile_counts(long long* out);
void profile_add(const long long* delta);
void profile_read(nezha_profile* out);
bool gemm_tc_supported(const GemmArgs& a);
void launch_gemm_tc(const GemmArgs& a, cudaStream_t st);
bool attention_tc_supported(const AttnArgs& a);
void launch_attention_tc(const AttnArgs& a, cudaStream_t st);
}  // namespace nz

using namespace nz;

namespace {

struct Carver {
  char* base; size_t off;
  template <typename T> T* take(size_t n) {
    off = (off + 255) & ~(size_t)255;
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
  void* take_bytes(size_t n) { return take<char>(n); }
};

struct LayerW { void *attn_norm, *wqkv, *wo, *mlp_norm, *w_gu, *w_down; };

}  // namespace

struct nezha_ctx {
  nezha_config cfg;
  bool bf16; size_t esz;
  int d, hd, Hq, Hkv, F, nl, L, Bmax, Kmax, S, vocab, Tmax, Nv, qkv_dim;
  long long Ms, Mv_max; int chunk_rows;
  size_t n_items; double load_factor;
  const int32_t* catalog;
  cudaStream_t st;
  char* arena; size_t arena_bytes;
  // weights (arena copies)
  void *embed, *lm_head, *final_norm, *draft_logit[kMaxLevels], *draft_wse, *draft_b_f32;
  std::vector<LayerW> layers;
  // caches
  void *k_ctx, *v_ctx, *k_ext, *v_ext;
  long long ctx_layer_elems, ext_layer_elems;
  float *rope_cos, *rope_sin;
  // scratch
  float* resid; void *xn, *qkv, *attn, *gu, *act, *xd, *a_se, *h_act;
  float *h_f32, *logits_v, *logits0, *logits_d;
  // fused tensor-core path: RMSNorm split around the GEMMs (partial sums of squares per output tile), SwiGLU and
  // rotary embedding + KV append in GEMM epilogues; weights of q/k heads and gate/up re-laid-out to match
  bool fused; float *ss_a, *ss_b, *ss_e;
  // draft head with merged products (fused path, default options): [W_logit_l ; W_s] per level, U = E W_e^T for every
  // code token, H_l = W_logit_l h_l per request, the level's states as a bf16 A operand, the level's product
  void* draft_wcat[kMaxLevels]; float* draft_u; float* draft_hl; void* draft_sact; float* draft_g;
  int* h_rows; unsigned long long* n_unique_dev;
  EngineState es;
  int* host_counters;       // pinned
  // CUDA graphs of the decode segments (one per round), keyed by everything that shapes the launch sequence
  struct Segment { int seen; cudaGraphExec_t exec; long long launches[kcCount]; };
  std::map<std::array<uintptr_t, 16>, Segment> segments;
  bool use_graphs;
  int opt_transition, opt_inputs, opt_filter;   // nezha_set_option (ablations of the draft head)
  int opt_mask;             // nezha_set_option: 0 = the primary model's last-level mask probes the hash set, 1 (default) = it reads the prefix map
  int opt_adaptive;         // nezha_set_option: 1 = a request stops drafting after a round that gained nothing from its drafts
  int opt_level_filter;     // nezha_set_option: 1 = validity filter at every level (prefixes of valid IDs), 0 (default) = last level only
  int m_expected;           // tokens the current verify pass is expected to hold (0 = unknown); shapes GEMM tiling only
  int m_seen[kMaxLevels + 1];   // tokens each round of the last decode call processed, rounded up to a row tile
  int chains_now;           // GemmArgs::chains of the products being queued: 2 inside a decode call, 0 otherwise
  // Weight-streaming products: an engine none of whose decode passes can exceed kSkinnyRows rows runs every product of a
  // decode call through that kernel (the choice is per engine, so both decode modes compute the same bits).
  bool skinny_decode;
  int skinny_now;           // GemmArgs::skinny of the products being queued
  int rounds_seen[3];       // rounds the last decode call of each mode needed: that many are launched without waiting
  int device;               // the GPU that was current at nezha_create
  int state;                // 0 created, 1 hash set built, 2 prefilled
  int batch;                // prefilled batch
  std::string err;
};

namespace {

nezha_status fail(nezha_ctx* c, nezha_status s, const std::string& msg) {
  if (c) c->err = msg;
  return s;
}

#define NZ_CUDA(c, call)                                                                   \
  do {                                                                                     \
    cudaError_t e_ = (call);                                                               \
    if (e_ != cudaSuccess)                                                                 \
      return fail((c), NEZHA_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); \
  } while (0)

bool check_config(const nezha_config* cfg, std::string* why) {
  auto bad = [&](const char* m) { *why = m; return false; };
  if (!cfg) return bad("null config");
  if (cfg->L < 1 || cfg->L > kMaxLevels) return bad("L out of range");
  if (cfg->n_layers < 1 || cfg->d_model < 8 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->d_ffn < 1)
    return bad("bad model shape");
  if (cfg->d_model % cfg->n_q_heads) return bad("d_model not divisible by n_q_heads");
  if (cfg->n_q_heads % cfg->n_kv_heads) return bad("n_q_heads not divisible by n_kv_heads");
  const int hd = cfg->d_model / cfg->n_q_heads;
  if (hd != 16 && hd != 32 && hd != 64 && hd != 128) return bad("head_dim must be 16, 32, 64 or 128");
  if (cfg->dtype != 0 && cfg->dtype != 1) return bad("dtype must be 0 or 1");
  if (cfg->max_batch < 1 || cfg->max_beam < 1 || cfg->max_beam > 128 || cfg->max_hist_items < 0)
    return bad("max_batch / max_beam (<= 128) / max_hist_items out of range");
  long double space = 1;
  for (int l = 0; l < cfg->L; ++l) {
    if (cfg->T[l] < 1 || cfg->T[l] > 1024) return bad("codebook size must be in [1, 1024]");
    space *= cfg->T[l];
  }
  if (space >= 18446744073709551615.0L) return bad("prod(T) must be below 2^64 - 1");
  return true;
}

unsigned long long bucket_count(size_t n_items, double lf) {
  double slots = ceil((double)(n_items ? n_items : 1) / lf);
  unsigned long long nb = (unsigned long long)ceil(slots / kBucketSlots);
  return nb < 2 ? 2 : nb;
}

// Lays the arena out; with c->arena == nullptr only the size is computed.
size_t carve(nezha_ctx* c) {
  const nezha_config& g = c->cfg;
  c->bf16 = g.dtype == 1; c->esz = c->bf16 ? 2 : 4;
  c->d = g.d_model; c->Hq = g.n_q_heads; c->Hkv = g.n_kv_heads; c->hd = c->d / c->Hq; c->F = g.d_ffn;
  c->nl = g.n_layers; c->L = g.L; c->Bmax = g.max_batch; c->Kmax = g.max_beam;
  c->S = 1 + g.max_hist_items * g.L + g.L;
  c->qkv_dim = (c->Hq + 2 * c->Hkv) * c->hd;
  LevelInfo& li = c->es.li;
  li.L = g.L; li.vocab_codes = 0; c->Tmax = 0;
  unsigned long long mult = 1;
  for (int l = 0; l < kMaxLevels; ++l) { li.T[l] = 0; li.off[l] = 0; li.mult[l] = 0; }
  for (int l = 0; l < g.L; ++l) {
    li.T[l] = g.T[l]; li.off[l] = li.vocab_codes; li.mult[l] = mult;
    li.vocab_codes += g.T[l]; mult *= (unsigned long long)g.T[l];
    if (g.T[l] > c->Tmax) c->Tmax = g.T[l];
  }
  c->vocab = li.vocab_codes + g.L + 1;
  c->Nv = li.vocab_codes - g.T[0];
  c->Mv_max = (long long)c->Bmax * c->Kmax * (g.L > 1 ? g.L - 1 : 1);
  c->chunk_rows = (int)(16384 / c->S); if (c->chunk_rows < 1) c->chunk_rows = 1;
  if (c->chunk_rows > c->Bmax) c->chunk_rows = c->Bmax;
  c->Ms = (long long)c->chunk_rows * c->S;
  if (c->Mv_max > c->Ms) c->Ms = c->Mv_max;
  if ((long long)c->Bmax * c->Kmax > c->Ms) c->Ms = (long long)c->Bmax * c->Kmax;

  Carver cv{c->arena, 0};
  EngineState& e = c->es;
  e.Bmax = c->Bmax; e.Kmax = c->Kmax; e.L = c->L; e.d = c->d; e.Hkv = c->Hkv; e.hd = c->hd;
  e.draft_use_h = 1; e.draft_use_s = 1; e.draft_additive = 0;
  e.status = cv.take<int>(8);
  e.counters = cv.take<int>(8);
  c->n_unique_dev = cv.take<unsigned long long>(1);
  e.hs.n_buckets = bucket_count(c->n_items, c->load_factor);
  e.hs.slots = cv.take<unsigned long long>(e.hs.n_buckets * kBucketSlots);
  {  // prefix map: for every prefix length n < L at most one slot per item and per possible prefix, at the hash set's
     // load factor; slots hold the bit set of the widest codebook
    const double items = (double)(c->n_items ? c->n_items : 1);
    double prefixes = 1.0;
    unsigned long long total = 0;
    for (int n = 0; n < g.L; ++n) {
      if (n > 0) prefixes *= (double)g.T[n - 1];
      const double n_pref = prefixes < items ? prefixes : items;
      e.pm.level_off[n] = total;
      e.pm.level_slots[n] = (unsigned long long)ceil(n_pref / c->load_factor) + 1;
      total += e.pm.level_slots[n];
    }
    for (int n = g.L; n < kMaxLevels; ++n) { e.pm.level_off[n] = 0; e.pm.level_slots[n] = 0; }
    e.pm.n_slots = total;
    int words = 1 + (c->Tmax + 63) / 64, stride = 2;
    while (stride < words) stride *= 2;
    e.pm.stride = stride;
    e.pm.slots = cv.take<unsigned long long>(e.pm.n_slots * (unsigned long long)stride);
  }
  // weights
  const size_t esz = c->esz;
  c->embed = cv.take_bytes((size_t)c->vocab * c->d * esz);
  c->lm_head = cv.take_bytes((size_t)c->vocab * c->d * esz);
  c->final_norm = cv.take_bytes((size_t)c->d * esz);
  c->layers.resize(c->nl);
  for (int i = 0; i < c->nl; ++i) {
    LayerW& w = c->layers[i];
    w.attn_norm = cv.take_bytes((size_t)c->d * esz);
    w.wqkv = cv.take_bytes((size_t)c->qkv_dim * c->d * esz);
    w.wo = cv.take_bytes((size_t)c->d * c->Hq * c->hd * esz);
    w.mlp_norm = cv.take_bytes((size_t)c->d * esz);
    w.w_gu = cv.take_bytes((size_t)2 * c->F * c->d * esz);
    w.w_down = cv.take_bytes((size_t)c->d * c->F * esz);
  }
  for (int l = 0; l < c->L; ++l) c->draft_logit[l] = cv.take_bytes((size_t)g.T[l] * c->d * esz);
  c->draft_wse = cv.take_bytes((size_t)c->d * 2 * c->d * esz);
  c->draft_b_f32 = cv.take<float>(c->d);
  // KV caches
  c->ctx_layer_elems = (long long)c->Bmax * c->Hkv * c->S * c->hd;
  c->ext_layer_elems = (long long)c->Bmax * (c->L > 1 ? c->L - 1 : 1) * c->Kmax * c->Hkv * c->hd;
  c->k_ctx = cv.take_bytes((size_t)c->nl * c->ctx_layer_elems * esz);
  c->v_ctx = cv.take_bytes((size_t)c->nl * c->ctx_layer_elems * esz);
  c->k_ext = cv.take_bytes((size_t)c->nl * c->ext_layer_elems * esz);
  c->v_ext = cv.take_bytes((size_t)c->nl * c->ext_layer_elems * esz);
  c->rope_cos = cv.take<float>((size_t)(c->S + c->L) * (c->hd / 2));
  c->rope_sin = cv.take<float>((size_t)(c->S + c->L) * (c->hd / 2));
  // scratch
  c->resid = cv.take<float>((size_t)c->Ms * c->d);
  c->xn = cv.take_bytes((size_t)c->Ms * c->d * esz);
  c->qkv = cv.take_bytes((size_t)c->Ms * c->qkv_dim * esz);
  c->attn = cv.take_bytes((size_t)c->Ms * c->Hq * c->hd * esz);
  c->gu = cv.take_bytes((size_t)c->Ms * 2 * c->F * esz);
  c->act = cv.take_bytes((size_t)c->Ms * c->F * esz);
  c->xd = cv.take_bytes((size_t)c->Bmax * c->Kmax * c->d * esz);
  c->a_se = cv.take_bytes((size_t)c->Bmax * c->Kmax * 2 * c->d * esz);
  c->h_act = cv.take_bytes((size_t)c->Bmax * (c->L + 1) * c->d * esz);
  c->h_f32 = cv.take<float>((size_t)c->Bmax * (c->L + 1) * c->d);
  c->logits_v = cv.take<float>((size_t)c->Mv_max * (c->Nv > 0 ? c->Nv : 1));
  c->logits0 = cv.take<float>((size_t)c->Bmax * g.T[0]);
  c->logits_d = cv.take<float>((size_t)c->Bmax * c->Kmax * c->Tmax);
  c->h_rows = cv.take<int>((size_t)c->Bmax * (c->L + 1));
  c->fused = c->bf16 && (c->hd == 64 || c->hd == 128) && c->d % 64 == 0 && c->F % 64 == 0;
  c->ss_a = c->ss_b = c->ss_e = nullptr;
  c->draft_u = c->draft_hl = c->draft_g = nullptr; c->draft_sact = nullptr;
  for (int l = 0; l < kMaxLevels; ++l) c->draft_wcat[l] = nullptr;
  if (c->fused) {
    for (int l = 0; l < c->L; ++l) c->draft_wcat[l] = cv.take_bytes((size_t)(g.T[l] + c->d) * c->d * esz);
    c->draft_u = cv.take<float>((size_t)li.vocab_codes * c->d);
    c->draft_hl = cv.take<float>((size_t)c->L * c->Bmax * c->Tmax);
    c->draft_sact = cv.take_bytes((size_t)c->Bmax * c->Kmax * c->d * esz);
    c->draft_g = cv.take<float>((size_t)c->Bmax * c->Kmax * (c->Tmax + c->d));
    c->ss_a = cv.take<float>((size_t)(c->d / 32) * c->Ms);      // one partial sum per 32 columns
    c->ss_b = cv.take<float>((size_t)(c->d / 32) * c->Ms);
    c->ss_e = cv.take<float>((size_t)c->Ms);
  }
  // engine state
  const size_t lbk = (size_t)(c->L + 1) * c->Bmax * c->Kmax;
  e.tb_codes = cv.take<int>(lbk * c->L); e.tb_score = cv.take<float>(lbk); e.tb_parent = cv.take<int>(lbk);
  e.tb_count = cv.take<int>((size_t)(c->L + 1) * c->Bmax);
  e.tb_anc = cv.take<int>(lbk * c->L); e.tb_self = cv.take<int>(lbk); e.tb_src = cv.take<int>(lbk);
  e.row_m = cv.take<int>(c->Bmax); e.row_cur = cv.take<int>(c->Bmax); e.row_P = cv.take<int>(c->Bmax);
  e.row_m_start = cv.take<int>(c->Bmax); e.row_spec = cv.take<int>(c->Bmax); e.draft_rows = cv.take<int>(1);
  e.dw_codes = cv.take<int>(lbk * c->L); e.dw_score = cv.take<float>(lbk); e.dw_parent = cv.take<int>(lbk);
  e.dw_count = cv.take<int>((size_t)(c->L + 1) * c->Bmax);
  e.d_m = cv.take<int>(c->Bmax);
  e.d_beam = cv.take<int>(lbk);
  e.state_lv = cv.take<float>(lbk * c->d);
  e.node_index = cv.take<int>((size_t)c->Bmax * c->L * c->Kmax);
  e.tok_row = cv.take<int>(c->Ms); e.tok_pos = cv.take<int>(c->Ms); e.tok_id = cv.take<int>(c->Ms);
  e.tok_ctx_len = cv.take<int>(c->Ms); e.tok_kv_dst = cv.take<long long>(c->Ms);
  e.tok_ext = cv.take<long long>((size_t)c->Mv_max * c->L);
  e.row_tok_count = cv.take<int>(c->Bmax); e.n_tokens = cv.take<int>(1);
  e.row_tok_start = cv.take<int>(c->Bmax); e.pf_row_start = cv.take<int>(c->Bmax); e.pf_row_count = cv.take<int>(c->Bmax);
  e.req_info = cv.take<int4>(c->Bmax); e.pf_req_info = cv.take<int4>(c->Bmax);
  e.h_f32 = c->h_f32;
  return (cv.off + 255) & ~(size_t)255;
}

void gemm(nezha_ctx* c, const void* A, long long lda, const void* W, long long ldw, void* C, long long ldc, long long M,
          const int* M_dev, int N, int K, int epi, const float* bias = nullptr) {
  GemmArgs a{A, lda, W, ldw, C, ldc, (int)M, M_dev, N, K, epi, bias, c->es.status};
  a.chains = c->chains_now;
  a.skinny = c->skinny_now;
  if (c->bf16 && gemm_tc_supported(a)) launch_gemm_tc(a, c->st);
  else launch_gemm_simt(a, c->bf16, c->st);
}

// A projection of the fused tensor-core path.  ss_in / parts: partial sums of squares of the A operand's rows (its
// RMSNorm scale is applied in the epilogue), or null.  Returns the number of partial sums per row a kEpiAddNorm
// epilogue of this launch writes (one per 32 columns).
int gemm_fused(nezha_ctx* c, const void* A, long long lda, const void* W, void* C, long long ldc, long long M,
               const int* M_dev, int N, int K, int epi, const float* ss_in, int ss_parts, const GemmFuse* extra) {
  GemmArgs a{A, lda, W, (long long)K, C, ldc, (int)M, M_dev, N, K, epi, nullptr, c->es.status};
  if (extra) a.f = *extra;
  a.f.ss_in = ss_in; a.f.ss_in_parts = ss_parts; a.f.ss_ld = c->Ms; a.f.inv_dim = 1.f / (float)c->d; a.f.eps = c->cfg.rms_eps;
  a.M_expected = c->m_expected;
  a.chains = c->chains_now;
  a.skinny = c->skinny_now;
  launch_gemm_tc(a, c->st);
  return N / 32;
}

// The layers of the primary model on the fused path.  On entry resid holds the embeddings, xn = embedding * gain of
// the first attention norm and ss_e the rows' sums of squares (launch_embed_norm).  Five kernels per layer:
// QKV projection (+ norm scale, rotary embedding, KV append) -> attention -> output projection (+ residual, next
// norm input) -> gate/up projection (+ norm scale, SwiGLU) -> down projection (+ residual, next norm input).
// On exit xn = resid * final-norm gain and *ss_out / *parts_out describe its row scale.
void run_layers_fused(nezha_ctx* c, long long M, const int* M_dev, bool verify, int n_rows, int max_tok_per_row,
                      const float** ss_out, int* parts_out) {
  const EngineState& e = c->es;
  const size_t esz = c->esz;
  const float* ss_cur = c->ss_e; int parts_cur = 1;
  for (int i = 0; i < c->nl; ++i) {
    const LayerW& w = c->layers[i];
    char* kc = (char*)c->k_ctx + (size_t)i * c->ctx_layer_elems * esz;
    char* vc = (char*)c->v_ctx + (size_t)i * c->ctx_layer_elems * esz;
    char* ke = (char*)c->k_ext + (size_t)i * c->ext_layer_elems * esz;
    char* ve = (char*)c->v_ext + (size_t)i * c->ext_layer_elems * esz;
    GemmFuse fr{};
    fr.tok_pos = e.tok_pos; fr.kv_dst = e.tok_kv_dst; fr.kv_head_stride = verify ? c->hd : (long long)c->S * c->hd;
    fr.k_cache = verify ? ke : kc; fr.v_cache = verify ? ve : vc; fr.cos_tab = c->rope_cos; fr.sin_tab = c->rope_sin;
    fr.Hq = c->Hq; fr.Hkv = c->Hkv; fr.hd = c->hd;
    gemm_fused(c, c->xn, c->d, w.wqkv, c->qkv, c->qkv_dim, M, M_dev, c->qkv_dim, c->d, kEpiRopeKV, ss_cur, parts_cur, &fr);
    AttnArgs t{};
    t.q = c->qkv; t.q_stride = c->qkv_dim; t.out = c->attn; t.out_stride = (long long)c->Hq * c->hd;
    t.k_ctx = kc; t.v_ctx = vc; t.ctx_row_stride = (long long)c->Hkv * c->S * c->hd; t.ctx_head_stride = (long long)c->S * c->hd;
    t.k_ext = ke; t.v_ext = ve; t.ext_head_stride = c->hd;
    t.tok_row = e.tok_row; t.tok_ctx_len = e.tok_ctx_len; t.tok_ext = e.tok_ext; t.n_ext_max = verify ? c->L : 0;
    t.M = (int)M; t.M_dev = M_dev; t.Hq = c->Hq; t.Hkv = c->Hkv; t.hd = c->hd; t.scale = 1.f / sqrtf((float)c->hd);
    t.row_start = verify ? e.row_tok_start : e.pf_row_start; t.row_count = verify ? e.row_tok_count : e.pf_row_count;
    t.req_info = verify ? e.req_info : e.pf_req_info;
    t.n_rows = n_rows; t.max_tokens_per_row = max_tok_per_row;
    t.rows_expected = (c->m_expected > 0 && n_rows > 0) ? (c->m_expected + n_rows - 1) / n_rows * (c->Hq / c->Hkv) : 0;
    t.ctx_rows_total = (long long)c->Bmax * c->Hkv * c->S; t.status = e.status;
    t.ext_positions = (c->L > 1 ? c->L - 1 : 1) * c->Kmax; t.ext_pos_stride = (long long)c->Hkv * c->hd;
    t.ext_req_stride = t.ext_positions * t.ext_pos_stride; t.ext_rows_total = (long long)c->Bmax * t.ext_positions;
    if (attention_tc_supported(t)) launch_attention_tc(t, c->st);
    else launch_attention_simt(t, true, c->st);
    GemmFuse fo{};
    fo.xg = c->xn; fo.gain = w.mlp_norm; fo.ss_out = c->ss_a;
    const int parts_a = gemm_fused(c, c->attn, (long long)c->Hq * c->hd, w.wo, c->resid, c->d, M, M_dev, c->d, c->Hq * c->hd,
                                   kEpiAddNorm, nullptr, 0, &fo);
    gemm_fused(c, c->xn, c->d, w.w_gu, c->act, c->F, M, M_dev, 2 * c->F, c->d, kEpiSwiGLU, c->ss_a, parts_a, nullptr);
    GemmFuse fd{};
    fd.xg = c->xn; fd.gain = (i + 1 < c->nl) ? c->layers[i + 1].attn_norm : c->final_norm; fd.ss_out = c->ss_b;
    parts_cur = gemm_fused(c, c->act, c->F, w.w_down, c->resid, c->d, M, M_dev, c->d, c->F, kEpiAddNorm, nullptr, 0, &fd);
    ss_cur = c->ss_b;
  }
  *ss_out = ss_cur; *parts_out = parts_cur;
}

// One pass of the primary model's layers over the tokens described by es.tok_* (resid already holds the
// embeddings).  verify = false: prefill (KV goes to the context cache, tokens see a causal prefix of it);
// verify = true: drafted codes (KV goes to the draft region, tokens see the whole context + their own tuple).
void run_layers(nezha_ctx* c, long long M, const int* M_dev, bool verify, int n_rows, int max_tok_per_row) {
  const EngineState& e = c->es;
  const size_t esz = c->esz;
  for (int i = 0; i < c->nl; ++i) {
    const LayerW& w = c->layers[i];
    launch_rmsnorm(c->resid, c->d, nullptr, w.attn_norm, c->bf16, c->xn, nullptr, (int)M, M_dev, c->d, c->cfg.rms_eps,
                   c->st);
    gemm(c, c->xn, c->d, w.wqkv, c->d, c->qkv, c->qkv_dim, M, M_dev, c->qkv_dim, c->d, kEpiStoreAct);
    char* kc = (char*)c->k_ctx + (size_t)i * c->ctx_layer_elems * esz;
    char* vc = (char*)c->v_ctx + (size_t)i * c->ctx_layer_elems * esz;
    char* ke = (char*)c->k_ext + (size_t)i * c->ext_layer_elems * esz;
    char* ve = (char*)c->v_ext + (size_t)i * c->ext_layer_elems * esz;
    RopeAppendArgs r{};
    r.qkv = c->qkv; r.tok_pos = e.tok_pos; r.kv_dst = e.tok_kv_dst;
    r.kv_head_stride = verify ? c->hd : (long long)c->S * c->hd;
    r.k_cache = verify ? ke : kc; r.v_cache = verify ? ve : vc;
    r.cos_tab = c->rope_cos; r.sin_tab = c->rope_sin;
    r.M = (int)M; r.M_dev = M_dev; r.Hq = c->Hq; r.Hkv = c->Hkv; r.hd = c->hd;
    launch_rope_append(r, c->bf16, c->st);
    AttnArgs t{};
    t.q = c->qkv; t.q_stride = c->qkv_dim; t.out = c->attn; t.out_stride = (long long)c->Hq * c->hd;
    t.k_ctx = kc; t.v_ctx = vc; t.ctx_row_stride = (long long)c->Hkv * c->S * c->hd; t.ctx_head_stride = (long long)c->S * c->hd;
    t.k_ext = ke; t.v_ext = ve; t.ext_head_stride = c->hd;
    t.tok_row = e.tok_row; t.tok_ctx_len = e.tok_ctx_len; t.tok_ext = e.tok_ext; t.n_ext_max = verify ? c->L : 0;
    t.M = (int)M; t.M_dev = M_dev; t.Hq = c->Hq; t.Hkv = c->Hkv; t.hd = c->hd; t.scale = 1.f / sqrtf((float)c->hd);
    t.row_start = verify ? e.row_tok_start : e.pf_row_start; t.row_count = verify ? e.row_tok_count : e.pf_row_count;
    t.req_info = verify ? e.req_info : e.pf_req_info;
    t.n_rows = n_rows; t.max_tokens_per_row = max_tok_per_row;
    t.ctx_rows_total = (long long)c->Bmax * c->Hkv * c->S; t.status = e.status;
    t.ext_positions = (c->L > 1 ? c->L - 1 : 1) * c->Kmax; t.ext_pos_stride = (long long)c->Hkv * c->hd;
    t.ext_req_stride = t.ext_positions * t.ext_pos_stride; t.ext_rows_total = (long long)c->Bmax * t.ext_positions;
    if (c->bf16 && attention_tc_supported(t)) launch_attention_tc(t, c->st);
    else launch_attention_simt(t, c->bf16, c->st);
    gemm(c, c->attn, (long long)c->Hq * c->hd, w.wo, (long long)c->Hq * c->hd, c->resid, c->d, M, M_dev, c->d,
         c->Hq * c->hd, kEpiAddF32);
    launch_rmsnorm(c->resid, c->d, nullptr, w.mlp_norm, c->bf16, c->xn, nullptr, (int)M, M_dev, c->d, c->cfg.rms_eps,
                   c->st);
    gemm(c, c->xn, c->d, w.w_gu, c->d, c->gu, 2 * c->F, M, M_dev, 2 * c->F, c->d, kEpiStoreAct);
    launch_swiglu(c->gu, c->act, (int)M, M_dev, c->F, c->bf16, c->st);
    gemm(c, c->act, c->F, w.w_down, c->F, c->resid, c->d, M, M_dev, c->d, c->F, kEpiAddF32);
  }
}

// The verify pass proper: embeddings of the node tokens, all layers, final norm, LM head of levels 2..L.
void verify_pass(nezha_ctx* c, long long M_bound, int n_rows, int max_tok_per_row) {
  const EngineState& e = c->es;
  if (M_bound <= 0 || c->L < 2) return;
  const char* w = (const char*)c->lm_head + (size_t)e.li.off[1] * c->d * c->esz;
  if (c->fused) {
    launch_embed_norm(c->embed, e.tok_id, (int)M_bound, e.n_tokens, c->d, c->resid, c->layers[0].attn_norm, c->xn, c->ss_e,
                      c->st);
    const float* ss; int parts;
    run_layers_fused(c, M_bound, e.n_tokens, true, n_rows, max_tok_per_row, &ss, &parts);
    gemm_fused(c, c->xn, c->d, w, c->logits_v, c->Nv, M_bound, e.n_tokens, c->Nv, c->d, kEpiStoreF32, ss, parts, nullptr);
    return;
  }
  launch_embed(c->embed, c->bf16, e.tok_id, (int)M_bound, e.n_tokens, c->d, c->resid, c->st);
  run_layers(c, M_bound, e.n_tokens, true, n_rows, max_tok_per_row);
  launch_rmsnorm(c->resid, c->d, nullptr, c->final_norm, c->bf16, c->xn, nullptr, (int)M_bound, e.n_tokens, c->d,
                 c->cfg.rms_eps, c->st);
  gemm(c, c->xn, c->d, w, c->d, c->logits_v, c->Nv, M_bound, e.n_tokens, c->Nv, c->d, kEpiStoreF32);
}

// Draft-head logits of level l (1-based) for every (request, beam slot): Eq. 2.
void draft_logits_level(nezha_ctx* c, int batch, int l) {
  launch_draft_x(c->es, batch, l, c->xd, c->bf16, c->st);
  const int T = c->cfg.T[l - 1];
  gemm(c, c->xd, c->d, c->draft_logit[l - 1], c->d, c->logits_d, T, (long long)batch * c->Kmax, nullptr, T, c->d,
       kEpiStoreF32);
}

// Eq. 3 for every (request, beam slot): s_{l+1} = tanh(W_s s_l + W_e e_l + b); s_l + e_l in the additive ablation;
// nothing at all when the head does not use the context state.
void draft_transition_level(nezha_ctx* c, int batch, int l) {
  if (!c->es.draft_use_s) return;
  if (c->es.draft_additive) { launch_trans_add(c->es, batch, l, c->embed, c->bf16, c->st); return; }
  launch_trans_gather(c->es, batch, l, c->embed, c->a_se, c->bf16, c->st);
  float* out = c->es.state_lv + (size_t)(l + 1) * c->Bmax * c->Kmax * c->d;
  gemm(c, c->a_se, 2 * c->d, c->draft_wse, 2 * c->d, out, c->d, (long long)batch * c->Kmax, nullptr, c->d, 2 * c->d,
       kEpiBiasTanhF32, (const float*)c->draft_b_f32);
}

SelectArgs select_base(nezha_ctx* c, int batch, int K) {
  SelectArgs s{};
  s.in_stride = c->Kmax; s.out_stride = c->Kmax; s.K = K; s.tuple_len = c->L; s.batch = batch;
  s.li = c->es.li; s.hs = c->es.hs;
  s.pm = c->es.pm; s.final_mask_from_map = c->opt_mask;
  return s;
}

// The draft head with its two per-level products merged into one (fused path, default options).  Eq. 2 is linear:
// W_l (h_l + s_l) = W_l h_l + W_l s_l, and W_l h_l is a per-request constant (draft_hl, computed after the prefill);
// Eq. 3's W_e e_l is a table look-up (draft_u) and its W_s s_l does not depend on which code gets chosen.  So one
// product per level, s_l [W_l ; W_s]^T, yields the logits (before the selection) and the state term (used after it).
bool draft_fast(const nezha_ctx* c) {
  return c->fused && c->opt_transition == 0 && c->opt_inputs == 0;
}
// in_round: inside a decode round, where the device knows whether any request still drafts (a round queued for nothing, or
// one in which the adaptive policy has switched every request's drafting off, runs its products over zero rows)
void draft_level_product(nezha_ctx* c, int batch, int l, bool with_state, bool in_round = false) {
  const int T = c->cfg.T[l - 1];
  gemm(c, c->draft_sact, c->d, c->draft_wcat[l - 1], c->d, c->draft_g, c->Tmax + c->d, (long long)batch * c->Kmax,
       in_round ? c->es.draft_rows : nullptr, T + (with_state ? c->d : 0), c->d, kEpiStoreF32);
}
void draft_level_step(nezha_ctx* c, int batch, int l) {
  launch_draft_step(c->es, batch, l, c->draft_g, c->Tmax + c->d, c->cfg.T[l - 1], c->draft_u, (const float*)c->draft_b_f32, c->draft_sact,
                    c->st);
}

// Algorithm 3's inference loop (from the empty beam), or its continuation from the true beams (Algorithm 2's drafting step).
// `first_level` = smallest level any request can still need drafting at (levels below are teacher-forced only).
void draft_phase(nezha_ctx* c, int batch, int K, bool from_scratch, int first_level, bool filter) {
  const EngineState& e = c->es;
  const bool fast = draft_fast(c);
  launch_draft_init(e, batch, from_scratch ? 1 : 0, fast ? c->draft_sact : nullptr, c->st);
  for (int l = 1; l <= c->L; ++l) {
    if (fast && (l >= first_level || l < c->L)) draft_level_product(c, batch, l, l < c->L, true);
    if (l >= first_level) {
      if (!fast) draft_logits_level(c, batch, l);
      SelectArgs s = select_base(c, batch, K);
      const size_t lv_in = (size_t)(l - 1) * c->Bmax * c->Kmax, lv_out = (size_t)l * c->Bmax * c->Kmax;
      s.logits = c->logits_d; s.row_stride = c->cfg.T[l - 1]; s.col_off = 0; s.src_row = nullptr; s.src_mul = c->Kmax;
      if (fast) {
        s.logits = c->draft_g; s.row_stride = c->Tmax + c->d;
        s.logit_bias = c->draft_hl + (size_t)(l - 1) * c->Bmax * c->Tmax; s.bias_stride = c->Tmax;
      }
      s.in_codes = e.dw_codes + lv_in * c->L; s.in_score = e.dw_score + lv_in; s.in_count = e.dw_count + (size_t)(l - 1) * c->Bmax;
      s.n = l - 1; s.T = c->cfg.T[l - 1]; s.per_beam = K < s.T ? K : s.T; s.filter = (filter && l == c->L) ? 1 : 0;
      s.prefix_filter = (filter && c->opt_level_filter && l < c->L) ? 1 : 0;
      s.gate = e.d_m; s.gate_mode = 2; s.gate_value = l;
      s.out_codes = e.dw_codes + lv_out * c->L; s.out_score = e.dw_score + lv_out; s.out_parent = e.dw_parent + lv_out;
      s.out_token = nullptr; s.out_count = e.dw_count + (size_t)l * c->Bmax;
      // The selection and the state update it feeds in one launch -- where a launch is what costs (narrow models).  The
      // fused kernel is one CTA per request; at d = 4096 its 20 x 4096 state elements per request take 64 us on 32 SMs
      // against 14 us for the update spread over (request, beam) CTAs.
      if (fast && l < c->L && c->d <= 1024) {
        launch_select_step(s, e, l, c->draft_g, c->Tmax + c->d, c->cfg.T[l - 1], c->draft_u, (const float*)c->draft_b_f32,
                           c->draft_sact, c->st);
        continue;
      }
      launch_select(s, c->st);
    }
    if (l < c->L) { if (fast) draft_level_step(c, batch, l); else draft_transition_level(c, batch, l); }
  }
}

nezha_status pending_device_error(nezha_ctx* c) {
  int st = 0;
  NZ_CUDA(c, cudaMemcpyAsync(c->host_counters + 8, c->es.status, 4 * sizeof(int), cudaMemcpyDeviceToHost, c->st));
  NZ_CUDA(c, cudaStreamSynchronize(c->st));
  st = c->host_counters[8];
  if (st) NZ_CUDA(c, cudaMemsetAsync(c->es.status, 0, 4 * sizeof(int), c->st));
  if (st & kStHashFull) return fail(c, NEZHA_ERR_HASH_FULL, "hash set insertion exhausted its probe bound");
  if (st & kStBadCode) return fail(c, NEZHA_ERR_CATALOG, "a code outside [0, T_l) was given");
  if (st)      // a kernel that records where it gave up leaves three more words (0 if it does not)
    return fail(c, NEZHA_ERR_CUDA, "a bounded device-side wait expired (kernel gave up and returned); where: " +
                                       std::to_string(c->host_counters[9]) + " " + std::to_string(c->host_counters[10]) + " " +
                                       std::to_string(c->host_counters[11]));
  return NEZHA_OK;
}

// Runs one segment of a decode call (the part before the rounds, or one round).  The launch sequence of a segment
// is fixed by its key, so after one eager run it is captured into a CUDA graph and replayed from then on: one
// launch per round instead of dozens, and no launch gaps between its kernels.  Eager when the stream cannot be
// captured, while per-launch event timing is on, or if capture fails.
template <typename F>
nezha_status run_segment(nezha_ctx* c, const std::array<uintptr_t, 16>& key, F&& body) {
  if (!c->use_graphs || profile_is_on()) { body(); return NEZHA_OK; }
  nezha_ctx::Segment& sg = c->segments[key];
  if (sg.exec) {
    NZ_CUDA(c, cudaGraphLaunch(sg.exec, c->st));
    profile_add(sg.launches);
    return NEZHA_OK;
  }
  if (sg.seen++ == 0 || sg.seen > 3) { body(); return NEZHA_OK; }    // first run eager (one-time set-up calls); give up after failures
  long long before[kcCount], after[kcCount];
  profile_counts(before);
  cudaGraph_t graph = nullptr;
  if (cudaStreamBeginCapture(c->st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); body(); return NEZHA_OK; }
  body();
  const cudaError_t e = cudaStreamEndCapture(c->st, &graph);
  profile_counts(after);
  if (e != cudaSuccess || !graph || cudaGraphInstantiate(&sg.exec, graph, 0) != cudaSuccess) {
    cudaGetLastError();
    if (graph) cudaGraphDestroy(graph);
    sg.exec = nullptr;
    body();                                       // nothing ran during the failed capture
    return NEZHA_OK;
  }
  cudaGraphDestroy(graph);
  for (int i = 0; i < kcCount; ++i) sg.launches[i] = after[i] - before[i];
  NZ_CUDA(c, cudaGraphLaunch(sg.exec, c->st));   // the capture itself executed nothing
  return NEZHA_OK;
}

// drafts / n_draft: round 1's drafted tuples, or (is_tree) round 1's whole draft tree and its per-level counts
nezha_status decode_impl(nezha_ctx* c, int batch, int K, int mode, const int* drafts, const int* n_draft, bool is_tree,
                         int* out_codes, float* out_scores, int* out_count, nezha_decode_stats* stats,
                         const nezha_trace* trace) {
  if (!c) return NEZHA_ERR_ARG;
  if (c->state < 2) return fail(c, NEZHA_ERR_STATE, "nezha_decode before nezha_prefill");
  if (batch != c->batch || K < 1 || K > c->Kmax || !out_codes || !out_scores || !out_count || mode < 0 || mode > 2)
    return fail(c, NEZHA_ERR_ARG, "nezha_decode: bad batch / beam_width / mode / output pointer");
  const EngineState& e = c->es;
  const int L = c->L;
  // Every product of a decode call asks for the two-partial-sum order on narrow outputs (two MMA issuers): the
  // choice is per call path, never per launch, so that the speculative and the autoregressive mode, whose passes differ
  // in size, still compute the same bits.  The prefill keeps the plain order and the widest tiles.
  struct ChainScope {
    nezha_ctx* c;
    explicit ChainScope(nezha_ctx* c_) : c(c_) {
      c->chains_now = 2;
      c->skinny_now = c->skinny_decode ? 1 : 0;
    }
    ~ChainScope() { c->chains_now = 0; c->skinny_now = 0; }
  } chain_scope(c);
  nezha_trace tr{};
  if (trace) tr = *trace;
  nezha_decode_stats sd{};
  const int R = L - 1;
  auto key_of = [&](int segment) {
    std::array<uintptr_t, 16> k{};
    k[0] = (uintptr_t)segment; k[1] = (uintptr_t)batch; k[2] = (uintptr_t)K; k[3] = (uintptr_t)(mode | c->opt_transition << 8 | c->opt_inputs << 12 | c->opt_filter << 16 | c->opt_mask << 20 | (is_tree ? 1 : 0) << 24 | c->opt_level_filter << 25 | c->opt_adaptive << 26);
    k[4] = (uintptr_t)drafts; k[5] = (uintptr_t)n_draft; k[6] = (uintptr_t)out_codes; k[7] = (uintptr_t)out_scores;
    k[8] = (uintptr_t)out_count; k[9] = (uintptr_t)tr.drafts; k[10] = (uintptr_t)tr.n_draft; k[11] = (uintptr_t)tr.accepted_len;
    k[12] = (uintptr_t)tr.level_reached; k[13] = (uintptr_t)tr.beams ^ ((uintptr_t)tr.tree_codes << 1);
    k[14] = (uintptr_t)tr.beam_scores ^ ((uintptr_t)tr.tree_count << 1);
    k[15] = (uintptr_t)c->m_seen[segment];           // the expected token count shapes the tiling of the round's GEMMs
    return k;
  };
  nezha_status rs = run_segment(c, key_of(0), [&] {
    if (tr.drafts) launch_fill_i32(tr.drafts, (long long)R * batch * K * L, -1, c->st);
    if (tr.n_draft) launch_fill_i32(tr.n_draft, (long long)R * batch, -1, c->st);
    if (tr.accepted_len) launch_fill_i32(tr.accepted_len, (long long)R * batch * K, -1, c->st);
    if (tr.level_reached) launch_fill_i32(tr.level_reached, (long long)R * batch, -1, c->st);
    if (tr.tree_codes) launch_fill_i32(tr.tree_codes, (long long)R * L * batch * K * L, -1, c->st);
    if (tr.tree_count) launch_fill_i32(tr.tree_count, (long long)R * L * batch, -1, c->st);
    launch_fill_i32(out_codes, (long long)batch * K * L, -1, c->st);
    launch_fill_f32(out_scores, (long long)batch * K, -INFINITY, c->st);
    launch_fill_i32(out_count, batch, 0, c->st);
    launch_init_decode(e, batch, c->st);
    if (mode == NEZHA_MODE_DRAFT) {
      draft_phase(c, batch, K, true, 1, c->opt_filter != 0);
      const size_t lv = (size_t)L * c->Bmax * c->Kmax;
      launch_write_out(e.dw_codes + lv * L, e.dw_score + lv, e.dw_count + (size_t)L * c->Bmax, c->Kmax, L, batch, K,
                       out_codes, out_scores, out_count, c->st);
      return;
    }
    // B_1 from the prefill hidden state h_0 (Algorithm 1's LM head, top-K and pruning at l = 1)
    gemm(c, c->h_act, (long long)(L + 1) * c->d, c->lm_head, c->d, c->logits0, c->cfg.T[0], batch, nullptr, c->cfg.T[0], c->d,
         kEpiStoreF32);
    SelectArgs s = select_base(c, batch, K);
    const size_t lv_out = (size_t)1 * c->Bmax * c->Kmax;
    s.logits = c->logits0; s.row_stride = c->cfg.T[0]; s.col_off = 0; s.src_row = nullptr; s.src_mul = 1;
    s.in_codes = e.tb_codes; s.in_score = e.tb_score; s.in_count = e.tb_count; s.n = 0; s.T = c->cfg.T[0];
    s.per_beam = s.T; s.filter = (L == 1) ? 1 : 0; s.gate_mode = 0;
    s.prefix_filter = (c->opt_level_filter && L > 1) ? 1 : 0;
    s.out_codes = e.tb_codes + lv_out * L; s.out_score = e.tb_score + lv_out; s.out_parent = e.tb_parent + lv_out;
    s.out_count = e.tb_count + (size_t)1 * c->Bmax;
    launch_select(s, c->st);
    // settle level 1 (for L == 1 this also writes the result)
    launch_fill_i32(e.row_cur, batch, 0, c->st);
    launch_advance(e, batch, 0, K, out_codes, out_scores, out_count, c->st);
  });
  if (rs != NEZHA_OK) return rs;
  if (mode == NEZHA_MODE_DRAFT) {
    nezha_status ps = pending_device_error(c);
    if (stats) *stats = sd;
    return ps;
  }
  for (int round = 1; round <= R; ++round) {
    // drafts are mostly rejected or mostly accepted in a steady workload, so the round's token count repeats: tile for it
    c->m_expected = c->m_seen[round];
    rs = run_segment(c, key_of(round), [&] {
      if (mode == NEZHA_MODE_AR) launch_draft_set(e, batch, K, nullptr, nullptr, c->st);
      else if (round == 1 && drafts && is_tree) launch_draft_tree_set(e, batch, K, drafts, n_draft, c->st);
      else if (round == 1 && drafts) launch_draft_set(e, batch, K, drafts, n_draft, c->st);
      else draft_phase(c, batch, K, round == 1, round == 1 ? 1 : round + 1, c->opt_filter != 0);
      launch_build_nodes(e, batch, c->st);
      verify_pass(c, (long long)batch * K * (L - round), batch, K * (L - round));
      for (int n = round; n < L; ++n) {
        SelectArgs s = select_base(c, batch, K);
        const size_t lv_in = (size_t)n * c->Bmax * c->Kmax, lv_out = (size_t)(n + 1) * c->Bmax * c->Kmax;
        s.logits = c->logits_v; s.row_stride = c->Nv; s.col_off = e.li.off[n] - e.li.off[1];
        s.src_row = e.tb_src + lv_in; s.src_mul = 0;
        s.in_codes = e.tb_codes + lv_in * L; s.in_score = e.tb_score + lv_in; s.in_count = e.tb_count + (size_t)n * c->Bmax;
        s.n = n; s.T = c->cfg.T[n]; s.per_beam = s.T; s.filter = (n + 1 == L) ? 1 : 0;
        s.prefix_filter = (c->opt_level_filter && n + 1 < L) ? 1 : 0;
        s.gate = e.row_cur; s.gate_mode = 1; s.gate_value = n;
        s.out_codes = e.tb_codes + lv_out * L; s.out_score = e.tb_score + lv_out; s.out_parent = e.tb_parent + lv_out;
        s.out_count = e.tb_count + (size_t)(n + 1) * c->Bmax;
        launch_select_advance(s, e, n, K, out_codes, out_scores, out_count, c->st);
      }
      launch_round_end(e, batch, K, round, tr, mode == NEZHA_MODE_VERIFIED ? c->opt_adaptive : 0, c->st);
      cudaMemcpyAsync(c->host_counters + 16 + 8 * round, e.counters, 8 * sizeof(int), cudaMemcpyDeviceToHost, c->st);
    });
    c->m_expected = 0;
    if (rs != NEZHA_OK) return rs;
    // Whether another round is needed is known only from this round's counters.  A steady workload needs the same
    // number of rounds call after call, so the rounds the last call needed are queued without waiting in between;
    // a round queued for nothing finds every request finished and each of its kernels returns at once.
    if (round < R && round < c->rounds_seen[mode]) continue;
    NZ_CUDA(c, cudaStreamSynchronize(c->st));
    NZ_CUDA(c, cudaGetLastError());
    bool finished = false;
    for (int r = sd.rounds + 1; r <= round && !finished; ++r) {
      const int* hc = c->host_counters + 16 + 8 * r;
      c->m_seen[r] = (hc[1] + 127) / 128 * 128;
      sd.rounds = r;
      sd.primary_tokens += hc[1];
      sd.accepted_levels += hc[2];
      if (r == 1) sd.drafted = hc[3];
      finished = hc[0] == 0;
    }
    if (finished) break;
  }
  c->rounds_seen[mode] = sd.rounds;
  if (tr.beams || tr.beam_scores) launch_trace_beams(e, batch, K, tr, c->st);
  nezha_status ps = pending_device_error(c);
  if (stats) *stats = sd;
  return ps;
}

}  // namespace

// ====================================================================================================
// C ABI
// ====================================================================================================
extern "C" {

size_t nezha_arena_bytes(const nezha_config* cfg, size_t n_items, double load_factor) {
  std::string why;
  if (!check_config(cfg, &why) || !(load_factor > 0.0 && load_factor < 1.0)) return 0;
  nezha_ctx tmp{};
  tmp.cfg = *cfg; tmp.n_items = n_items; tmp.load_factor = load_factor; tmp.arena = nullptr;
  return carve(&tmp);
}

nezha_status nezha_create(const nezha_config* cfg, const nezha_weights* w, const int32_t* catalog_codes, size_t n_items,
                          double load_factor, void* arena, size_t arena_bytes, void* cuda_stream, nezha_ctx** out) {
  if (!out) return NEZHA_ERR_ARG;
  *out = nullptr;
  std::string why;
  if (!check_config(cfg, &why) || !w || !arena || !(load_factor > 0.0 && load_factor < 1.0) ||
      (n_items && !catalog_codes) || ((uintptr_t)arena & 255))
    return NEZHA_ERR_ARG;
  nezha_ctx* c = new nezha_ctx();
  c->cfg = *cfg; c->n_items = n_items; c->load_factor = load_factor; c->catalog = catalog_codes;
  c->st = (cudaStream_t)cuda_stream; c->arena = nullptr; c->state = 0; c->batch = 0;
  c->device = 0;
  if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return NEZHA_ERR_CUDA; }
  // the legacy default stream cannot be captured; NEZHA_NO_GRAPHS=1 keeps every launch eager
  c->use_graphs = cuda_stream != nullptr && !getenv("NEZHA_NO_GRAPHS");
  c->m_expected = 0;
  for (int i = 0; i <= kMaxLevels; ++i) c->m_seen[i] = 0;
  for (int i = 0; i < 3; ++i) c->rounds_seen[i] = 0;
  c->chains_now = 0;
  c->skinny_now = 0;
  c->opt_transition = 0; c->opt_inputs = 0; c->opt_filter = 1; c->opt_mask = 1; c->opt_level_filter = 0; c->opt_adaptive = 0;
  const size_t need = carve(c);
  if (need > arena_bytes) { delete c; return NEZHA_ERR_ARENA_TOO_SMALL; }
  c->arena = (char*)arena; c->arena_bytes = arena_bytes;
  carve(c);
  auto bail = [&](nezha_status s) { if (c->host_counters) cudaFreeHost(c->host_counters); delete c; return s; };
  c->host_counters = nullptr;
  if (cudaMallocHost((void**)&c->host_counters, (16 + 8 * (kMaxLevels + 1)) * sizeof(int)) != cudaSuccess) return bail(NEZHA_ERR_CUDA);
  if (select_configure(c->Kmax) != cudaSuccess) return bail(NEZHA_ERR_CUDA);
  if (c->fused) {                  // needs the tensor-core GEMM (TMA descriptors) for every projection
    GemmArgs probe{c->xn, c->d, c->layers[0].wqkv, c->d, c->qkv, c->qkv_dim, 128, nullptr, c->qkv_dim, c->d, kEpiStoreAct, nullptr,
                   c->es.status};
    if (!gemm_tc_supported(probe)) c->fused = false;
  }
  const size_t esz = c->esz;
  cudaStream_t st = c->st;
  auto cp = [&](void* dst, const void* src, size_t bytes) {
    return src && cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  };
  bool ok = cudaMemsetAsync(c->es.status, 0, 8 * sizeof(int), st) == cudaSuccess;
  {
    const long long pass_rows = c->Mv_max > (long long)c->Bmax * c->Kmax ? c->Mv_max : (long long)c->Bmax * c->Kmax;
    c->skinny_decode = c->fused && pass_rows <= kSkinnyRows && !getenv("NEZHA_NO_SKINNY");
  }
  // the caches start as zeros: tiles may overhang into never-written rows, whose (masked) values must be finite
  ok = ok && cudaMemsetAsync(c->k_ctx, 0, (size_t)c->nl * c->ctx_layer_elems * c->esz, st) == cudaSuccess &&
       cudaMemsetAsync(c->v_ctx, 0, (size_t)c->nl * c->ctx_layer_elems * c->esz, st) == cudaSuccess &&
       cudaMemsetAsync(c->k_ext, 0, (size_t)c->nl * c->ext_layer_elems * c->esz, st) == cudaSuccess &&
       cudaMemsetAsync(c->v_ext, 0, (size_t)c->nl * c->ext_layer_elems * c->esz, st) == cudaSuccess;
  ok = ok && cp(c->embed, w->embed, (size_t)c->vocab * c->d * esz) && cp(c->lm_head, w->lm_head, (size_t)c->vocab * c->d * esz) &&
       cp(c->final_norm, w->final_norm, (size_t)c->d * esz);
  const size_t q_b = (size_t)c->Hq * c->hd * c->d * esz, kv_b = (size_t)c->Hkv * c->hd * c->d * esz, f_b = (size_t)c->F * c->d * esz;
  for (int i = 0; ok && i < c->nl; ++i) {
    LayerW& lw = c->layers[i];
    ok = ok && w->attn_norm && w->wq && w->wk && w->wv && w->wo && w->mlp_norm && w->w_gate && w->w_up && w->w_down;
    ok = ok && cp(lw.attn_norm, w->attn_norm[i], (size_t)c->d * esz) && cp(lw.wqkv, w->wq[i], q_b) &&
         cp((char*)lw.wqkv + q_b, w->wk[i], kv_b) && cp((char*)lw.wqkv + q_b + kv_b, w->wv[i], kv_b) &&
         cp(lw.wo, w->wo[i], q_b) && cp(lw.mlp_norm, w->mlp_norm[i], (size_t)c->d * esz) && cp(lw.w_down, w->w_down[i], f_b);
    if (ok && c->fused) {          // rows of the q / k heads grouped into rotary pairs; gate and up rows interleaved
      launch_permute_rotary_rows(w->wq[i], lw.wqkv, c->Hq * c->hd, c->hd, c->d, st);
      launch_permute_rotary_rows(w->wk[i], (char*)lw.wqkv + q_b, c->Hkv * c->hd, c->hd, c->d, st);
      launch_interleave_gate_up(w->w_gate[i], w->w_up[i], lw.w_gu, c->F, c->d, st);
    } else {
      ok = ok && cp(lw.w_gu, w->w_gate[i], f_b) && cp((char*)lw.w_gu + f_b, w->w_up[i], f_b);
    }
  }
  for (int l = 0; ok && l < c->L; ++l)
    ok = ok && w->draft_logit && cp(c->draft_logit[l], w->draft_logit[l], (size_t)cfg->T[l] * c->d * esz);
  // [W_s | W_e] side by side along the input dimension: row o = [W_s[o, :], W_e[o, :]]
  ok = ok && w->draft_ws && w->draft_we && w->draft_b &&
       cudaMemcpy2DAsync(c->draft_wse, 2 * c->d * esz, w->draft_ws, c->d * esz, c->d * esz, c->d, cudaMemcpyDeviceToDevice, st) == cudaSuccess &&
       cudaMemcpy2DAsync((char*)c->draft_wse + c->d * esz, 2 * c->d * esz, w->draft_we, c->d * esz, c->d * esz, c->d,
                         cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (ok) {
    // bias as fp32 via a width-1 "norm-free" conversion: reuse the embed kernel on a 1-row table
    int zero = 0;
    ok = cudaMemcpyAsync(c->es.n_tokens, &zero, sizeof(int), cudaMemcpyHostToDevice, st) == cudaSuccess;
    launch_embed(w->draft_b, c->bf16, c->es.n_tokens, 1, nullptr, c->d, (float*)c->draft_b_f32, st);
  }
  if (ok && c->fused) {
    // [W_logit_l ; W_s] per level, and U = E W_e^T (fp32) for every code token: Eq. 3's input term of a chosen code
    for (int l = 0; ok && l < c->L; ++l)
      ok = cp(c->draft_wcat[l], w->draft_logit[l], (size_t)cfg->T[l] * c->d * esz) &&
           cp((char*)c->draft_wcat[l] + (size_t)cfg->T[l] * c->d * esz, w->draft_ws, (size_t)c->d * c->d * esz);
    gemm(c, c->embed, c->d, (char*)c->draft_wse + (size_t)c->d * esz, 2 * c->d, c->draft_u, c->d, c->es.li.vocab_codes, nullptr,
         c->d, c->d, kEpiStoreF32);
  }
  // rotary tables in double precision on the host
  if (ok) {
    const int half = c->hd / 2, np = c->S + c->L;
    std::vector<float> cs((size_t)np * half), sn((size_t)np * half);
    for (int p = 0; p < np; ++p)
      for (int i = 0; i < half; ++i) {
        const double ang = (double)p * pow((double)cfg->rope_theta, -2.0 * i / (double)c->hd);
        cs[(size_t)p * half + i] = (float)cos(ang); sn[(size_t)p * half + i] = (float)sin(ang);
      }
    ok = cudaMemcpyAsync(c->rope_cos, cs.data(), cs.size() * sizeof(float), cudaMemcpyHostToDevice, st) == cudaSuccess &&
         cudaMemcpyAsync(c->rope_sin, sn.data(), sn.size() * sizeof(float), cudaMemcpyHostToDevice, st) == cudaSuccess &&
         cudaStreamSynchronize(st) == cudaSuccess;
  }
  if (!ok || cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) return bail(NEZHA_ERR_CUDA);
  *out = c;
  return NEZHA_OK;
}

nezha_status nezha_build_hashset(nezha_ctx* c, uint64_t* n_unique) {
  if (!c) return NEZHA_ERR_ARG;
  NZ_CUDA(c, cudaMemsetAsync(c->n_unique_dev, 0, sizeof(unsigned long long), c->st));
  launch_hs_clear(c->es.hs, c->st);
  launch_hs_insert(c->es.li, c->es.hs, c->catalog, c->n_items, c->n_unique_dev, c->es.status, c->st);
  launch_pm_build(c->es.li, c->es.pm, c->catalog, c->n_items, c->es.status, c->st);
  unsigned long long nu = 0;
  NZ_CUDA(c, cudaMemcpyAsync(&nu, c->n_unique_dev, sizeof(nu), cudaMemcpyDeviceToHost, c->st));
  NZ_CUDA(c, cudaStreamSynchronize(c->st));
  NZ_CUDA(c, cudaGetLastError());
  if (n_unique) *n_unique = nu;
  nezha_status ps = pending_device_error(c);
  if (ps != NEZHA_OK) return ps;
  if (c->state < 1) c->state = 1;
  return NEZHA_OK;
}

nezha_status nezha_pack(nezha_ctx* c, const int32_t* codes, size_t n, uint64_t* keys) {
  if (!c || (n && (!codes || !keys))) return c ? fail(c, NEZHA_ERR_ARG, "nezha_pack: null pointer") : NEZHA_ERR_ARG;
  launch_hs_pack(c->es.li, codes, n, (unsigned long long*)keys, c->es.status, c->st);
  NZ_CUDA(c, cudaGetLastError());
  return NEZHA_OK;
}

nezha_status nezha_probe(nezha_ctx* c, const uint64_t* keys, size_t n, uint8_t* found) {
  if (!c || (n && (!keys || !found))) return c ? fail(c, NEZHA_ERR_ARG, "nezha_probe: null pointer") : NEZHA_ERR_ARG;
  if (c->state < 1) return fail(c, NEZHA_ERR_STATE, "nezha_probe before nezha_build_hashset");
  launch_hs_probe(c->es.hs, (const unsigned long long*)keys, n, found, c->st);
  NZ_CUDA(c, cudaGetLastError());
  return NEZHA_OK;
}

nezha_status nezha_prefill(nezha_ctx* c, const int32_t* hist_codes, const int32_t* n_hist, int32_t batch, int32_t max_n) {
  if (!c) return NEZHA_ERR_ARG;
  if (c->state < 1) return fail(c, NEZHA_ERR_STATE, "nezha_prefill before nezha_build_hashset");
  if (batch < 1 || batch > c->Bmax || max_n < 0 || max_n > c->cfg.max_hist_items || !n_hist || (max_n && !hist_codes))
    return fail(c, NEZHA_ERR_ARG, "nezha_prefill: batch / max_n out of the configured range or null pointer");
  const EngineState& e = c->es;
  const int S_call = 1 + max_n * c->L + c->L;
  for (int b0 = 0; b0 < batch; b0 += c->chunk_rows) {
    const int rows = (batch - b0 < c->chunk_rows) ? batch - b0 : c->chunk_rows;
    const long long M = (long long)rows * S_call;
    // a prompt chunk of at most kSkinnyRows tokens in an engine of the weight-streaming class (one short history): the same
    // kernel as its decode passes.  The prefill is shared by all decode modes, so their equality is not touched.
    c->skinny_now = c->skinny_decode && M <= kSkinnyRows ? 1 : 0;
    launch_prefill_tokens(e, hist_codes, n_hist, b0, rows, max_n, S_call, c->S, c->h_rows, c->st);
    if (c->fused) {
      launch_embed_norm(c->embed, e.tok_id, (int)M, nullptr, c->d, c->resid, c->layers[0].attn_norm, c->xn, c->ss_e, c->st);
      const float* ss; int parts;
      run_layers_fused(c, M, nullptr, false, rows, S_call, &ss, &parts);
    } else {
      launch_embed(c->embed, c->bf16, e.tok_id, (int)M, nullptr, c->d, c->resid, c->st);
      run_layers(c, M, nullptr, false, rows, S_call);
    }
    const size_t ho = (size_t)b0 * (c->L + 1) * c->d;
    launch_rmsnorm(c->resid, c->d, c->h_rows, c->final_norm, c->bf16, (char*)c->h_act + ho * c->esz, c->h_f32 + ho,
                   rows * (c->L + 1), nullptr, c->d, c->cfg.rms_eps, c->st);
    if (c->fused)                  // the request-constant half of Eq. 2: W_logit_l h_l for every level
      for (int l = 1; l <= c->L; ++l)
        gemm(c, (char*)c->h_act + (ho + (size_t)l * c->d) * c->esz, (long long)(c->L + 1) * c->d, c->draft_logit[l - 1], c->d,
             c->draft_hl + ((size_t)(l - 1) * c->Bmax + b0) * c->Tmax, c->Tmax, rows, nullptr, c->cfg.T[l - 1], c->d, kEpiStoreF32);
  }
  c->skinny_now = 0;
  NZ_CUDA(c, cudaGetLastError());
  c->batch = batch;
  c->state = 2;
  return NEZHA_OK;
}

nezha_status nezha_decode(nezha_ctx* c, int32_t batch, int32_t beam_width, int32_t mode, int32_t* out_codes,
                          float* out_scores, int32_t* out_count, nezha_decode_stats* stats, const nezha_trace* trace) {
  return decode_impl(c, batch, beam_width, mode, nullptr, nullptr, false, out_codes, out_scores, out_count, stats, trace);
}

nezha_status nezha_decode_with_drafts(nezha_ctx* c, int32_t batch, int32_t beam_width, const int32_t* drafts,
                                      const int32_t* n_draft, int32_t* out_codes, float* out_scores, int32_t* out_count,
                                      nezha_decode_stats* stats, const nezha_trace* trace) {
  if (!c) return NEZHA_ERR_ARG;
  if (!drafts || !n_draft) return fail(c, NEZHA_ERR_ARG, "nezha_decode_with_drafts: null drafts");
  return decode_impl(c, batch, beam_width, NEZHA_MODE_VERIFIED, drafts, n_draft, false, out_codes, out_scores, out_count,
                     stats, trace);
}

nezha_status nezha_decode_with_draft_tree(nezha_ctx* c, int32_t batch, int32_t beam_width, const int32_t* tree_codes,
                                          const int32_t* tree_count, int32_t* out_codes, float* out_scores,
                                          int32_t* out_count, nezha_decode_stats* stats, const nezha_trace* trace) {
  if (!c) return NEZHA_ERR_ARG;
  if (!tree_codes || !tree_count) return fail(c, NEZHA_ERR_ARG, "nezha_decode_with_draft_tree: null tree");
  return decode_impl(c, batch, beam_width, NEZHA_MODE_VERIFIED, tree_codes, tree_count, true, out_codes, out_scores,
                     out_count, stats, trace);
}

nezha_status nezha_set_option(nezha_ctx* c, int32_t option, int32_t value) {
  if (!c) return NEZHA_ERR_ARG;
  switch (option) {
    case NEZHA_OPT_DRAFT_TRANSITION:
      if (value != 0 && value != 1) return fail(c, NEZHA_ERR_ARG, "nezha_set_option: transition must be 0 or 1");
      c->opt_transition = value; c->es.draft_additive = value; break;
    case NEZHA_OPT_DRAFT_INPUTS:
      if (value < 0 || value > 2) return fail(c, NEZHA_ERR_ARG, "nezha_set_option: inputs must be 0, 1 or 2");
      c->opt_inputs = value; c->es.draft_use_h = value != 2; c->es.draft_use_s = value != 1; break;
    case NEZHA_OPT_DRAFT_FILTER:
      if (value != 0 && value != 1) return fail(c, NEZHA_ERR_ARG, "nezha_set_option: filter must be 0 or 1");
      c->opt_filter = value; break;
    case NEZHA_OPT_FINAL_MASK:
      if (value != 0 && value != 1) return fail(c, NEZHA_ERR_ARG, "nezha_set_option: final mask must be 0 or 1");
      c->opt_mask = value; break;
    case NEZHA_OPT_ADAPTIVE_DRAFT:
      if (value != 0 && value != 1) return fail(c, NEZHA_ERR_ARG, "nezha_set_option: adaptive drafting must be 0 or 1");
      c->opt_adaptive = value; break;
    case NEZHA_OPT_LEVEL_FILTER:
      if (value != 0 && value != 1) return fail(c, NEZHA_ERR_ARG, "nezha_set_option: level filter must be 0 or 1");
      c->opt_level_filter = value; break;
    default: return fail(c, NEZHA_ERR_ARG, "nezha_set_option: unknown option");
  }
  return NEZHA_OK;
}

nezha_status nezha_get_hidden(nezha_ctx* c, float* out) {
  if (!c || !out) return NEZHA_ERR_ARG;
  if (c->state < 2) return fail(c, NEZHA_ERR_STATE, "nezha_get_hidden before nezha_prefill");
  NZ_CUDA(c, cudaMemcpyAsync(out, c->h_f32, (size_t)c->batch * (c->L + 1) * c->d * sizeof(float), cudaMemcpyDeviceToDevice,
                             c->st));
  return NEZHA_OK;
}

nezha_status nezha_primary_logits(nezha_ctx* c, int32_t batch, int32_t n_beams, int32_t level, const int32_t* prefixes,
                                  float* logits) {
  if (!c) return NEZHA_ERR_ARG;
  if (c->state < 2) return fail(c, NEZHA_ERR_STATE, "nezha_primary_logits before nezha_prefill");
  if (batch != c->batch || n_beams < 1 || n_beams > c->Kmax || level < 0 || level >= c->L || !logits || (level && !prefixes))
    return fail(c, NEZHA_ERR_ARG, "nezha_primary_logits: bad argument");
  const EngineState& e = c->es;
  if (level == 0) {
    gemm(c, c->h_act, (long long)(c->L + 1) * c->d, c->lm_head, c->d, c->logits0, c->cfg.T[0], batch, nullptr, c->cfg.T[0],
         c->d, kEpiStoreF32);
    launch_copy_logits(c->logits0, c->cfg.T[0], 0, nullptr, 1, 0, batch, n_beams, 0, c->cfg.T[0], logits, c->st);
  } else {
    launch_nodes_from_prefixes(e, batch, n_beams, level, prefixes, c->st);
    verify_pass(c, (long long)batch * n_beams * level, batch, n_beams * level);
    launch_copy_logits(c->logits_v, c->Nv, e.li.off[level] - e.li.off[1], e.node_index + (size_t)level * c->Kmax, 0, 0, batch,
                       n_beams, c->L * c->Kmax, c->cfg.T[level], logits, c->st);
  }
  NZ_CUDA(c, cudaGetLastError());
  return NEZHA_OK;
}

nezha_status nezha_draft_logits(nezha_ctx* c, int32_t batch, int32_t n_beams, int32_t level, const int32_t* prefixes,
                                float* logits) {
  if (!c) return NEZHA_ERR_ARG;
  if (c->state < 2) return fail(c, NEZHA_ERR_STATE, "nezha_draft_logits before nezha_prefill");
  if (batch != c->batch || n_beams < 1 || n_beams > c->Kmax || level < 0 || level >= c->L || !logits || (level && !prefixes))
    return fail(c, NEZHA_ERR_ARG, "nezha_draft_logits: bad argument");
  const EngineState& e = c->es;
  // start set = the given prefixes at level `level`; teacher-force the transitions, then Eq. 2 for the next level
  launch_init_decode(e, batch, c->st);
  launch_fill_i32(e.d_m, batch, level, c->st);
  launch_fill_i32(e.dw_count + (size_t)level * c->Bmax, batch, n_beams, c->st);
  if (level > 0) {
    const size_t lv = (size_t)level * c->Bmax * c->Kmax;
    launch_fill_i32(e.dw_codes + lv * c->L, (long long)c->Bmax * c->Kmax * c->L, 0, c->st);
    for (int b = 0; b < batch; ++b)
      NZ_CUDA(c, cudaMemcpy2DAsync(e.dw_codes + (lv + (size_t)b * c->Kmax) * c->L, (size_t)c->L * sizeof(int),
                                   prefixes + (size_t)b * n_beams * level, (size_t)level * sizeof(int),
                                   (size_t)level * sizeof(int), (size_t)n_beams, cudaMemcpyDeviceToDevice, c->st));
  }
  if (draft_fast(c)) {
    launch_draft_state_init(e, batch, c->draft_sact, c->st);
    for (int l = 1; l <= level; ++l) { draft_level_product(c, batch, l, true); draft_level_step(c, batch, l); }
    draft_level_product(c, batch, level + 1, false);
    launch_copy_logits_bias(c->draft_g, c->Tmax + c->d, c->Kmax, batch, n_beams, c->cfg.T[level],
                            c->draft_hl + (size_t)level * c->Bmax * c->Tmax, c->Tmax, logits, c->st);
  } else {
    for (int l = 1; l <= level; ++l) draft_transition_level(c, batch, l);
    draft_logits_level(c, batch, level + 1);
    launch_copy_logits(c->logits_d, c->cfg.T[level], 0, nullptr, c->Kmax, 1, batch, n_beams, 0, c->cfg.T[level], logits, c->st);
  }
  NZ_CUDA(c, cudaGetLastError());
  return NEZHA_OK;
}

nezha_status nezha_select(nezha_ctx* c, int32_t batch, int32_t n_beams, int32_t beam_width, int32_t level, int32_t per_beam,
                          int32_t filter, const float* logits, const float* beam_scores, const int32_t* beam_codes,
                          const int32_t* n_live, int32_t* out_parent, int32_t* out_code, float* out_score,
                          int32_t* out_count) {
  if (!c) return NEZHA_ERR_ARG;
  if (batch < 1 || n_beams < 1 || n_beams > 128 || beam_width < 1 || beam_width > c->Kmax || n_beams > c->Kmax ||
      level < 0 || level >= c->L || per_beam < 1 || !logits || !beam_scores || (level && !beam_codes) || !n_live ||
      !out_score || !out_count)
    return fail(c, NEZHA_ERR_ARG, "nezha_select: bad argument");
  if (filter && c->state < 1) return fail(c, NEZHA_ERR_STATE, "nezha_select with filter before nezha_build_hashset");
  SelectArgs s{};
  s.logits = logits; s.row_stride = c->cfg.T[level]; s.col_off = 0; s.src_row = nullptr; s.src_mul = n_beams;
  s.in_codes = beam_codes; s.in_score = beam_scores; s.in_count = n_live; s.in_stride = n_beams;
  s.n = level; s.T = c->cfg.T[level]; s.K = beam_width; s.per_beam = per_beam;
  s.filter = (filter && level + 1 == c->L) ? 1 : 0; s.prefix_filter = (filter && level + 1 < c->L) ? 1 : 0;
  s.pm = c->es.pm; s.final_mask_from_map = 0;
  s.gate_mode = 0;
  s.out_codes = nullptr; s.out_token = out_code; s.out_score = out_score; s.out_parent = out_parent; s.out_count = out_count;
  s.out_stride = beam_width; s.tuple_len = level; s.batch = batch; s.li = c->es.li; s.hs = c->es.hs;
  launch_select(s, c->st);
  NZ_CUDA(c, cudaGetLastError());
  return NEZHA_OK;
}

nezha_status nezha_gemm(nezha_ctx* c, const void* A, const void* W, void* C, int32_t M, int32_t N, int32_t K,
                        int32_t epilogue, const float* bias, int32_t path) {
  if (!c) return NEZHA_ERR_ARG;
  if (!A || !W || !C || M < 1 || N < 1 || K < 1 || epilogue < 0 || epilogue > 3 || (epilogue == 3 && !bias) || path < 0 ||
      path > 4)
    return fail(c, NEZHA_ERR_ARG, "nezha_gemm: bad argument");
  GemmArgs a{A, K, W, K, C, N, M, nullptr, N, K, epilogue, bias, c->es.status};
  a.chains = path == 3 ? 2 : 0;
  if (path == 4) {
    if (M > kSkinnyRows || !c->bf16)
      return fail(c, NEZHA_ERR_UNSUPPORTED, "nezha_gemm: the weight-streaming kernel takes bf16 products of at most 128 rows");
    a.skinny = 1;
  }
  const bool tc_ok = c->bf16 && gemm_tc_supported(a);
  if (path >= 2 && !tc_ok) return fail(c, NEZHA_ERR_UNSUPPORTED, "nezha_gemm: shape not covered by the tcgen05 kernel");
  if (path != 1 && tc_ok) launch_gemm_tc(a, c->st);
  else launch_gemm_simt(a, c->bf16, c->st);
  NZ_CUDA(c, cudaGetLastError());
  return NEZHA_OK;
}

uint64_t nezha_launch_count(void) { return profile_total_launches(); }

nezha_status nezha_profile_enable(nezha_ctx* c, int32_t on) {
  if (!c) return NEZHA_ERR_ARG;
  NZ_CUDA(c, cudaStreamSynchronize(c->st));
  profile_enable(on != 0);
  return NEZHA_OK;
}

nezha_status nezha_profile_read(nezha_ctx* c, nezha_profile* out) {
  if (!c || !out) return NEZHA_ERR_ARG;
  NZ_CUDA(c, cudaStreamSynchronize(c->st));
  profile_read(out);
  return NEZHA_OK;
}

nezha_status nezha_sync(nezha_ctx* c) {
  if (!c) return NEZHA_ERR_ARG;
  NZ_CUDA(c, cudaStreamSynchronize(c->st));
  NZ_CUDA(c, cudaGetLastError());
  return pending_device_error(c);
}

// ---- membership test for callers that cannot allocate device memory ------------------------------------
// The packed keys of the tuples are an intermediate result: nezha_pack writes them to a caller-allocated buffer and
// nezha_probe reads them back.  Here they live in a fixed array that is part of the loaded library image instead,
// so nothing is allocated by anyone.  The array is shared by every call on the device and keeps whatever the last
// call wrote; each call overwrites the first n entries before it reads them, so nothing needs clearing.
static __device__ __align__(256) unsigned long long g_noalloc_keys[NEZHA_NOALLOC_MAX_TUPLES];

namespace {
constexpr int kMaxDevices = 64;
unsigned long long* g_noalloc_keys_addr[kMaxDevices] = {nullptr};   // device address of the array, per device

// `g_noalloc_keys` in host code is only a handle of the symbol; the address a kernel can use has to be asked for,
// once per device, with that device current.
cudaError_t noalloc_keys_address(unsigned long long** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_noalloc_keys_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_keys);
    if (e != cudaSuccess) return e;
    g_noalloc_keys_addr[dev] = static_cast<unsigned long long*>(p);
  }
  *out = g_noalloc_keys_addr[dev];
  return cudaSuccess;
}
}  // namespace

nezha_status nezha_contains_noalloc(nezha_ctx* c, const int32_t* codes, size_t n, uint8_t* found) {
  if (!c) return NEZHA_ERR_ARG;
  if (n && (!codes || !found)) return fail(c, NEZHA_ERR_ARG, "nezha_contains_noalloc: null pointer");
  if (n > (size_t)NEZHA_NOALLOC_MAX_TUPLES)
    return fail(c, NEZHA_ERR_ARG, "nezha_contains_noalloc: n exceeds NEZHA_NOALLOC_MAX_TUPLES (the size of the built-in "
                                  "key buffer); split the request or use nezha_pack + nezha_probe");
  if (c->state < 1) return fail(c, NEZHA_ERR_STATE, "nezha_contains_noalloc before nezha_build_hashset");
  if (!n) return NEZHA_OK;
  int dev = -1;
  NZ_CUDA(c, cudaGetDevice(&dev));
  if (dev != c->device)          // the built-in buffer is per device: the address looked up must be the context's GPU's
    return fail(c, NEZHA_ERR_ARG, "nezha_contains_noalloc: the context's GPU must be the current device");
  unsigned long long* keys = nullptr;
  NZ_CUDA(c, noalloc_keys_address(&keys));
  launch_hs_pack(c->es.li, codes, n, keys, c->es.status, c->st);
  launch_hs_probe(c->es.hs, keys, n, found, c->st);
  NZ_CUDA(c, cudaGetLastError());
  return NEZHA_OK;
}

const char* nezha_last_error(const nezha_ctx* c) { return c ? c->err.c_str() : "null context"; }

void nezha_destroy(nezha_ctx* c) {
  if (!c) return;
  for (auto& kv : c->segments)
    if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
  if (c->host_counters) cudaFreeHost(c->host_counters);
  delete c;
}

}  // extern "C"
