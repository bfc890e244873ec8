// Device-resident state of one decode call and the launchers of the beam-search kernels that work on it.
//
// Indexing convention: a "level n" beam has n codes (n = 0 is the empty beam).  Arrays named tb_* hold the true
// beam sets B_n of the primary model for n = 0..L; dw_* hold the draft head's working beam sets.
#pragma once

#include "common.cuh"

namespace nz {

struct EngineState {
  int Bmax, Kmax, L, d, Hkv, hd;
  LevelInfo li;
  HashSetView hs;
  PrefixMapView pm;
  int* status;
  // draft-head variants (the ablations of Section 4.3); defaults 1, 1, 0 = Eq. 2 and Eq. 3 as printed
  int draft_use_h, draft_use_s, draft_additive;

  // true beams, [L+1][Bmax][Kmax]([L])
  int* tb_codes; float* tb_score; int* tb_parent; int* tb_count;   // tb_count: [L+1][Bmax]
  int* tb_anc;      // [L+1][Bmax][Kmax][L]: slot (in the draft-KV slab of level i+1) of the ancestor with i+1 codes
  int* tb_self;     // [L+1][Bmax][Kmax]: slot of the beam's own KV in the slab of its level
  int* tb_src;      // [L+1][Bmax][Kmax]: token index whose hidden state predicts the beam's next code

  int* row_m;       // [Bmax] levels settled (L = row finished)
  int* row_cur;     // [Bmax] level whose beams have logits in the current pass, -1 = row stopped this round
  int* row_P;       // [Bmax] context length of the row (BOS + history tokens)
  int* row_m_start; // [Bmax] levels the row had settled when the current round began
  int* draft_rows;  // [1] rows of the draft head's products in the coming round: batch * Kmax, or 0 when no request drafts
  int* row_spec;    // [Bmax] 1: the draft head drafts for the row in the next round (always 1 unless the adaptive policy is on)

  // The round's draft tree, [L+1][Bmax][Kmax]([L]): level l holds the drafted nodes with l codes (the draft head's beam
  // set of that level, or the distinct l-prefixes of caller-supplied tuples); dw_parent = slot of the node's parent in
  // level l - 1.  The drafted tuples of the round are level L.
  int* dw_codes; float* dw_score; int* dw_parent; int* dw_count;
  int* d_m;         // [Bmax] level the row's drafting started from this round (L = the draft head takes no part)
  int* d_beam;      // [L+1][Bmax][Kmax] for a node in this round's pass: rank of the true beam of B_m it descends from
                    //                   (-1: the node is dead -- its first m codes are no beam, or it has no parent)
  float* state_lv;  // [L+1][Bmax][Kmax][d] draft-head context states s_l (l = 2..L used; s_1 = h_0)

  // verify-pass token list
  int* node_index;  // [Bmax][L][Kmax] token index of node (level n = 1..L-1 stored at n, slot), -1 if absent
  int* tok_row; int* tok_pos; int* tok_id; int* tok_ctx_len; long long* tok_kv_dst; long long* tok_ext;  // tok_ext [Mv][L]
  int* row_tok_count;   // [Bmax]
  int* row_tok_start;   // [Bmax] first token of the request in the list
  int* pf_row_start; int* pf_row_count;   // [Bmax] the same for a prefill chunk (indexed by row within the chunk)
  int4* req_info; int4* pf_req_info;      // [Bmax] {first token, token count, cache row, context length or -1 = causal}:
                                          //        all the attention kernel needs to know about a request, in one load
  int* n_tokens;        // [1]
  int* counters;        // [8]: 0 unfinished rows, 1 primary tokens (round), 2 accepted levels (round), 3 drafted (round)

  const float* h_f32;   // [Bmax][L+1][d]
};

inline __host__ __device__ long long lvl_bk(const EngineState& e, int n, int b, int k) {
  return ((long long)n * e.Bmax + b) * e.Kmax + k;
}

struct SelectArgs {
  const float* logits; long long row_stride; int col_off;
  const int* src_row; int src_mul;      // logits row of beam r of request b: src_row ? src_row[b*in_stride+r] : b*src_mul+r
  const int* in_codes; const float* in_score; const int* in_count; int in_stride;
  int n;                                // codes the input beams have; the level's codebook is T[n]
  int T, K, per_beam, filter;
  const int* gate; int gate_mode, gate_value;   // 0: none, 1: run iff gate[b] == value, 2: run iff gate[b] < value
  const float* logit_bias; long long bias_stride;   // optional: logits of request b get logit_bias[b * bias_stride + t] added
  int* out_codes; int* out_token; float* out_score; int* out_parent; int* out_count; int out_stride;
  int tuple_len;                        // row length of in_codes / out_codes (L)
  int batch;
  LevelInfo li; HashSetView hs;
  PrefixMapView pm;
  int final_mask_from_map;              // 1: the last-level mask of a beam (all T_L extensions) reads the prefix map; 0: hash probes
  int prefix_filter;                    // 1: this is an earlier level and candidates that begin no valid ID are dropped
};
void launch_select(const SelectArgs& a, cudaStream_t st);
// launch_select (gated on row_cur == n) followed, in the same launch, by launch_advance of level n
void launch_select_advance(const SelectArgs& a, const EngineState& e, int n, int K, int* out_codes, float* out_score,
                           int* out_count, cudaStream_t st);
// launch_select followed, in the same launch, by launch_draft_step of level l (same arguments as there)
void launch_select_step(const SelectArgs& a, const EngineState& e, int l, const float* G, long long g_stride, int t_cols,
                        const float* U, const float* bias, void* s_act, cudaStream_t st);
size_t select_smem_bytes(int in_stride, int K);
cudaError_t select_configure(int max_beam);

void launch_init_decode(const EngineState& e, int batch, cudaStream_t st);
void launch_draft_init(const EngineState& e, int batch, int from_scratch, void* s_act, cudaStream_t st);   // s_act may be null
void launch_draft_set(const EngineState& e, int batch, int K, const int* drafts, const int* n_draft, cudaStream_t st);
// the whole tree given by the caller: tree_codes [L][batch][K][L], tree_count [L][batch]
void launch_draft_tree_set(const EngineState& e, int batch, int K, const int* tree_codes, const int* tree_count, cudaStream_t st);
void launch_draft_x(const EngineState& e, int batch, int l, void* x, bool bf16, cudaStream_t st);
void launch_trans_gather(const EngineState& e, int batch, int l, const void* embed, void* A, bool bf16,
                         cudaStream_t st);
void launch_trans_add(const EngineState& e, int batch, int l, const void* embed, bool bf16, cudaStream_t st);
// The draft head with its two per-level products merged (see DraftFast in api.cu)
void launch_draft_state_init(const EngineState& e, int batch, void* s_act, cudaStream_t st);
void launch_draft_step(const EngineState& e, int batch, int l, const float* G, long long g_stride, int t_cols, const float* U,
                       const float* bias, void* s_act, cudaStream_t st);
void launch_copy_logits_bias(const float* src, long long row_stride, int row_mul, int batch, int n_beams, int T,
                             const float* bias, long long bias_stride, float* dst, cudaStream_t st);
void launch_build_nodes(const EngineState& e, int batch, cudaStream_t st);
void launch_nodes_from_prefixes(const EngineState& e, int batch, int n_beams, int level, const int* prefixes,
                                cudaStream_t st);
void launch_advance(const EngineState& e, int batch, int n, int K, int* out_codes, float* out_score, int* out_count,
                    cudaStream_t st);
void launch_round_end(const EngineState& e, int batch, int K, int round, const nezha_trace& tr, int adaptive, cudaStream_t st);
void launch_write_out(const int* codes, const float* score, const int* count, int stride, int L, int batch, int K,
                      int* out_codes, float* out_score, int* out_count, cudaStream_t st);
void launch_copy_logits(const float* src, long long row_stride, int col_off, const int* row_index, int row_mul,
                        int beam_mul, int batch, int n_beams, int idx_stride, int T, float* dst, cudaStream_t st);
void launch_fill_i32(int* p, long long n, int v, cudaStream_t st);
void launch_fill_f32(float* p, long long n, float v, cudaStream_t st);
void launch_trace_beams(const EngineState& e, int batch, int K, const nezha_trace& tr, cudaStream_t st);

}  // namespace nz
