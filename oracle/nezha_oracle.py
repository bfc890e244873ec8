"""CPU oracle for the speculative semantic-ID decode step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy statement of what the decode path computes, written from the paper's
equations and algorithms.  It shares no code with the CUDA library and must never be imported by the
product path: only tests, the smoke check and the benchmark's CPU-baseline leg use it.

What follows the paper, and where:
  pack_keys / unpack_keys        Eq. 4  (mixed-radix index of a semantic ID, level 1 least significant)
  ValidSet                       Eq. 5  (the set V of valid IDs; membership by binary search in a sorted array)
  draft_logits / draft_transition  Eq. 1-3 (s_1 = h_0, p_l = logit_head_l(h_l, s_l), s_{l+1} = Transition(s_l, e_l))
  nezha_draft                    Algorithm 3, inference part (draft-head beam search, hash filter at l = L)
  ar_beam_search                 Algorithm 1 with the validity filter of Eq. 5 at the last level
  speculative_decode             Algorithm 2 instantiated with NEZHA's draft head and hash set
  PrimaryModel                   the decoder-only LLM M_p of Algorithms 1-3 (architecture: see readings below)

Readings where the paper is silent (the same readings bind the CUDA path):
  * prompt: [BOS, history codes..., SP_1..SP_L]; empty query; token ids: level-l code c -> off_l + c with
    off_l = sum_{j<l} T_j, SP_l -> sum(T) + l - 1, BOS -> sum(T) + L.
  * M_p: Llama-style (RMSNorm, rotary embedding on half-split pairs, grouped-query causal attention,
    SwiGLU MLP, no biases, untied LM head).  h_0..h_L are the final-norm outputs at the last context
    position and the L placeholder positions.
  * logit_head_l(h, s) = W_l (h + s);  Transition(s, e) = tanh(W_s s + W_e e + b), shared over levels,
    e = the input-embedding row of the chosen token.
  * probabilities are a softmax over the level's own codebook (T_l logits); cumulative probability is kept
    as a sum of log-probabilities, stored in fp32; order: higher score first, ties to the smaller
    (parent rank, token).
  * plain autoregressive decoding sees no placeholders: the level-j code sits at position P + j - 1.
  * Algorithm 2's "verify in parallel" takes the draft head's whole level-wise beam tree (the beam sets of every level
    of Algorithm 3, one node per distinct prefix), not only the prefixes of its K final tuples.

Pinned by tests/test_oracle_*.py:  Eq. 4 by the paper's worked example and bijectivity; ValidSet by python
sets; PrimaryModel by an independent library implementation of the same architecture, closed forms and
cached-vs-recomputed equality; nezha_draft and ar_beam_search by brute-force enumeration, independently
recomputed joint log-probabilities and closed forms under zero heads; speculative_decode by equality with
ar_beam_search for any drafts, and its walk (rounds, rejection levels, accepted lengths, tokens in the pass) by
hand-worked cases on heads of all zeros, where the tie rule fixes every beam set in closed form.  How Algorithm 2's
parallel verification is combined with NEZHA's head (which nodes the pass holds) is this file's reading: the paper
never runs the two together.  DraftHead.logits / .transition follow readings of Section 4.1's one-line description
(sum then one matmul; one shared Elman cell): pinned by hand-computed numbers and the ablation identities of
Section 4.3, with no external implementation to compare against.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

NEG_INF = np.float32(-np.inf)


# ----------------------------------------------------------------------------------------------------
# Eq. 4 / Eq. 5
# ----------------------------------------------------------------------------------------------------

def pack_keys(codes: np.ndarray, T: Sequence[int]) -> np.ndarray:
    """Eq. 4: V = sum_l t_l * prod_{j<l} T_j  (codes [..., L] -> uint64 [...])."""
    codes = np.asarray(codes)
    key = np.zeros(codes.shape[:-1], dtype=np.uint64)
    mult = 1
    for l in range(len(T)):
        key = key + codes[..., l].astype(np.uint64) * np.uint64(mult)
        mult *= int(T[l])
    return key


def unpack_keys(keys: np.ndarray, T: Sequence[int]) -> np.ndarray:
    """Inverse of Eq. 4 (it is a bijection onto [0, prod T))."""
    keys = np.asarray(keys, dtype=np.uint64)
    out = np.zeros(keys.shape + (len(T),), dtype=np.int64)
    rest = keys.copy()
    for l in range(len(T)):
        out[..., l] = (rest % np.uint64(T[l])).astype(np.int64)
        rest = rest // np.uint64(T[l])
    return out


class ValidSet:
    """Eq. 5: the set V of valid item indices.  Exact: sorted unique keys, membership by binary search."""

    def __init__(self, catalog_codes: np.ndarray, T: Sequence[int]):
        self.T = tuple(int(t) for t in T)
        self.keys = np.unique(pack_keys(catalog_codes, self.T))
        self._prefix: Dict[int, np.ndarray] = {}

    def __len__(self) -> int:
        return int(self.keys.size)

    def contains_keys(self, keys: np.ndarray) -> np.ndarray:
        keys = np.asarray(keys, dtype=np.uint64)
        pos = np.searchsorted(self.keys, keys)
        pos = np.minimum(pos, self.keys.size - 1)
        return self.keys[pos] == keys

    def contains(self, codes: np.ndarray) -> np.ndarray:
        return self.contains_keys(pack_keys(codes, self.T))

    def prefix_keys(self, n: int) -> np.ndarray:
        """The sorted packed keys of the distinct n-code prefixes of the valid IDs.  Level 1 is the least significant digit
        of Eq. 4, so the key of an ID's first n codes is its own key modulo prod_{j<=n} T_j."""
        if n not in self._prefix:
            self._prefix[n] = np.unique(self.keys % np.uint64(int(np.prod([int(t) for t in self.T[:n]], dtype=object))))
        return self._prefix[n]

    def contains_prefix(self, codes: np.ndarray) -> np.ndarray:
        """Is each code tuple [..., n] (n <= L) the beginning of at least one valid ID?  (n = L: Eq. 5 itself.)"""
        codes = np.asarray(codes)
        n = codes.shape[-1]
        if n == len(self.T):
            return self.contains(codes)
        table = self.prefix_keys(n)
        keys = pack_keys(codes, self.T[:n])
        pos = np.minimum(np.searchsorted(table, keys), table.size - 1)
        return table[pos] == keys


# ----------------------------------------------------------------------------------------------------
# primary model M_p
# ----------------------------------------------------------------------------------------------------

@dataclass
class ModelShape:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    d_ffn: int
    L: int
    T: Tuple[int, ...]
    rope_theta: float = 10000.0
    rms_eps: float = 1e-6

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_q_heads

    @property
    def level_offset(self) -> List[int]:
        return [int(sum(self.T[:l])) for l in range(self.L)]

    def code_token(self, level: int, code: int) -> int:      # level is 0-based here
        return self.level_offset[level] + int(code)

    def sp_token(self, level: int) -> int:
        return int(sum(self.T)) + level

    @property
    def bos_token(self) -> int:
        return int(sum(self.T)) + self.L


def log_softmax(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    m = z.max(axis=-1, keepdims=True)
    return z - m - np.log(np.exp(z - m).sum(axis=-1, keepdims=True))


def rms_norm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding on x [n, heads, hd]: pair (i, i + hd/2) is rotated by pos * theta^(-2i/hd)."""
    hd = x.shape[-1]
    half = hd // 2
    inv = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / hd)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv[None, :]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


class PrimaryModel:
    """M_p.  Weights are given as float arrays (already rounded to their storage type); all arithmetic is fp64."""

    def __init__(self, shape: ModelShape, weights: Dict[str, object], cache_f64: bool = True, dtype=np.float64):
        """dtype: arithmetic type of the forward pass.  fp64 by default; fp32 is offered only so that a multi-billion
        parameter model can be checked in minutes (its rounding, ~1e-6 relative, is far below the bf16 tolerance)."""
        self.s = shape
        self.w = weights
        self.dtype = dtype
        self._cache: Optional[Dict[Tuple[str, Optional[int]], np.ndarray]] = {} if cache_f64 else None

    def _f64(self, name: str, layer: Optional[int] = None) -> np.ndarray:
        """The named weight as fp64 (converted copies are kept unless the model is too large for that)."""
        if self._cache is not None and (name, layer) in self._cache:
            return self._cache[(name, layer)]
        a = self.w[name] if layer is None else self.w[name][layer]
        a = np.asarray(a, dtype=self.dtype)
        if self._cache is not None:
            self._cache[(name, layer)] = a
        return a

    def forward(self, tokens: np.ndarray, positions: np.ndarray,
                past: Optional[List[Tuple[np.ndarray, np.ndarray]]] = None,
                visible_new: Optional[np.ndarray] = None):
        """Forward of `tokens` placed at `positions`, after an optional cached past.

        past[layer] = (K [n_past, kv_heads, hd], V [...]) -- rotated keys, as cached.
        visible_new [n, n] (bool): which of this call's tokens each token attends to; default = causal
        (token i sees tokens 0..i).  Every token sees the whole past.
        Returns (final-norm hidden [n, d], [(K_new, V_new)] per layer).
        """
        s = self.s
        tokens = np.asarray(tokens, dtype=np.int64)
        n = tokens.shape[0]
        hd, G = s.head_dim, s.n_q_heads // s.n_kv_heads
        x = self._f64("embed")[tokens]
        new_kv = []
        for layer in range(s.n_layers):
            xn = rms_norm(x, self._f64("attn_norm", layer), s.rms_eps)
            q = (xn @ self._f64("wq", layer).T).reshape(n, s.n_q_heads, hd)
            k = (xn @ self._f64("wk", layer).T).reshape(n, s.n_kv_heads, hd)
            v = (xn @ self._f64("wv", layer).T).reshape(n, s.n_kv_heads, hd)
            q = rope(q, positions, s.rope_theta).astype(self.dtype)
            k = rope(k, positions, s.rope_theta).astype(self.dtype)
            new_kv.append((k, v))
            if past is not None:
                k_all = np.concatenate([past[layer][0], k], axis=0)
                v_all = np.concatenate([past[layer][1], v], axis=0)
            else:
                k_all, v_all = k, v
            n_past = k_all.shape[0] - n
            attn = np.zeros((n, s.n_q_heads, hd), dtype=self.dtype)
            if visible_new is None:
                visible_new = np.tril(np.ones((n, n), dtype=bool))
            visible = np.concatenate([np.ones((n, n_past), dtype=bool), visible_new], axis=1)
            for h in range(s.n_q_heads):
                kv = h // G
                sc = q[:, h, :] @ k_all[:, kv, :].T / np.sqrt(hd)
                sc = np.where(visible, sc, -np.inf)
                p = np.exp(log_softmax(sc)).astype(self.dtype)
                attn[:, h, :] = p @ v_all[:, kv, :]
            x = x + attn.reshape(n, s.n_q_heads * hd) @ self._f64("wo", layer).T
            xn = rms_norm(x, self._f64("mlp_norm", layer), s.rms_eps)
            act = silu(xn @ self._f64("w_gate", layer).T) * (xn @ self._f64("w_up", layer).T)
            x = x + act @ self._f64("w_down", layer).T
        return rms_norm(x, self._f64("final_norm"), s.rms_eps), new_kv

    # -- request-level helpers ------------------------------------------------------------------------
    def prompt_tokens(self, hist_codes: np.ndarray) -> np.ndarray:
        """[BOS, history codes flattened item by item, level by level] for one request (hist [N, L])."""
        s = self.s
        toks = [s.bos_token]
        for item in np.asarray(hist_codes):
            toks.extend(s.code_token(l, item[l]) for l in range(s.L))
        return np.asarray(toks, dtype=np.int64)

    def prefill(self, hist_codes: np.ndarray) -> "Request":
        """Prefill step of Algorithm 3 (inference): one pass over context + L placeholders -> h_0..h_L; keeps the context KV only."""
        s = self.s
        ctx = self.prompt_tokens(hist_codes)
        P = ctx.shape[0]
        toks = np.concatenate([ctx, [s.sp_token(l) for l in range(s.L)]])
        hidden, kv = self.forward(toks, np.arange(P + s.L))
        return Request(P=P, h=hidden[P - 1: P + s.L].copy(), ctx_kv=[(k[:P], v[:P]) for k, v in kv])

    def next_level_logits(self, req: "Request", prefix: Sequence[int]) -> np.ndarray:
        """Model call and LM head of Algorithm 1 for one beam: logits over the codebook of level len(prefix)+1.

        M_p runs on the context plus the beam's codes (no placeholders); the LM head rows of the next level
        are applied to the hidden state of the last position.
        """
        return self.next_level_logits_many(req, [tuple(prefix)])[0]

    def next_level_logits_many(self, req: "Request", prefixes: Sequence[Tuple[int, ...]]) -> List[np.ndarray]:
        """The same for several beams of equal length j in one call: the beams' codes are laid side by side,
        each token attending to the context and to its own beam's codes up to itself (block-diagonal causal)."""
        s = self.s
        if not prefixes:
            return []
        j = len(prefixes[0])
        assert all(len(p) == j for p in prefixes)
        off = s.level_offset[j]
        head = self._f64("lm_head")[off: off + s.T[j]]
        if j == 0:
            return [head @ req.h[0] for _ in prefixes]
        toks, pos, owner = [], [], []
        for b, p in enumerate(prefixes):
            for l in range(j):
                toks.append(s.code_token(l, p[l]))
                pos.append(req.P + l)
                owner.append(b)
        owner = np.asarray(owner)
        idx = np.arange(len(toks))
        vis = (owner[:, None] == owner[None, :]) & (idx[None, :] <= idx[:, None])
        hidden, _ = self.forward(np.asarray(toks), np.asarray(pos), past=req.ctx_kv, visible_new=vis)
        return [head @ hidden[b * j + j - 1] for b in range(len(prefixes))]


@dataclass
class Request:
    P: int                                               # context length (BOS + history tokens)
    h: np.ndarray                                        # [L+1, d]: h_0 .. h_L
    ctx_kv: List[Tuple[np.ndarray, np.ndarray]] = field(default_factory=list)


# ----------------------------------------------------------------------------------------------------
# draft head, Eq. 1-3
# ----------------------------------------------------------------------------------------------------

class DraftHead:
    def __init__(self, shape: ModelShape, weights: Dict[str, object], additive_transition: bool = False,
                 use_hidden: bool = True, use_state: bool = True):
        """The switches are the ablation variants of Section 4.3: additive_transition = NEZHA-3 (Transition replaced by
        addition), use_state=False = NEZHA-1 (no context state, hence no transition), use_hidden=False = NEZHA-2."""
        self.s = shape
        self.w_logit = [np.asarray(a, dtype=np.float64) for a in weights["draft_logit"]]
        self.ws = np.asarray(weights["draft_ws"], dtype=np.float64)
        self.we = np.asarray(weights["draft_we"], dtype=np.float64)
        self.b = np.asarray(weights["draft_b"], dtype=np.float64)
        self.embed = weights["embed"]
        self.additive = additive_transition
        self.use_hidden, self.use_state = use_hidden, use_state

    def logits(self, level: int, h_l: np.ndarray, s_l: np.ndarray) -> np.ndarray:
        """Eq. 2 (level is 0-based: level 0 predicts the first code from h_1 and s_1)."""
        x = (h_l if self.use_hidden else 0.0) + (s_l if self.use_state else 0.0)
        return self.w_logit[level] @ (x + np.zeros_like(h_l))

    def transition(self, level: int, s_l: np.ndarray, code: int) -> np.ndarray:
        """Eq. 3 with e_l = embedding of the chosen level-`level` code."""
        e = np.asarray(self.embed[self.s.code_token(level, code)], dtype=np.float64)
        if self.additive:
            return s_l + e
        return np.tanh(self.ws @ s_l + self.we @ e + self.b)


# ----------------------------------------------------------------------------------------------------
# beam bookkeeping
# ----------------------------------------------------------------------------------------------------

@dataclass
class Beam:
    codes: Tuple[int, ...]
    score: np.float32
    parent: int = -1                                     # rank of the parent beam in the previous level


def _keep_best(cands: List[Tuple[np.float32, int, int]], K: int) -> List[Tuple[np.float32, int, int]]:
    """Keep the K candidates (score, parent rank, token) with the largest score; ties to smaller (parent, token)."""
    return sorted(cands, key=lambda c: (-float(c[0]), c[1], c[2]))[:K]


def _extend_score(parent_score: np.float32, logp: float) -> np.float32:
    """Cumulative log-probability, kept in fp32 (the precision the decision is taken in)."""
    return np.float32(np.float64(parent_score) + logp)


def expand_level(beams: List[Beam], logits: List[np.ndarray], K: int, per_beam: int,
                 valid: Optional[ValidSet]) -> List[Beam]:
    """One level of beam search.

    For every beam: log-softmax over the level's codebook, its `per_beam` most probable codes (the top-K step
    of Algorithm 1 / Algorithm 3), candidates = beam + code.  If `valid` is given, candidates that are not
    valid IDs are dropped (the verification step of Algorithm 3; Eq. 5).  The K candidates with the largest cumulative
    probability survive (the pruning step of Algorithm 1 / Algorithm 3).

    per_beam = K is the draft-head setting of Algorithm 3 (K x K candidates before the filter); per_beam = T_l
    applies the filter to every extension before the top-K (top-k restricted to valid tuples).
    The paper verifies at the last level only; the per-step variant it mentions (verification at every level, Section 3.4)
    passes `valid` at the earlier levels too, where a partial ID counts as valid if some valid ID begins with it.
    """
    cands: List[Tuple[np.float32, int, int]] = []
    for r, beam in enumerate(beams):
        logp = log_softmax(logits[r])
        order = sorted(range(logp.shape[0]), key=lambda t: (-logp[t], t))[:per_beam]
        for t in order:
            cands.append((_extend_score(beam.score, float(logp[t])), r, t))
    if valid is not None and cands:
        tuples = np.asarray([beams[r].codes + (t,) for _, r, t in cands], dtype=np.int64)
        ok = valid.contains_prefix(tuples)               # full-length tuples: Eq. 5; shorter ones: prefix of a valid ID
        cands = [c for c, keep in zip(cands, ok) if keep]
    return [Beam(beams[r].codes + (t,), sc, r) for sc, r, t in _keep_best(cands, K)]


# ----------------------------------------------------------------------------------------------------
# Algorithm 3 (inference): NEZHA draft-head beam search with hash-set verification
# ----------------------------------------------------------------------------------------------------

def teacher_forced_state(head: DraftHead, req: Request, codes: Sequence[int]) -> np.ndarray:
    """s_{len(codes)+1} along a fixed code prefix: Eq. 1 then Eq. 3 once per code."""
    s = req.h[0]
    for l, c in enumerate(codes):
        s = head.transition(l, s, c)
    return s


def nezha_draft(head: DraftHead, req: Request, K: int, valid: Optional[ValidSet],
                start: Optional[List[Beam]] = None, every_level: bool = False) -> List[List[Beam]]:
    """Algorithm 3, inference after the prefill.  Returns the beam sets of every level reached (last entry = final drafts).

    start = None is the paper's inference from the empty beam.  Otherwise drafting continues from the given
    beams of level m (the drafting step of Algorithm 2): their states are teacher-forced along their codes and their scores
    seed the cumulative probabilities.
    """
    L = head.s.L
    if start is None:
        beams, m = [Beam((), np.float32(0.0))], 0
    else:
        beams, m = list(start), len(start[0].codes) if start else L
    states = [teacher_forced_state(head, req, b.codes) for b in beams]
    levels: List[List[Beam]] = []
    for l in range(m, L):
        if not beams:
            levels.append([])
            continue
        logits = [head.logits(l, req.h[l + 1], st) for st in states]
        per_beam = min(K, head.s.T[l])
        nxt = expand_level(beams, logits, K, per_beam, valid if (l == L - 1 or every_level) else None)
        states = [head.transition(l, states[b.parent], b.codes[-1]) for b in nxt] if l < L - 1 else []
        beams = nxt
        levels.append(beams)
    return levels


# ----------------------------------------------------------------------------------------------------
# Algorithm 1: plain autoregressive beam search of M_p under the same validity filter
# ----------------------------------------------------------------------------------------------------

def ar_beam_search(model: PrimaryModel, req: Request, K: int, valid: Optional[ValidSet],
                   every_level: bool = False) -> List[List[Beam]]:
    """Returns [B_1, ..., B_L]; B_L is the result.  every_level: the validity filter at every level (prefixes of valid IDs)."""
    s = model.s
    beams = [Beam((), np.float32(0.0))]
    out = []
    for l in range(s.L):
        logits = model.next_level_logits_many(req, [b.codes for b in beams])
        beams = expand_level(beams, logits, K, s.T[l], valid if (l == s.L - 1 or every_level) else None)
        out.append(beams)
    return out


# ----------------------------------------------------------------------------------------------------
# Algorithm 2 instantiated: draft (Algorithm 3) -> one parallel M_p pass -> accept / roll back
# ----------------------------------------------------------------------------------------------------

@dataclass
class SpecStats:
    rounds: int = 0
    primary_tokens: int = 0                              # code tokens M_p processed, over all rounds
    accepted_len: List[List[int]] = field(default_factory=list)   # per round, per drafted tuple (the tree's level-L nodes)
    reject_level: List[int] = field(default_factory=list)         # per round: level m the round ended at
    tree_nodes: List[List[int]] = field(default_factory=list)     # per round: nodes of levels m+1..L-1 that were in the pass


def tree_from_tuples(tuples: Sequence[Tuple[int, ...]], L: int) -> List[List[Tuple[int, ...]]]:
    """The prefix tree of a list of drafted L-tuples: level j (1-based) holds their distinct j-prefixes, in order of
    first appearance.  Tuples that share a prefix share its node (one M_p token, not one per tuple)."""
    tree: List[List[Tuple[int, ...]]] = []
    for j in range(1, L + 1):
        seen: List[Tuple[int, ...]] = []
        for t in tuples:
            p = tuple(int(c) for c in t[:j])
            if p not in seen:
                seen.append(p)
        tree.append(seen)
    return tree


def alive_nodes(tree: List[List[Tuple[int, ...]]], B: List[Beam], m: int, L: int) -> Dict[int, List[Tuple[int, ...]]]:
    """Nodes of the draft tree that the pass holds, per level m..L-1: a level-m node is alive if it is a beam of B_m, a
    higher node if its parent is alive (its own prefix's earlier codes must be in the pass for it to attend to)."""
    beam_set = {b.codes for b in B}
    alive = {m: [t for t in tree[m - 1] if t in beam_set]}
    for j in range(m + 1, L):
        parents = set(alive[j - 1])
        alive[j] = [t for t in tree[j - 1] if t[:-1] in parents]
    return alive


def verification_walk(tree: List[List[Tuple[int, ...]]], B: List[Beam], m: int, L: int, next_beams):
    """One round of Algorithm 2 after drafting: the pass holds B_m and the alive nodes of levels m+1..L-1; B_{j+1} is
    selected from the logits at B_j (`next_beams(B_j, j)`), level after level, while every beam of B_j is an alive node
    (so its logits are in the pass).  The first level where that fails is the rejection level.  Returns the new true beam
    sets [B_{m+1}, ..., B_j] and the number of tree nodes of each level m+1..L-1 that were in the pass."""
    alive = alive_nodes(tree, B, m, L)
    new_sets: List[List[Beam]] = []
    j = m
    while True:
        B = next_beams(B, j)
        j += 1
        new_sets.append(B)
        if j == L:
            break
        in_pass = set(alive[j])
        if not all(b.codes in in_pass for b in B):
            break
    return new_sets, [len(alive[i]) for i in range(m + 1, L)]


def accepted_lengths(tuples: Sequence[Tuple[int, ...]], true_sets: List[List[Beam]], reached: int) -> List[int]:
    """Accepted length of every drafted tuple: the largest i <= `reached` such that each of its prefixes of 1..i codes is
    a beam of the true set of that level (accept until the first rejection, Section 2.2)."""
    acc = []
    for t in tuples:
        a = 0
        for i in range(1, reached + 1):
            if t[:i] in {b.codes for b in true_sets[i - 1]}:
                a = i
            else:
                break
        acc.append(a)
    return acc


def speculative_decode(model: PrimaryModel, head: DraftHead, req: Request, K: int, valid: Optional[ValidSet],
                       drafts_round1: Optional[List[Tuple[int, ...]]] = None,
                       draft_tree_round1: Optional[List[List[Tuple[int, ...]]]] = None,
                       use_drafts: bool = True, every_level: bool = False,
                       adaptive: bool = False) -> Tuple[List[List[Beam]], SpecStats]:
    """Algorithm 2 with the readings listed in the module header.

    B_1 comes from the prefill hidden state h_0.  Each round, with m levels settled (true beams B_m):
      * draft tree: what the draft model proposes is the whole level-wise beam tree of Algorithm 3, one node per distinct
        drafted prefix: round 1 = the beam sets D_1..D_L of NEZHA's search from the empty beam; later rounds = the sets
        D_{m+1}..D_L of the search continued from B_m.  `draft_tree_round1` overrides round 1's tree (level j = a list
        of j-tuples); `drafts_round1` gives final tuples only, whose prefixes form the tree.
      * a node of level m is *alive* if it is a beam of B_m; a node of a higher level if its parent is an alive node.
      * the M_p pass ("verify in parallel", Section 2.2) processes the level-m code of every beam of B_m and the last code
        of every alive node of levels m+1..L-1 (each token attends to the context and to its own prefix's earlier codes).
      * selection walks forward: B_{j+1} from the logits at the beams of B_j, while every beam of B_j is an alive node
        (so its logits are in the pass); the first level where that fails is the rejection level of Algorithm 2; the
        round ends there and m <- that level.
      * accepted length of a drafted tuple = the largest i <= (level reached) whose i-prefix is a beam of B_i.
    Every B_j is computed from M_p's logits only, so the result equals ar_beam_search whatever the drafts.
    use_drafts=False gives L-1 rounds of plain autoregressive steps.  every_level: the validity filter at every level,
    in the draft head's search and in the primary model's alike.  adaptive: a request stops drafting once a round has
    gained nothing from its drafts -- it settled only the one level that the pass settles anyway -- and finishes with plain
    autoregressive steps (an engine policy, not part of Algorithm 2; the result is Algorithm 1's either way).
    """
    s = model.s
    L = s.L
    stats = SpecStats()
    true_sets: List[List[Beam]] = []
    B = expand_level([Beam((), np.float32(0.0))], [model.next_level_logits(req, ())], K, s.T[0],
                     valid if (L == 1 or every_level) else None)
    true_sets.append(B)
    m = 1
    speculate = True
    while m < L:
        stats.rounds += 1
        # ---- draft (Algorithm 2, drafting step): tree[j - 1] = drafted nodes of level j
        tree: List[List[Tuple[int, ...]]] = [[] for _ in range(L)]
        if not use_drafts or not speculate:
            pass
        elif stats.rounds == 1 and draft_tree_round1 is not None:
            tree = [[tuple(int(c) for c in t) for t in lv] for lv in draft_tree_round1]
        elif stats.rounds == 1 and drafts_round1 is not None:
            tree = tree_from_tuples(drafts_round1, L)
        elif stats.rounds == 1:
            tree = [[b.codes for b in lv] for lv in nezha_draft(head, req, K, valid, every_level=every_level)]
        else:
            lv = nezha_draft(head, req, K, valid, start=B, every_level=every_level)   # levels m+1 .. L
            tree[m - 1] = [b.codes for b in B]
            for i, beams in enumerate(lv):
                tree[m + i] = [b.codes for b in beams]
        # ---- the parallel verification pass, progressive selection / rejection (Algorithm 2, rejection and update steps)
        def next_beams(beams: List[Beam], j: int) -> List[Beam]:
            logits = model.next_level_logits_many(req, [b.codes for b in beams])
            return expand_level(beams, logits, K, s.T[j], valid if (j + 1 == L or every_level) else None)
        new_sets, nodes = verification_walk(tree, B, m, L, next_beams)
        true_sets.extend(new_sets)                       # true_sets[i - 1] is B_i
        B = true_sets[-1]
        j = len(true_sets)
        stats.tree_nodes.append(nodes)
        stats.primary_tokens += len(true_sets[m - 1]) + sum(nodes)
        stats.accepted_len.append(accepted_lengths(tree[L - 1], true_sets, j))
        stats.reject_level.append(j)
        if adaptive:
            speculate = j - m >= 2
        m = j
    return true_sets, stats


# ----------------------------------------------------------------------------------------------------
# brute force (tiny code spaces only)
# ----------------------------------------------------------------------------------------------------

def joint_logprob_primary(model: PrimaryModel, req: Request, codes: Sequence[int]) -> float:
    """log p(codes) under M_p by teacher forcing, one level at a time."""
    total = 0.0
    for l in range(len(codes)):
        total += float(log_softmax(model.next_level_logits(req, tuple(codes[:l])))[codes[l]])
    return total


def joint_logprob_draft(head: DraftHead, req: Request, codes: Sequence[int]) -> float:
    """log p(codes) under the draft head by teacher forcing (the teacher-forced loop of Algorithm 3's training part)."""
    total = 0.0
    st = req.h[0]
    for l in range(len(codes)):
        total += float(log_softmax(head.logits(l, req.h[l + 1], st))[codes[l]])
        st = head.transition(l, st, codes[l])
    return total


def outputs_as_arrays(beams: List[Beam], K: int, L: int):
    """Fixed-size result: codes [K, L] padded with -1, scores [K] padded with -inf, count."""
    codes = -np.ones((K, L), dtype=np.int32)
    scores = np.full((K,), NEG_INF, dtype=np.float32)
    for r, b in enumerate(beams[:K]):
        codes[r, : len(b.codes)] = b.codes
        scores[r] = b.score
    return codes, scores, min(len(beams), K)
