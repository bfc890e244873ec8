"""Pins of the CPU oracle to things other than itself: the paper's worked example, closed forms,
an independent library implementation of the backbone, brute-force enumeration.  No GPU needed."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import nezha_oracle as O
from paper_2511_18793_b200 import synth
from helpers import MICRO, codes_of, oracle_bundle, oracle_shape, scores_of

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------------------- Eq. 4 / 5
def test_eq4_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "eq4_worked_example.txt")) if not l.startswith("#")]
    for t1, t2, t3, T, idx in rows:
        key = O.pack_keys(np.array([int(t1), int(t2), int(t3)]), (int(T),) * 3)
        assert int(key) == int(idx)


def test_eq4_level1_is_least_significant_and_bijective():
    T = (32, 32, 32)
    grid = np.stack(np.meshgrid(*[np.arange(t) for t in T], indexing="ij"), axis=-1).reshape(-1, 3)
    keys = O.pack_keys(grid, T)
    assert np.array_equal(np.sort(keys), np.arange(32 ** 3, dtype=np.uint64))       # onto [0, prod T)
    assert np.array_equal(O.unpack_keys(keys, T), grid)                              # round trip
    assert int(O.pack_keys(np.array([1, 0, 0]), T)) == 1
    assert int(O.pack_keys(np.array([0, 0, 1]), T)) == 32 * 32
    T2 = (3, 5, 7, 11)                                                                # unequal radices
    grid2 = np.stack(np.meshgrid(*[np.arange(t) for t in T2], indexing="ij"), axis=-1).reshape(-1, 4)
    k2 = O.pack_keys(grid2, T2)
    assert np.array_equal(np.sort(k2), np.arange(3 * 5 * 7 * 11, dtype=np.uint64))
    assert int(O.pack_keys(np.array([2, 4, 6, 10]), T2)) == 2 + 4 * 3 + 6 * 15 + 10 * 105


def test_eq4_no_overflow_at_256_pow_4_and_larger():
    assert int(O.pack_keys(np.array([255, 255, 255, 255]), (256,) * 4)) == 2 ** 32 - 1
    assert int(O.pack_keys(np.array([255] * 7), (256,) * 7)) == 2 ** 56 - 1


def test_valid_set_matches_python_set():
    w = synth.WORKLOADS["tiny"]
    cat = synth.make_catalog(w)
    cat_dup = np.concatenate([cat, cat[:100]])                                       # duplicates count once
    V = O.ValidSet(cat_dup, w.T)
    ref = {tuple(r) for r in cat.tolist()}
    assert len(V) == len(ref) == w.n_items
    grid = np.stack(np.meshgrid(*[np.arange(t) for t in w.T], indexing="ij"), axis=-1).reshape(-1, w.L)
    got = V.contains(grid)
    want = np.array([tuple(r) in ref for r in grid.tolist()])
    assert np.array_equal(got, want)
    assert got.sum() == w.n_items
    # a key beyond the largest stored key
    assert not V.contains_keys(np.array([2 ** 40], dtype=np.uint64))[0]


# ---------------------------------------------------------------------------------------- backbone
def _hf_llama(w, W):
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(vocab_size=w.vocab, hidden_size=w.d_model, intermediate_size=w.d_ffn,
                      num_hidden_layers=w.n_layers, num_attention_heads=w.n_q_heads,
                      num_key_value_heads=w.n_kv_heads, rms_norm_eps=w.rms_eps, rope_theta=w.rope_theta,
                      attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
                      max_position_embeddings=4096, head_dim=w.head_dim)
    cfg._attn_implementation = "eager"
    m = LlamaForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": W["embed"], "model.norm.weight": W["final_norm"], "lm_head.weight": W["lm_head"]}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj", "wo": "self_attn.o_proj",
             "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj",
             "attn_norm": "input_layernorm", "mlp_norm": "post_attention_layernorm"}
    for i in range(w.n_layers):
        for k, n in names.items():
            sd[f"model.layers.{i}.{n}.weight"] = W[k][i]
    sd = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in sd.items()}
    missing = m.load_state_dict(sd, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k], missing
    return m


@pytest.mark.parametrize("kv_heads", [4, 2, 1])
def test_backbone_matches_library_llama(kv_heads):
    """The backbone reading (RMSNorm, half-split rotary, GQA, SwiGLU, untied head) is the Llama architecture:
    the oracle's forward must equal the library implementation on the same weights."""
    w = synth.scaled(synth.WORKLOADS["tiny"], n_kv_heads=kv_heads)
    W = synth.weights_to_numpy(synth.make_weights(w))
    model = O.PrimaryModel(oracle_shape(w), W)
    hist = synth.make_histories(w, None)[0]
    toks = model.prompt_tokens(hist)
    hidden, _ = model.forward(toks, np.arange(toks.shape[0]))
    hf = _hf_llama(w, W)
    with torch.no_grad():
        out = hf(input_ids=torch.from_numpy(toks)[None])
        ref_hidden = hf.model(input_ids=torch.from_numpy(toks)[None]).last_hidden_state[0].numpy()
    # the library builds its rotary tables in fp32 even for an fp64 model: agreement is to ~1e-7, while a
    # wrong convention (pairing, GQA grouping, norm placement) is off by O(0.1)
    assert np.abs(hidden - ref_hidden).max() < 5e-6
    logits = hidden @ np.asarray(W["lm_head"], dtype=np.float64).T
    assert np.abs(logits - out.logits[0].numpy()).max() < 5e-6


def test_prompt_layout_and_hidden_positions():
    w = synth.WORKLOADS["tiny"]
    W = synth.weights_to_numpy(synth.make_weights(w))
    model = O.PrimaryModel(oracle_shape(w), W)
    hist = synth.make_histories(w, None)[1]
    toks = model.prompt_tokens(hist)
    assert toks.shape[0] == 1 + w.n_hist * w.L == w.ctx_tokens
    assert toks[0] == sum(w.T) + w.L                                                # BOS
    assert toks[1] == hist[0, 0] and toks[2] == w.T[0] + hist[0, 1] and toks[3] == w.T[0] + w.T[1] + hist[0, 2]
    req = model.prefill(hist)
    full = np.concatenate([toks, [sum(w.T) + l for l in range(w.L)]])
    hidden, kv = model.forward(full, np.arange(full.shape[0]))
    assert np.array_equal(req.h, hidden[req.P - 1:])                                # h_0 .. h_L
    assert req.h.shape == (w.L + 1, w.d_model)
    assert req.ctx_kv[0][0].shape[0] == req.P                                       # placeholders not cached


def test_cached_continuation_equals_full_recompute():
    """Plain autoregressive decoding: context + codes, no placeholders; cached == recomputed."""
    w = synth.scaled(synth.WORKLOADS["tiny"], n_kv_heads=2)
    W = synth.weights_to_numpy(synth.make_weights(w))
    model = O.PrimaryModel(oracle_shape(w), W)
    hist = synth.make_histories(w, None)[2]
    req = model.prefill(hist)
    prefixes = [(3, 7), (3, 9), (30, 1)]
    got = model.next_level_logits_many(req, prefixes)
    ctx = model.prompt_tokens(hist)
    for p, g in zip(prefixes, got):
        toks = np.concatenate([ctx, [p[0], w.T[0] + p[1]]])
        hidden, _ = model.forward(toks, np.arange(toks.shape[0]))
        ref = np.asarray(W["lm_head"], dtype=np.float64)[w.T[0] + w.T[1]: sum(w.T)] @ hidden[-1]
        assert np.abs(g - ref).max() < 1e-10
    # level 1 uses h_0 and the first codebook's head rows
    z1 = model.next_level_logits(req, ())
    assert np.allclose(z1, np.asarray(W["lm_head"], dtype=np.float64)[: w.T[0]] @ req.h[0], atol=0, rtol=0)


def test_backbone_closed_forms():
    w = synth.WORKLOADS["tiny"]
    W = synth.weights_to_numpy(synth.make_weights(w))
    # zero output projections: every layer adds nothing, hidden = RMSNorm(embedding)
    W0 = dict(W)
    W0["wo"] = [np.zeros_like(a) for a in W["wo"]]
    W0["w_down"] = [np.zeros_like(a) for a in W["w_down"]]
    model = O.PrimaryModel(oracle_shape(w), W0)
    toks = np.array([5, 40, 70, 99])
    hidden, _ = model.forward(toks, np.arange(4))
    e = np.asarray(W["embed"], dtype=np.float64)[toks]
    ref = e / np.sqrt((e ** 2).mean(-1, keepdims=True) + w.rms_eps) * np.asarray(W["final_norm"], dtype=np.float64)
    assert np.abs(hidden - ref).max() < 1e-12
    # rotary: position 0 is the identity, norms are preserved, scores depend on relative position only
    rng = np.random.default_rng(0)
    x = rng.standard_normal((1, 2, 16))
    y = rng.standard_normal((1, 2, 16))
    assert np.allclose(O.rope(x, np.array([0]), 10000.0), x)
    assert np.allclose(np.linalg.norm(O.rope(x, np.array([17]), 10000.0)), np.linalg.norm(x))
    a = (O.rope(x, np.array([9]), 10000.0) * O.rope(y, np.array([4]), 10000.0)).sum()
    b = (O.rope(x, np.array([25]), 10000.0) * O.rope(y, np.array([20]), 10000.0)).sum()
    assert abs(a - b) < 1e-12
    # first pair (i = 0) rotates by exactly `pos` radians between elements 0 and hd/2
    v = np.zeros((1, 1, 16)); v[0, 0, 0] = 1.0
    r = O.rope(v, np.array([1]), 10000.0)[0, 0]
    assert abs(r[0] - np.cos(1.0)) < 1e-15 and abs(r[8] - np.sin(1.0)) < 1e-15
    # library routines
    z = rng.standard_normal((3, 11))
    assert np.allclose(O.log_softmax(z), torch.log_softmax(torch.from_numpy(z), -1).numpy(), atol=1e-14)
    assert np.allclose(O.silu(z), torch.nn.functional.silu(torch.from_numpy(z)).numpy(), atol=1e-14)


# ---------------------------------------------------------------------------------------- draft head
def _micro():
    w = MICRO
    W = synth.weights_to_numpy(synth.make_weights(w, std=0.5))       # large std: well-separated scores
    cat = synth.make_catalog(w)
    model, head, V = oracle_bundle(w, W, cat)
    hist = synth.make_histories(w, None)
    return w, W, cat, model, head, V, hist


def _all_tuples(T):
    return list(itertools.product(*[range(t) for t in T]))


def test_draft_equations_1_to_3():
    w, W, cat, model, head, V, hist = _micro()
    req = model.prefill(hist[0])
    f = lambda n: np.asarray(W[n], dtype=np.float64)
    s1 = req.h[0]                                                                    # Eq. 1
    z1 = np.asarray(W["draft_logit"][0], dtype=np.float64) @ (req.h[1] + s1)         # Eq. 2
    assert np.array_equal(head.logits(0, req.h[1], s1), z1)
    code = 2
    e = f("embed")[code]
    s2 = np.tanh(f("draft_ws") @ s1 + f("draft_we") @ e + f("draft_b"))              # Eq. 3
    assert np.array_equal(head.transition(0, s1, code), s2)
    # level-2 code ids are offset by T_1 in the embedding table
    e2 = f("embed")[w.T[0] + 3]
    s3 = np.tanh(f("draft_ws") @ s2 + f("draft_we") @ e2 + f("draft_b"))
    assert np.array_equal(head.transition(1, s2, 3), s3)
    lp = O.joint_logprob_draft(head, req, (2, 3, 1))
    z2 = np.asarray(W["draft_logit"][1], dtype=np.float64) @ (req.h[2] + s2)
    z3 = np.asarray(W["draft_logit"][2], dtype=np.float64) @ (req.h[3] + s3)
    want = sum(float(torch.log_softmax(torch.from_numpy(z), -1)[c]) for z, c in ((z1, 2), (z2, 3), (z3, 1)))
    assert abs(lp - want) < 1e-12


def test_nezha_draft_equals_brute_force_when_nothing_is_pruned():
    """K >= prod_{l<L} T_l: no level prunes, so Algorithm 3 must return the K best valid tuples."""
    w, W, cat, model, head, V, hist = _micro()
    valid = {tuple(r) for r in cat.tolist()}
    for b in range(hist.shape[0]):
        req = model.prefill(hist[b])
        K = 16
        out = O.nezha_draft(head, req, K, V)[-1]
        scored = sorted(((O.joint_logprob_draft(head, req, t), t) for t in _all_tuples(w.T) if t in valid),
                        key=lambda x: -x[0])
        # per-beam top-K at the last level keeps min(K, T) = all 4 codes, so nothing else is lost
        assert codes_of(out) == [t for _, t in scored[:K]]
        assert np.allclose(scores_of(out), [s for s, _ in scored[:K]], atol=1e-5)
        assert all(t in valid for t in codes_of(out))


def test_nezha_draft_pruned_scores_and_validity():
    """Small K: outputs are valid, scores are the independently recomputed joint log-probabilities,
    ordered, and the number of last-level candidates before filtering is at most K x K."""
    w, W, cat, model, head, V, hist = _micro()
    valid = {tuple(r) for r in cat.tolist()}
    req = model.prefill(hist[1])
    for K in (1, 2, 3, 5):
        levels = O.nezha_draft(head, req, K, V)
        assert [len(lv) <= K for lv in levels] == [True] * w.L
        out = levels[-1]
        assert all(t in valid for t in codes_of(out))
        for bm in out:
            assert abs(float(bm.score) - O.joint_logprob_draft(head, req, bm.codes)) < 1e-5
        sc = scores_of(out)
        assert np.all(sc[:-1] >= sc[1:])
        # every output extends a surviving beam of the previous level (filtering happens at l = L only)
        prev = set(codes_of(levels[-2]))
        assert all(t[:-1] in prev for t in codes_of(out))
    # K = 1 is greedy on the first L-1 levels
    lv = O.nezha_draft(head, req, 1, None)
    t1 = int(np.argmax(head.logits(0, req.h[1], req.h[0])))
    assert lv[0][0].codes == (t1,)


def test_nezha_draft_without_filter_is_plain_beam_search_of_the_head():
    w, W, cat, model, head, V, hist = _micro()
    req = model.prefill(hist[0])
    out = O.nezha_draft(head, req, 16, None)[-1]
    scored = sorted(((O.joint_logprob_draft(head, req, t), t) for t in _all_tuples(w.T)), key=lambda x: -x[0])
    assert codes_of(out) == [t for _, t in scored[:16]]


def test_zero_heads_closed_form_pins_tie_rule():
    """All-zero logit heads: every tuple scores -sum(log T_l); the survivors are decided by the tie rule
    (smaller parent rank, then smaller token) = lexicographic order."""
    w, W, cat, model, head, V, hist = _micro()
    Wz = dict(W)
    Wz["draft_logit"] = [np.zeros_like(a) for a in W["draft_logit"]]
    Wz["lm_head"] = np.zeros_like(W["lm_head"])
    model, head, V = oracle_bundle(w, Wz, cat)
    req = model.prefill(hist[0])
    valid = sorted({tuple(r) for r in cat.tolist()})
    K = 16                                                    # = T_1 * T_2: no pruning before the last level
    uniform = np.float32(-np.log(4.0) * 3)
    for out in (O.nezha_draft(head, req, K, V)[-1], O.ar_beam_search(model, req, K, V)[-1]):
        assert codes_of(out) == valid[:K]
        assert np.allclose(scores_of(out), uniform, atol=1e-6)
    # K = 3 < T: level 1 keeps codes 0,1,2; level 2 keeps (0,0),(0,1),(0,2); the draft path then takes the
    # 3 smallest codes of each beam *before* filtering, the primary path filters all 4 first.
    vs = set(valid)
    d = [(0, b, c) for b in range(3) for c in range(3) if (0, b, c) in vs][:3]
    p = [(0, b, c) for b in range(3) for c in range(4) if (0, b, c) in vs][:3]
    assert codes_of(O.nezha_draft(head, req, 3, V)[-1]) == d
    assert codes_of(O.ar_beam_search(model, req, 3, V)[-1]) == p


# ---------------------------------------------------------------------------------------- Algorithm 1
def _joint_primary_full_recompute(model, W, w, hist_row, codes):
    """Independent path: one uncached forward over [context, codes], log-softmax per level's head rows."""
    ctx = model.prompt_tokens(hist_row)
    offs = [sum(w.T[:l]) for l in range(w.L)]
    toks = np.concatenate([ctx, [offs[l] + codes[l] for l in range(w.L - 1)]])
    hidden, _ = model.forward(toks, np.arange(toks.shape[0]))
    P = ctx.shape[0]
    head = np.asarray(W["lm_head"], dtype=np.float64)
    total = 0.0
    for l in range(w.L):
        z = torch.from_numpy(head[offs[l]: offs[l] + w.T[l]] @ hidden[P - 1 + l])
        total += float(torch.log_softmax(z, -1)[codes[l]])
    return total


def test_ar_beam_search_equals_brute_force_and_has_no_hallucinations():
    w, W, cat, model, head, V, hist = _micro()
    valid = {tuple(r) for r in cat.tolist()}
    for b in range(hist.shape[0]):
        req = model.prefill(hist[b])
        K = 16
        out = O.ar_beam_search(model, req, K, V)[-1]
        scored = sorted(((_joint_primary_full_recompute(model, W, w, hist[b], t), t)
                         for t in _all_tuples(w.T) if t in valid), key=lambda x: -x[0])
        assert codes_of(out) == [t for _, t in scored[:K]]
        assert np.allclose(scores_of(out), [s for s, _ in scored[:K]], atol=1e-5)
        # pruned search: still valid, scores still the true joint log-probabilities
        for K2 in (1, 2, 5):
            o2 = O.ar_beam_search(model, req, K2, V)[-1]
            assert all(t in valid for t in codes_of(o2))
            for bm in o2:
                assert abs(float(bm.score) - _joint_primary_full_recompute(model, W, w, hist[b], bm.codes)) < 1e-5
        # K = 1: greedy on levels 1..L-1
        g = O.ar_beam_search(model, req, 1, None)
        assert g[0][0].codes == (int(np.argmax(model.next_level_logits(req, ()))),)
        assert O.joint_logprob_primary(model, req, out[0].codes) == pytest.approx(float(out[0].score), abs=1e-5)


def test_fewer_valid_than_k_and_k_larger_than_codebook():
    w, W, cat, model, head, V, hist = _micro()
    few = cat[:3]
    Vs = O.ValidSet(few, w.T)
    req = model.prefill(hist[0])
    out = O.ar_beam_search(model, req, 16, Vs)
    assert len(out[0]) == 4 and len(out[1]) == 16                   # |B_1| = min(K, T_1)
    assert sorted(codes_of(out[-1])) == sorted(tuple(r) for r in few.tolist())
    codes, scores, cnt = O.outputs_as_arrays(out[-1], 16, w.L)
    assert cnt == 3 and np.all(codes[3:] == -1) and np.all(np.isneginf(scores[3:]))
    d = O.nezha_draft(head, req, 16, O.ValidSet(np.array([[9, 9, 9]]), (16, 16, 16)))
    assert d[-1] == []


# ---------------------------------------------------------------------------------------- Algorithm 2
def test_speculative_decode_equals_autoregressive_beam_search():
    """The zero-sacrifice invariant: whatever is drafted, the verified result is Algorithm 1's."""
    w = synth.WORKLOADS["tiny"]
    W = synth.weights_to_numpy(synth.make_weights(w))
    cat = synth.make_catalog(w)
    model, head, V = oracle_bundle(w, W, cat)
    hist = synth.make_histories(w, None)
    valid = {tuple(r) for r in cat.tolist()}
    for b in range(w.batch):
        req = model.prefill(hist[b])
        ar = O.ar_beam_search(model, req, w.beam, V)
        for kw in ({}, {"use_drafts": False}):
            sp, st = O.speculative_decode(model, head, req, w.beam, V, **kw)
            assert [codes_of(x) for x in sp] == [codes_of(x) for x in ar]
            assert all(np.array_equal(scores_of(x), scores_of(y)) for x, y in zip(sp, ar))
            assert st.rounds <= w.L - 1
            assert all(t in valid for t in codes_of(sp[-1]))
        _, st = O.speculative_decode(model, head, req, w.beam, V, use_drafts=False)
        assert st.rounds == w.L - 1 and st.primary_tokens == sum(len(x) for x in ar[:-1])
        # perfect draft tree (the true beam sets themselves): one round, every tuple accepted in full, and the pass costs
        # exactly the tokens plain autoregressive decoding needs over its L-1 calls
        sp, st = O.speculative_decode(model, head, req, w.beam, V, draft_tree_round1=[codes_of(x) for x in ar])
        assert codes_of(sp[-1]) == codes_of(ar[-1])
        assert st.rounds == 1 and st.accepted_len == [[w.L] * len(ar[-1])] and st.reject_level == [w.L]
        assert st.primary_tokens == sum(len(x) for x in ar[:-1])
        # the true final tuples alone: every prefix of a tuple of B_L is a beam of its level, so each tuple is accepted up
        # to the level the round reached, whatever that level is
        sp, st = O.speculative_decode(model, head, req, w.beam, V, drafts_round1=codes_of(ar[-1]))
        assert codes_of(sp[-1]) == codes_of(ar[-1])
        assert st.accepted_len[0] == [st.reject_level[0]] * len(ar[-1])
        # drafts whose first code is not in B_1: nothing accepted, L-1 rounds
        b1 = {t[0] for t in codes_of(ar[0])}
        bad = [c for c in range(w.T[0]) if c not in b1][: w.beam]
        sp, st = O.speculative_decode(model, head, req, w.beam, V, drafts_round1=[(c, 0, 0) for c in bad])
        assert codes_of(sp[-1]) == codes_of(ar[-1])
        assert st.accepted_len[0] == [0] * len(bad) and st.rounds == w.L - 1


def test_speculative_round_two_drafts_extend_true_beams():
    w = synth.WORKLOADS["tiny"]
    W = synth.weights_to_numpy(synth.make_weights(w))
    cat = synth.make_catalog(w)
    model, head, V = oracle_bundle(w, W, cat)
    req = model.prefill(synth.make_histories(w, None)[0])
    ar = O.ar_beam_search(model, req, w.beam, V)
    lv = O.nezha_draft(head, req, w.beam, V, start=ar[1])             # continue from B_2
    b2 = set(codes_of(ar[1]))
    assert all(t[:2] in b2 for t in codes_of(lv[-1]))
    for bm in lv[-1]:                                                   # true score of the prefix + head's log-prob
        parent = [x for x in ar[1] if x.codes == bm.codes[:2]][0]
        st = O.teacher_forced_state(head, req, bm.codes[:2])
        lp = float(O.log_softmax(head.logits(2, req.h[3], st))[bm.codes[2]])
        assert abs(float(bm.score) - (float(parent.score) + lp)) < 1e-5


def _zero_head_case(catalog):
    """MICRO with every logit head zero: all probabilities are uniform, so the tie rule (smaller parent rank, then
    smaller code) fixes every beam set by hand.  With K = 2: B_1 = {(0), (1)}, B_2 = {(0,0), (0,1)}, B_3 = the first two
    valid tuples among (0,0,c), (0,1,c) in that order; the draft head's sets are the same before its filter."""
    w = MICRO
    W = synth.weights_to_numpy(synth.make_weights(w, std=0.5))
    W = dict(W)
    W["draft_logit"] = [np.zeros_like(a) for a in W["draft_logit"]]
    W["lm_head"] = np.zeros_like(W["lm_head"])
    model, head, V = oracle_bundle(w, W, np.asarray(catalog, dtype=np.int32))
    req = model.prefill(synth.make_histories(w, None)[0])
    return model, head, V, req


def test_speculative_walk_hand_worked_cases():
    """Accept-until-first-rejection (Section 2.2), worked by hand on the zero-head case.  Expected values below are
    derived in the comments from the rule, not from the oracle."""
    cat = [(0, 0, 2), (0, 1, 1), (0, 1, 3), (1, 0, 0), (3, 3, 3)]
    model, head, V, req = _zero_head_case(cat)
    K = 2
    ar = O.ar_beam_search(model, req, K, V)
    assert [codes_of(x) for x in ar] == [[(0,), (1,)], [(0, 0), (0, 1)], [(0, 0, 2), (0, 1, 1)]]
    # (a) partly right.  Tree of the tuples: level 1 {(0),(1)}, level 2 {(0,0),(1,0)}.  Round 1 (m = 1): the pass holds
    #     B_1's 2 tokens + the 2 level-2 nodes (both have an alive parent) = 4.  B_2 = {(0,0),(0,1)}; (0,1) is no node:
    #     rejection at level 2.  (0,0,2): prefixes (0) in B_1, (0,0) in B_2 -> 2.  (1,0,0): (1) in B_1, (1,0) not in B_2 -> 1.
    #     Round 2 (m = 2 = L-1): only B_2's 2 tokens; the zero draft head proposes codes 0,1 of each beam, of which only
    #     (0,1,1) is valid -> one drafted tuple, which is in B_3 -> 3.
    sp, st = O.speculative_decode(model, head, req, K, V, drafts_round1=[(0, 0, 2), (1, 0, 0)])
    assert codes_of(sp[-1]) == [(0, 0, 2), (0, 1, 1)]
    assert (st.rounds, st.reject_level, st.accepted_len, st.primary_tokens) == (2, [2, 3], [[2, 1], [3]], 6)
    assert st.tree_nodes == [[2], []]
    # (b) first codes wrong: no node of level 1 is a beam, nothing beyond B_1 is in the pass (2 tokens), rejection at
    #     level 2, accepted lengths 0; round 2 as above.  Total = the 4 tokens of plain autoregressive decoding.
    sp, st = O.speculative_decode(model, head, req, K, V, drafts_round1=[(2, 0, 0), (3, 3, 3)])
    assert (st.rounds, st.reject_level, st.accepted_len, st.primary_tokens) == (2, [2, 3], [[0, 0], [3]], 4)
    # (c) the true tuples: level 1 of their tree is {(0)} only, but B_1's own tokens are always in the pass; level 2 is
    #     {(0,0),(0,1)} = B_2 -> the walk reaches level 3 in one round; 2 + 2 tokens.
    sp, st = O.speculative_decode(model, head, req, K, V, drafts_round1=[(0, 0, 2), (0, 1, 1)])
    assert (st.rounds, st.reject_level, st.accepted_len, st.primary_tokens) == (1, [3], [[3, 3]], 4)
    # (d) shared prefixes are one node: four tuples under (0,0) and (0,1) still cost 2 level-2 tokens; (0,0,0) is not
    #     in B_3 but its first two codes are beams -> 2.
    sp, st = O.speculative_decode(model, head, req, K, V, drafts_round1=[(0, 0, 0), (0, 0, 2), (0, 1, 1), (0, 1, 3)])
    assert (st.rounds, st.primary_tokens, st.tree_nodes) == (1, 4, [[2]])
    assert st.accepted_len == [[2, 3, 3, 2]]
    # (e) a level-2 node whose parent is no beam is dead: (2,0) costs no token; (0,0) alone does not cover B_2
    sp, st = O.speculative_decode(model, head, req, K, V, draft_tree_round1=[[(0,), (2,)], [(0, 0), (2, 0)], [(0, 0, 2), (2, 0, 0)]])
    assert (st.rounds, st.reject_level, st.tree_nodes[0], st.accepted_len[0]) == (2, [2, 3], [1], [2, 0])
    # (f) the natural path (zero draft head): its level sets are D_1 = {(0),(1)}, D_2 = {(0,0),(0,1)} = the true ones,
    #     D_3 = valid among (0,0,0),(0,0,1),(0,1,0),(0,1,1) = {(0,1,1)} -> one round, that tuple accepted in full
    sp, st = O.speculative_decode(model, head, req, K, V)
    assert (st.rounds, st.reject_level, st.accepted_len, st.primary_tokens) == (1, [3], [[3]], 4)
    assert codes_of(sp[-1]) == [(0, 0, 2), (0, 1, 1)]


def test_adaptive_drafting_stops_after_a_round_without_gain():
    """The engine policy on top of Algorithm 2: a round that settled only the one level the pass settles anyway turns the
    request's drafting off.  Hand-worked on the zero-head case, and against plain drafting on random trees: same result,
    never more tokens."""
    cat = [(0, 0, 2), (0, 1, 1), (0, 1, 3), (1, 0, 0), (3, 3, 3)]
    model, head, V, req = _zero_head_case(cat)
    # first codes wrong: round 1 gains nothing (reaches level 2 = 1 + 1) -> round 2 drafts nothing: no drafted tuple, no
    # tree node, B_2's 2 tokens only
    sp, st = O.speculative_decode(model, head, req, 2, V, drafts_round1=[(2, 0, 0), (3, 3, 3)], adaptive=True)
    assert codes_of(sp[-1]) == [(0, 0, 2), (0, 1, 1)]
    assert (st.rounds, st.reject_level, st.accepted_len, st.primary_tokens, st.tree_nodes) == (2, [2, 3], [[0, 0], []], 4, [[0], []])
    # the true tuples: one round, nothing to adapt
    sp, st = O.speculative_decode(model, head, req, 2, V, drafts_round1=[(0, 0, 2), (0, 1, 1)], adaptive=True)
    assert (st.rounds, st.accepted_len, st.primary_tokens) == (1, [[3, 3]], 4)
    # four levels (T = 2 each, every tuple valid, zero heads, K = 2): B_1 = {0, 1}, B_2 = {00, 01}, B_3 = {000, 001},
    # B_4 = {0000, 0001}.  Drafted tuples 0011 and 0100: tree level 2 = {00, 01} = B_2, level 3 = {001, 010} misses 000:
    # round 1 settles levels 2 and 3 (a gain of two: keep drafting); the zero draft head continues from B_3 with the
    # true level-4 set, round 2 finishes.
    shape4 = synth.Workload("micro4", "fp32", 1, 16, 2, 1, 32, 4, (2, 2, 2, 2), 16, "uniform", 3, 2, 16, 5)
    W4 = dict(synth.weights_to_numpy(synth.make_weights(shape4, std=0.5)))
    W4["draft_logit"] = [np.zeros_like(a) for a in W4["draft_logit"]]
    W4["lm_head"] = np.zeros_like(W4["lm_head"])
    cat4 = np.asarray(list(itertools.product(range(2), repeat=4)), dtype=np.int32)
    model4, head4, V4 = oracle_bundle(shape4, W4, cat4)
    req4 = model4.prefill(synth.make_histories(shape4, None)[0])
    sp, st = O.speculative_decode(model4, head4, req4, 2, V4, drafts_round1=[(0, 0, 1, 1), (0, 1, 0, 0)], adaptive=True)
    assert [codes_of(x) for x in sp] == [[(0,), (1,)], [(0, 0), (0, 1)], [(0, 0, 0), (0, 0, 1)], [(0, 0, 0, 0), (0, 0, 0, 1)]]
    assert (st.rounds, st.reject_level, st.accepted_len) == (2, [3, 4], [[3, 2], [4, 4]])
    # one drafted tuple whose first code is a beam but whose second is not: its nodes (1,1) and (1,1,1) descend from the
    # beam (1), so both are in round 1's pass (2 + 2 tokens), which gains nothing; rounds 2 and 3 are plain steps of 2 tokens
    sp, st = O.speculative_decode(model4, head4, req4, 2, V4, drafts_round1=[(1, 1, 1, 1)], adaptive=True)
    assert (st.rounds, st.reject_level, st.primary_tokens, st.accepted_len) == (3, [2, 3, 4], 4 + 2 + 2, [[1], [], []])
    assert st.tree_nodes == [[1, 1], [0], []]
    w, W, cat, model, head, V, hist = _micro()
    rng = np.random.default_rng(9)
    req = model.prefill(hist[0])
    for trial in range(20):
        tuples = [tuple(int(rng.integers(0, t)) for t in w.T) for _ in range(3)]
        a = O.speculative_decode(model, head, req, 3, V, drafts_round1=tuples, adaptive=True)
        p = O.speculative_decode(model, head, req, 3, V, drafts_round1=tuples)
        assert [codes_of(x) for x in a[0]] == [codes_of(x) for x in p[0]]
        assert a[1].primary_tokens <= p[1].primary_tokens and a[1].rounds >= p[1].rounds


def test_tree_from_tuples_shares_prefixes():
    tree = O.tree_from_tuples([(1, 2, 3), (1, 2, 0), (1, 0, 3), (2, 2, 3), (1, 2, 3)], 3)
    assert tree == [[(1,), (2,)], [(1, 2), (1, 0), (2, 2)], [(1, 2, 3), (1, 2, 0), (1, 0, 3), (2, 2, 3)]]


def test_speculative_random_trees_keep_the_result_and_the_token_bound():
    """Whatever tree is drafted: the result is Algorithm 1's, a round's pass never exceeds |B_m| + K per further level,
    the rounds never exceed L - 1, and accepted lengths obey the prefix rule recomputed here from the true sets."""
    w, W, cat, model, head, V, hist = _micro()
    rng = np.random.default_rng(5)
    req = model.prefill(hist[1])
    K = 3
    ar = O.ar_beam_search(model, req, K, V)
    true_sets = [set(codes_of(x)) for x in ar]
    for trial in range(30):
        tuples = [tuple(int(rng.integers(0, t)) for t in w.T) for _ in range(K)]
        for i in range(K):                                 # splice in true prefixes so that every regime occurs
            cut = int(rng.integers(0, w.L + 1))
            src = codes_of(ar[-1])[int(rng.integers(0, len(ar[-1])))]
            tuples[i] = src[:cut] + tuples[i][cut:]
        sp, st = O.speculative_decode(model, head, req, K, V, drafts_round1=tuples)
        assert [codes_of(x) for x in sp] == [codes_of(x) for x in ar]
        assert 1 <= st.rounds <= w.L - 1 and st.reject_level[-1] == w.L
        assert all(n <= K for nodes in st.tree_nodes for n in nodes)
        reached = st.reject_level[0]
        uniq = []
        for t in tuples:
            if t not in uniq:
                uniq.append(t)
        want = []
        for t in uniq:
            a = 0
            while a < reached and t[: a + 1] in true_sets[a]:
                a += 1
            want.append(a)
        assert st.accepted_len[0] == want


def test_draft_head_hand_computed_numbers():
    """Eq. 2 and Eq. 3 on a two-dimensional head with numbers small enough to work by hand (a swapped W_s / W_e, a
    dropped bias or a wrong sign changes them)."""
    shape = O.ModelShape(1, 2, 1, 1, 2, 2, (2, 2))
    W = {"draft_logit": [np.array([[1.0, 0.0], [0.0, 1.0]]), np.array([[2.0, -1.0], [0.0, 3.0]])],
         "draft_ws": np.array([[0.5, 0.0], [0.0, 0.25]]), "draft_we": np.array([[1.0, 1.0], [0.0, -1.0]]),
         "draft_b": np.array([0.1, -0.1]),
         # rows: level-1 codes 0, 1; level-2 codes 0, 1; placeholders and BOS
         "embed": np.array([[9.0, 9.0], [0.2, 0.4], [7.0, 7.0], [-1.0, 0.5], [0, 0], [0, 0], [0, 0]])}
    head = O.DraftHead(shape, W)
    h1, s1 = np.array([0.5, -0.25]), np.array([1.0, 2.0])
    assert np.allclose(head.logits(0, h1, s1), [1.5, 1.75], atol=1e-15)            # identity head: z = h + s
    assert np.allclose(head.logits(1, h1, s1), [2 * 1.5 - 1.75, 3 * 1.75], atol=1e-15)
    # Eq. 3 with the level-1 code 1 (embedding (0.2, 0.4)):
    #   W_s s = (0.5, 0.5);  W_e e = (0.6, -0.4);  + b = (1.2, 0.0)  ->  s_2 = (tanh 1.2, 0)
    s2 = head.transition(0, s1, 1)
    assert np.allclose(s2, [0.8336546070121553, 0.0], atol=1e-15)
    # level-2 code 1 sits at embedding row T_1 + 1 = 3: e = (-1, 0.5); W_s s_2 = (0.41682730350607766, 0);
    #   W_e e = (-0.5, -0.5); + b = (0.01682730350607766, -0.6)
    s3 = head.transition(1, s2, 1)
    assert np.allclose(s3, [np.tanh(0.01682730350607766), np.tanh(-0.6)], atol=1e-15)
    assert abs(s3[1] + 0.5370495669980353) < 1e-15                                  # tanh(0.6), a table value


def test_draft_head_ablation_identities():
    """Section 4.3: NEZHA-1 removes the context state, so its distribution ignores the prefix; NEZHA-2 removes the hidden
    state, so it ignores h_l; the full head uses both and, being one linear layer over their sum, treats them alike."""
    w, W, cat, model, head, V, hist = _micro()
    shape = oracle_shape(w)
    req = model.prefill(hist[0])
    rng = np.random.default_rng(1)
    s_a, s_b = rng.standard_normal(w.d_model), rng.standard_normal(w.d_model)
    h1 = O.DraftHead(shape, W, use_state=False)
    h2 = O.DraftHead(shape, W, use_hidden=False)
    for l in range(w.L):
        assert np.array_equal(h1.logits(l, req.h[l + 1], s_a), h1.logits(l, req.h[l + 1], s_b))
        assert np.array_equal(h2.logits(l, s_a, req.h[0]), h2.logits(l, s_b, req.h[0]))
        assert not np.allclose(head.logits(l, req.h[l + 1], s_a), head.logits(l, req.h[l + 1], s_b))
        assert not np.allclose(head.logits(l, s_a, req.h[0]), head.logits(l, s_b, req.h[0]))
        assert np.allclose(head.logits(l, s_a, s_b), head.logits(l, s_b, s_a), atol=1e-12)
        assert np.allclose(head.logits(l, s_a, s_b), h1.logits(l, s_a, s_b) + h2.logits(l, s_a, s_b), atol=1e-12)
    # NEZHA-1's drafts do not depend on which codes were chosen before: the per-level distributions of two different
    # prefixes are the same
    assert np.array_equal(h1.logits(1, req.h[2], O.teacher_forced_state(h1, req, (0,))),
                          h1.logits(1, req.h[2], O.teacher_forced_state(h1, req, (3,))))


def test_prefix_validity_matches_python_sets():
    w = synth.WORKLOADS["tiny"]
    cat = synth.make_catalog(w)
    V = O.ValidSet(cat, w.T)
    rows = cat.tolist()
    for n in (1, 2):
        ref = {tuple(r[:n]) for r in rows}
        grid = np.stack(np.meshgrid(*[np.arange(t) for t in w.T[:n]], indexing="ij"), axis=-1).reshape(-1, n)
        got = V.contains_prefix(grid)
        assert np.array_equal(got, np.array([tuple(r) in ref for r in grid.tolist()]))
        assert got.sum() == len(ref) == V.prefix_keys(n).size
    grid3 = np.asarray(rows[:50] + [[31, 31, 31], [0, 0, 0]])
    assert np.array_equal(V.contains_prefix(grid3), V.contains(grid3))       # full length: Eq. 5 itself
    # unequal radices: the prefix of a key is the key modulo the product of the leading radices
    V2 = O.ValidSet(np.array([[2, 4, 6], [1, 0, 3]]), (3, 5, 7))
    assert V2.prefix_keys(2).tolist() == sorted([2 + 4 * 3, 1 + 0 * 3])
    assert V2.contains_prefix(np.array([[2, 4], [1, 0], [2, 0], [1, 4]])).tolist() == [True, True, False, False]


def test_validity_at_every_level():
    """The per-step variant of the verification (Section 3.4): with the filter at every level every surviving beam of
    every level is the beginning of a valid ID; without pruning (K >= the number of prefixes) the result is unchanged;
    with pruning a search that wastes no beam on dead prefixes returns at least as many items."""
    w, W, cat, model, head, V, hist = _micro()
    valid = [tuple(r) for r in cat.tolist()]
    for b in range(hist.shape[0]):
        req = model.prefill(hist[b])
        for K in (1, 2, 3, 5, 16):
            for search in (lambda **kw: O.ar_beam_search(model, req, K, V, **kw),
                           lambda **kw: O.nezha_draft(head, req, K, V, **kw),
                           lambda **kw: O.speculative_decode(model, head, req, K, V, **kw)[0]):
                on, off = search(every_level=True), search()
                for n, level in enumerate(on):
                    assert all(any(v[: n + 1] == bm.codes for v in valid) for bm in level)
                assert len(on[-1]) >= len(off[-1])
                if K == 16:                                        # nothing is pruned before the last level
                    assert codes_of(on[-1]) == codes_of(off[-1])
                    assert np.array_equal(scores_of(on[-1]), scores_of(off[-1]))
            # Algorithm 2 still returns Algorithm 1's result under the same filter
            assert codes_of(O.speculative_decode(model, head, req, K, V, every_level=True)[0][-1]) == \
                codes_of(O.ar_beam_search(model, req, K, V, every_level=True)[-1])
    # hand-worked, zero heads, K = 2: valid IDs (1,2,0), (1,3,1), (2,0,0).  Level 1: codes 0..3 tie, 0 and 3 begin no
    # valid ID -> B_1 = {(1),(2)}.  Level 2: (1,2),(1,3),(2,0) are the live prefixes; ties go to the smaller parent rank
    # -> B_2 = {(1,2),(1,3)}.  Level 3 -> {(1,2,0),(1,3,1)}.  Without the per-level filter B_1 = {(0),(1)} and
    # B_2 = {(0,0),(0,1)}, which no valid ID continues: nothing is returned.
    model, head, V, req = _zero_head_case([(1, 2, 0), (1, 3, 1), (2, 0, 0)])
    on = O.ar_beam_search(model, req, 2, V, every_level=True)
    assert [codes_of(x) for x in on] == [[(1,), (2,)], [(1, 2), (1, 3)], [(1, 2, 0), (1, 3, 1)]]
    assert O.ar_beam_search(model, req, 2, V)[-1] == []
    # the draft head takes its top-2 codes per beam BEFORE the filter (Algorithm 3's order): at level 1 codes 0 and 1,
    # of which only (1) is live; then (1,0),(1,1) -- both dead: no draft survives
    d = O.nezha_draft(head, req, 2, V, every_level=True)
    assert [codes_of(x) for x in d] == [[(1,)], [], []]


# ---------------------------------------------------------------------------------------- ablation variants (Section 4.3)
def test_ablation_variants_of_the_draft_head():
    """NEZHA-1 (no context state): every level's distribution ignores the prefix, so the joint log-probability is a sum
    of per-level terms and the beam search equals the brute-force top-K of that sum over the valid tuples.
    NEZHA-2 (no hidden state): the logits are W s_l, i.e. the default head's on a request whose h_1..h_L are zero.
    NEZHA-3 (additive transition): s_{l+1} = s_l + e_l, written out here from the weights."""
    w, W, cat, model, head, V, hist = _micro()
    shape = oracle_shape(w)
    req = model.prefill(hist[1])
    f = lambda n: np.asarray(W[n], dtype=np.float64)
    # NEZHA-1
    h1 = O.DraftHead(shape, W, use_state=False)
    per_level = [torch.log_softmax(torch.from_numpy(np.asarray(W["draft_logit"][l], dtype=np.float64) @ req.h[l + 1]), -1).numpy()
                 for l in range(w.L)]
    brute = sorted(((sum(per_level[l][t[l]] for l in range(w.L)), t) for t in _all_tuples(w.T) if V.contains(np.asarray([t]))[0]),
                   key=lambda x: (-x[0], x[1]))
    got = O.nezha_draft(h1, req, w.beam, V)[-1]
    assert codes_of(got) == [t for _, t in brute[: len(got)]] and len(got) == min(w.beam, len(brute))
    assert np.allclose(scores_of(got), [s for s, _ in brute[: len(got)]], atol=1e-5)
    # NEZHA-2
    h2 = O.DraftHead(shape, W, use_hidden=False)
    req0 = O.Request(P=req.P, h=np.concatenate([req.h[:1], np.zeros_like(req.h[1:])]), ctx_kv=req.ctx_kv)
    assert codes_of(O.nezha_draft(h2, req, w.beam, V)[-1]) == codes_of(O.nezha_draft(head, req0, w.beam, V)[-1])
    assert np.array_equal(h2.logits(1, req.h[2], req.h[0]), np.asarray(W["draft_logit"][1], dtype=np.float64) @ req.h[0])
    assert codes_of(O.nezha_draft(h2, req, w.beam, V)[-1]) != codes_of(O.nezha_draft(head, req, w.beam, V)[-1])
    # NEZHA-3
    h3 = O.DraftHead(shape, W, additive_transition=True)
    s2 = h3.transition(0, req.h[0], 3)
    assert np.array_equal(s2, req.h[0] + f("embed")[3])
    assert np.array_equal(h3.transition(1, s2, 1), req.h[0] + f("embed")[3] + f("embed")[w.T[0] + 1])
    lp = O.joint_logprob_draft(h3, req, (3, 1, 2))
    zs = [np.asarray(W["draft_logit"][0], dtype=np.float64) @ (req.h[1] + req.h[0]),
          np.asarray(W["draft_logit"][1], dtype=np.float64) @ (req.h[2] + s2),
          np.asarray(W["draft_logit"][2], dtype=np.float64) @ (req.h[3] + s2 + f("embed")[w.T[0] + 1])]
    want = sum(float(torch.log_softmax(torch.from_numpy(z), -1)[c]) for z, c in zip(zs, (3, 1, 2)))
    assert abs(lp - want) < 1e-12
