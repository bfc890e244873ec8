"""GPU parity tests: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import nezha_oracle as O
from paper_2511_18793_b200 import synth
from helpers import codes_of
from gpu_helpers import Case, assert_topk_matches, check_levels, check_walk_against_trace, tolerance, wide_tolerance

pytestmark = pytest.mark.gpu


def _as_u64(t):
    return t.cpu().numpy().view(np.uint64)


@pytest.fixture(scope="module")
def tiny():
    return Case(synth.WORKLOADS["tiny"]).prefill()


# ---------------------------------------------------------------------------------------- hash set
@pytest.mark.parametrize("name,n_items", [("tiny", None), ("small", 200_000)])
def test_hashset_build_and_probe_bit_exact(name, n_items):
    w = synth.WORKLOADS[name]
    if n_items:
        w = synth.scaled(w, n_items=n_items, n_layers=1, batch=2, n_hist=2)
    cat = synth.make_catalog(w)
    cat_dup = np.concatenate([cat, cat[: len(cat) // 10]])            # duplicated tuples are counted once
    case = Case(w, catalog=cat_dup)
    V = O.ValidSet(cat, w.T)
    assert case.n_unique == len(V) == len(cat)
    dev = case.dev
    # Eq. 4: keys bit-identical
    probe_codes = synth.probe_keys_mix(w, cat, 100_000)
    keys = case.eng.pack(torch.from_numpy(probe_codes).to(dev))
    assert np.array_equal(_as_u64(keys), O.pack_keys(probe_codes, w.T))
    # Eq. 5: (i) every catalogue key, (ii) a hit/miss mix, (iii) siblings of catalogue prefixes
    found = case.eng.probe(case.eng.pack(torch.from_numpy(cat).to(dev)))
    assert bool(found.all())
    found = case.eng.probe(keys).cpu().numpy().astype(bool)
    assert np.array_equal(found, V.contains(probe_codes))
    pre = cat[np.random.default_rng(0).integers(0, len(cat), 500)]
    sib = np.repeat(pre, w.T[-1], axis=0)
    sib[:, -1] = np.tile(np.arange(w.T[-1]), len(pre))
    found = case.eng.probe(case.eng.pack(torch.from_numpy(sib.astype(np.int32)).to(dev))).cpu().numpy().astype(bool)
    assert np.array_equal(found, V.contains(sib))
    assert found.sum() >= len(pre)
    # empty probe is a no-op
    assert case.eng.probe(torch.empty(0, dtype=torch.int64, device=dev)).numel() == 0


def test_error_paths(tiny):
    b = tiny.binding
    w = tiny.w
    # out-of-range catalogue code
    bad = tiny.catalog.copy(); bad[7, 1] = w.T[1]
    c2 = None
    with pytest.raises(b.NezhaError) as ei:
        c2 = Case(w, catalog=bad)
    assert ei.value.status == 6
    # decode before prefill, wrong batch, beam too wide
    c3 = Case(w)
    with pytest.raises(b.NezhaError) as ei:
        c3.eng.batch = w.batch
        c3.eng.decode(w.beam)
    assert ei.value.status == 2
    with pytest.raises(b.NezhaError) as ei:
        tiny.eng.decode(w.beam + 1)
    assert ei.value.status == 1
    # arena too small
    import ctypes as C
    cfg = b.make_config(w)
    h = C.c_void_p()
    wts = b.NezhaWeights()
    arena = torch.empty(1024, dtype=torch.uint8, device="cuda")
    st = b.lib.nezha_create(C.byref(cfg), C.byref(wts), tiny.cat_dev.data_ptr(), 5000, 0.5, arena.data_ptr(), 1024, None,
                            C.byref(h))
    assert st == 3
    # a history code out of range is reported by the next synchronising call
    hist = tiny.hist.copy(); hist[0, 0, 0] = 99
    c3.eng.prefill(torch.from_numpy(hist).cuda(), c3.n_hist)
    with pytest.raises(b.NezhaError) as ei:
        c3.eng.sync()
    assert ei.value.status == 6


def test_invalid_drafts_are_dropped_and_reported(tiny):
    """Drafted tuples / tree nodes with a code outside [0, T_l) are no semantic IDs: the call reports NEZHA_ERR_CATALOG, the
    tuple (node) takes no part, the items are Algorithm 1's all the same, and the next call is clean."""
    b = tiny.binding
    w = tiny.w
    K = w.beam
    ar = tiny.eng.decode(K, mode=2, trace=True)
    drafts = ar["codes"].clone().clamp_(min=0)
    drafts[:, 0, 1] = w.T[1]                                     # one bad tuple per request
    out = tiny.eng.alloc_outputs(w.batch, K, trace=True)
    with pytest.raises(b.NezhaError) as ei:
        tiny.eng.decode_with_drafts(K, drafts, ar["count"].clone(), out=out)
    assert ei.value.status == 6
    assert torch.equal(out["codes"], ar["codes"]) and torch.equal(out["count"], ar["count"])
    n_draft = out["trace"]["n_draft"][0].cpu().numpy()
    assert np.array_equal(n_draft, np.maximum(ar["count"].cpu().numpy() - 1, 0))     # the bad tuple is not in the tree
    beams = ar["trace"]["beams"].clone()
    counts = (beams[:, :, :, 0] >= 0).sum(dim=2).to(torch.int32)
    beams[1, :, 0, 0] = -5                                       # a bad node at level 2: it and its subtree are dead
    with pytest.raises(b.NezhaError) as ei:
        tiny.eng.decode_with_draft_tree(K, beams, counts, out=out)
    assert ei.value.status == 6
    assert torch.equal(out["codes"], ar["codes"])
    check_walk_against_trace(tiny.eng.decode(K, mode=1, trace=True), w.batch, w.L)     # and the next call is clean
    with pytest.raises(b.NezhaError) as ei:                       # null tree
        b.lib.nezha_decode_with_draft_tree.argtypes
        tiny.eng._check(b.lib.nezha_decode_with_draft_tree(tiny.eng._h, w.batch, K, None, None, out["codes"].data_ptr(),
                                                            out["scores"].data_ptr(), out["count"].data_ptr(), None, None))
    assert ei.value.status == 1


# ---------------------------------------------------------------------------------------- stage-wise FP parity
def test_prefill_hidden_states(tiny):
    h = tiny.eng.get_hidden().cpu().numpy()
    for b in range(tiny.w.batch):
        assert np.abs(h[b] - tiny.req(b).h).max() < 2e-5


def test_primary_logits_teacher_forced(tiny):
    w = tiny.w
    model = tiny.oracle[0]
    rng = np.random.default_rng(3)
    for level in range(w.L):
        nb = w.beam
        pre = np.stack([rng.integers(0, w.T[l], size=(w.batch, nb)) for l in range(level)], axis=2).astype(np.int32) \
            if level else None
        got = tiny.eng.primary_logits(nb, level, None if pre is None else torch.from_numpy(pre).cuda()).cpu().numpy()
        for b in range(w.batch):
            ref = model.next_level_logits_many(tiny.req(b), [tuple(pre[b, r]) if level else () for r in range(nb)])
            assert np.abs(got[b] - np.stack(ref)).max() < tolerance(w)


def test_draft_logits_teacher_forced(tiny):
    w = tiny.w
    head = tiny.oracle[1]
    rng = np.random.default_rng(4)
    for level in range(w.L):
        nb = w.beam
        pre = np.stack([rng.integers(0, w.T[l], size=(w.batch, nb)) for l in range(level)], axis=2).astype(np.int32) \
            if level else None
        got = tiny.eng.draft_logits(nb, level, None if pre is None else torch.from_numpy(pre).cuda()).cpu().numpy()
        for b in range(w.batch):
            req = tiny.req(b)
            for r in range(nb):
                st = O.teacher_forced_state(head, req, tuple(pre[b, r]) if level else ())
                ref = head.logits(level, req.h[level + 1], st)
                assert np.abs(got[b, r] - ref).max() < tolerance(w)


# ---------------------------------------------------------------------------------------- select (integer stage)
@pytest.mark.parametrize("level,per_beam_all,filt", [(0, True, False), (1, True, False), (2, True, True), (2, False, True),
                                                     (1, False, False)])
def test_select_on_identical_logits(tiny, level, per_beam_all, filt):
    w = tiny.w
    V = tiny.oracle[2]
    rng = np.random.default_rng(10 + level)
    K = w.beam
    nb = 1 if level == 0 else K
    logits = rng.standard_normal((w.batch, nb, w.T[level])).astype(np.float32) * 2
    scores = (-rng.random((w.batch, nb)) * 3).astype(np.float32)
    if level == 2:                                   # prefixes that have valid completions
        idx = rng.integers(0, len(tiny.catalog), size=(w.batch, nb))
        codes = tiny.catalog[idx][:, :, :level].astype(np.int32)
    else:
        codes = np.stack([rng.integers(0, w.T[l], size=(w.batch, nb)) for l in range(level)], axis=2).astype(np.int32) \
            if level else None
    n_live = np.full((w.batch,), nb, dtype=np.int32); n_live[-1] = max(1, nb - 2)
    per_beam = w.T[level] if per_beam_all else min(K, w.T[level])
    parent, code, score, count = tiny.eng.select(
        torch.from_numpy(logits).cuda(), torch.from_numpy(scores).cuda(),
        None if codes is None else torch.from_numpy(codes).cuda(), torch.from_numpy(n_live).cuda(), K, level, per_beam, filt)
    parent, code, score, count = [t.cpu().numpy() for t in (parent, code, score, count)]
    for b in range(w.batch):
        beams = [O.Beam(tuple(codes[b, r]) if level else (), np.float32(scores[b, r])) for r in range(n_live[b])]
        ref = O.expand_level(beams, [logits[b, r].astype(np.float64) for r in range(n_live[b])], K, per_beam,
                             V if filt else None)
        assert count[b] == len(ref)
        got = [(int(parent[b, k]), int(code[b, k])) for k in range(count[b])]
        want = [(bm.parent, bm.codes[-1]) for bm in ref]
        if got != want:       # only near-ties (fp32 vs fp64 log-softmax) may differ
            gs, ws = score[b, : count[b]], np.asarray([float(x.score) for x in ref])
            assert np.abs(np.sort(gs) - np.sort(ws)).max() < 1e-5
            assert len(set(got) ^ set(want)) <= 2
        else:
            assert np.allclose(score[b, : count[b]], [float(x.score) for x in ref], atol=2e-6)
        assert np.all(parent[b, count[b]:] == -1) and np.all(np.isneginf(score[b, count[b]:]))


# ---------------------------------------------------------------------------------------- end to end, tiny (fp32)
def test_mode_draft_equals_algorithm3(tiny):
    w = tiny.w
    head, V = tiny.oracle[1], tiny.oracle[2]
    out = tiny.eng.decode(w.beam, mode=0)
    codes, scores, count = [out[k].cpu().numpy() for k in ("codes", "scores", "count")]
    for b in range(w.batch):
        ref = O.nezha_draft(head, tiny.req(b), w.beam, V)[-1]
        assert assert_topk_matches(codes[b], scores[b], count[b], ref, w.beam, tolerance(w))
        assert V.contains(codes[b, : count[b]]).all()                      # zero hallucinations


def test_mode_ar_equals_algorithm1(tiny):
    w = tiny.w
    model, _, V = tiny.oracle
    out = tiny.eng.decode(w.beam, mode=2, trace=True)
    codes, scores, count = [out[k].cpu().numpy() for k in ("codes", "scores", "count")]
    beams = out["trace"]["beams"].cpu().numpy()
    assert out["stats"].rounds == w.L - 1
    for b in range(w.batch):
        ref = O.ar_beam_search(model, tiny.req(b), w.beam, V)
        assert assert_topk_matches(codes[b], scores[b], count[b], ref[-1], w.beam, tolerance(w))
        for n in range(w.L):                                                # every intermediate beam set too
            got = [tuple(int(c) for c in beams[n, b, k, : n + 1]) for k in range(len(ref[n]))]
            assert got == codes_of(ref[n])
        assert V.contains(codes[b, : count[b]]).all()


def test_mode_verified_equals_ar_and_matches_oracle_trace(tiny):
    w = tiny.w
    model, head, V = tiny.oracle
    out = tiny.eng.decode(w.beam, mode=1, trace=True)
    ar = tiny.eng.decode(w.beam, mode=2)
    assert torch.equal(out["codes"], ar["codes"]) and torch.equal(out["count"], ar["count"])      # zero sacrifice
    assert torch.allclose(out["scores"], ar["scores"], atol=1e-5)
    codes, scores, count = [out[k].cpu().numpy() for k in ("codes", "scores", "count")]
    tr = {k: v.cpu().numpy() for k, v in out["trace"].items()}
    tot_tokens, max_rounds = 0, 0
    for b in range(w.batch):
        sets, st = O.speculative_decode(model, head, tiny.req(b), w.beam, V)
        assert assert_topk_matches(codes[b], scores[b], count[b], sets[-1], w.beam, tolerance(w))
        for r in range(st.rounds):
            nd = tr["n_draft"][r, b]
            assert list(tr["accepted_len"][r, b, :nd]) == st.accepted_len[r]
            assert tr["level_reached"][r, b] == st.reject_level[r]
            want_tree = [len(x) for x in O.nezha_draft(head, tiny.req(b), w.beam, V)] if r == 0 else None
            if want_tree is not None:
                assert list(tr["tree_count"][0, :, b]) == want_tree
        assert np.all(tr["level_reached"][st.rounds:, b] == -1)
        tot_tokens += st.primary_tokens
        max_rounds = max(max_rounds, st.rounds)
    assert out["stats"].primary_tokens == tot_tokens and out["stats"].rounds == max_rounds
    assert check_walk_against_trace(out, w.batch, w.L) == (tot_tokens, max_rounds)


def test_decode_with_drafts_acceptance_regimes(tiny):
    w = tiny.w
    model, head, V = tiny.oracle
    K = w.beam
    ar = tiny.eng.decode(K, mode=2)
    ar_codes = ar["codes"].cpu().numpy()
    rng = np.random.default_rng(5)
    for rho in (0.0, 0.5, 1.0):
        drafts = ar_codes.copy()
        n_draft = ar["count"].cpu().numpy().copy()
        for b in range(w.batch):
            for k in range(n_draft[b]):
                if rng.random() < rho:
                    lvl = int(rng.integers(0, w.L))
                    drafts[b, k, lvl] = (drafts[b, k, lvl] + 1 + rng.integers(0, w.T[lvl] - 1)) % w.T[lvl]
        out = tiny.eng.decode_with_drafts(K, torch.from_numpy(drafts).cuda(), torch.from_numpy(n_draft).cuda(), trace=True)
        assert torch.equal(out["codes"], ar["codes"])                        # result never depends on the drafts
        tr = {k: v.cpu().numpy() for k, v in out["trace"].items()}
        tot = 0
        for b in range(w.batch):
            D = [tuple(int(c) for c in drafts[b, k]) for k in range(n_draft[b])]
            sets, st = O.speculative_decode(model, head, tiny.req(b), K, V, drafts_round1=D)
            assert codes_of(sets[-1]) == [tuple(int(c) for c in ar_codes[b, k]) for k in range(len(sets[-1]))]
            n = len(st.accepted_len[0])                                      # distinct tuples
            assert tr["n_draft"][0, b] == n
            assert list(tr["accepted_len"][0, b, :n]) == st.accepted_len[0]
            assert tr["level_reached"][0, b] == st.reject_level[0]
            assert list(tr["tree_count"][0, :, b]) == [len(x) for x in O.tree_from_tuples(D, w.L)]
            if rho == 0.0:                                                   # true tuples: accepted as far as the round got
                assert st.accepted_len[0] == [st.reject_level[0]] * n
            tot += st.primary_tokens
        assert out["stats"].primary_tokens == tot
        check_walk_against_trace(out, w.batch, w.L)
    # the true beam sets of every level as the draft tree: one round, everything accepted, no token beyond plain decoding's
    art = tiny.eng.decode(K, mode=2, trace=True)
    beams = art["trace"]["beams"]
    counts = (beams[:, :, :, 0] >= 0).sum(dim=2).to(torch.int32)
    out = tiny.eng.decode_with_draft_tree(K, beams, counts, trace=True)
    assert torch.equal(out["codes"], ar["codes"]) and torch.allclose(out["scores"], art["scores"], atol=1e-5)
    assert out["stats"].rounds == 1
    assert out["stats"].primary_tokens == int(counts[: w.L - 1].sum())
    tr = {k: v.cpu().numpy() for k, v in out["trace"].items()}
    for b in range(w.batch):
        n = int(counts[w.L - 1, b])
        assert list(tr["accepted_len"][0, b, :n]) == [w.L] * n and tr["level_reached"][0, b] == w.L
    check_walk_against_trace(out, w.batch, w.L)
    # repeated tuples and tuples with shared prefixes: one node per distinct prefix
    dup = ar_codes.copy()
    dup[:, 1] = dup[:, 0]
    nd = torch.full((w.batch,), K, dtype=torch.int32, device="cuda")
    out = tiny.eng.decode_with_drafts(K, torch.from_numpy(dup).cuda(), nd, trace=True)
    assert torch.equal(out["codes"], ar["codes"])
    tr = {k: v.cpu().numpy() for k, v in out["trace"].items()}
    for b in range(w.batch):
        D = [tuple(int(c) for c in dup[b, k]) for k in range(K)]
        assert list(tr["tree_count"][0, :, b]) == [len(x) for x in O.tree_from_tuples(D, w.L)]
        got = [tuple(int(c) for c in tr["drafts"][0, b, k]) for k in range(tr["n_draft"][0, b])]
        assert got == O.tree_from_tuples(D, w.L)[-1]
    check_walk_against_trace(out, w.batch, w.L)
    # decode is repeatable from the same prefilled state
    again = tiny.eng.decode(K, mode=1)
    assert torch.equal(again["codes"], ar["codes"])


def test_ragged_histories_and_small_beams():
    w = synth.scaled(synth.WORKLOADS["tiny"], n_kv_heads=2, batch=3)
    case = Case(w)
    n_hist = torch.tensor([w.n_hist, 7, 0], dtype=torch.int32, device="cuda")
    case.eng.prefill(case.hist_dev, n_hist)
    model, head, V = case.oracle
    for K in (1, 3):
        out = case.eng.decode(K, mode=1)
        codes, scores, count = [out[k].cpu().numpy() for k in ("codes", "scores", "count")]
        for b, n in enumerate([w.n_hist, 7, 0]):
            ref = O.ar_beam_search(model, case.req(b, n), K, V)[-1]
            assert assert_topk_matches(codes[b], scores[b], count[b], ref, K, tolerance(w))


# ---------------------------------------------------------------------------------------- ablation variants (Section 4.3)
VARIANTS = {                       # name -> (options to set, oracle head arguments, hash filter on)
    "nezha1_no_state": ({1: 1}, dict(use_state=False), True),
    "nezha2_no_hidden": ({1: 2}, dict(use_hidden=False), True),
    "nezha3_additive": ({0: 1}, dict(additive_transition=True), True),
    "nezha4_no_filter": ({2: 0}, dict(), False),
}


@pytest.mark.parametrize("variant", sorted(VARIANTS))
@pytest.mark.parametrize("name", ["tiny", "small_cut"])
def test_draft_head_variants(name, variant):
    """nezha_set_option against the oracle's draft head with the same switch: teacher-forced logits, mode 0 output, and
    mode 1 still equal to mode 2 (the variants never touch the primary model)."""
    w = synth.WORKLOADS["tiny"] if name == "tiny" else \
        synth.scaled(synth.WORKLOADS["small"], n_layers=2, n_items=100_000, batch=4, n_hist=20)
    case = Case(w).prefill()
    opts, head_kw, filt = VARIANTS[variant]
    for k, v in opts.items():
        case.eng.set_option(k, v)
    model, _, V = case.oracle
    from helpers import oracle_shape
    head = O.DraftHead(oracle_shape(w), synth.weights_to_numpy(case.weights), **head_kw)
    rng = np.random.default_rng(3)
    tol = tolerance(w)
    for level in range(w.L):
        pre = np.stack([rng.integers(0, w.T[l], size=(w.batch, w.beam)) for l in range(level)], axis=2).astype(np.int32) \
            if level else None
        got = case.eng.draft_logits(w.beam, level, None if pre is None else torch.from_numpy(pre).cuda()).cpu().numpy()
        for b in range(w.batch):
            for r in range(w.beam):
                st = O.teacher_forced_state(head, case.req(b), tuple(pre[b, r]) if level else ())
                assert np.abs(got[b, r] - head.logits(level, case.req(b).h[level + 1], st)).max() < tol
    out = case.eng.decode(w.beam, mode=0)
    codes, scores, count = (out[k].cpu().numpy() for k in ("codes", "scores", "count"))
    for b in range(w.batch):
        ref = O.nezha_draft(head, case.req(b), w.beam, V if filt else None)[-1]
        assert_topk_matches(codes[b], scores[b], count[b], ref, w.beam, tol)
    if not filt:
        live = np.arange(w.beam)[None, :] < count[:, None]
        assert not V.contains(codes[live]).all() or w.name == "tiny"     # without Eq. 5 hallucinated tuples get through
    m1, m2 = case.eng.decode(w.beam, mode=1), case.eng.decode(w.beam, mode=2)
    assert torch.equal(m1["codes"], m2["codes"]) and torch.equal(m1["count"], m2["count"])
    with pytest.raises(case.binding.NezhaError):
        case.eng.set_option(7, 0)
    with pytest.raises(case.binding.NezhaError):
        case.eng.set_option(1, 3)


# ---------------------------------------------------------------------------------------- the library's size limits
def test_maximum_beam_and_codebook_sizes():
    """Beam 128 over codebooks of 1024 codes (both the largest the library takes): every mode against the oracle."""
    w = synth.scaled(synth.WORKLOADS["tiny"], L=2, T=(1024, 1024), n_items=30_000, batch=2, beam=128, n_hist=6)
    case = Case(w).prefill()
    model, head, V = case.oracle
    tol = tolerance(w)
    ar = case.eng.decode(w.beam, mode=2)
    sp = case.eng.decode(w.beam, mode=1)
    dr = case.eng.decode(w.beam, mode=0)
    assert torch.equal(ar["codes"], sp["codes"]) and torch.equal(ar["count"], sp["count"])
    for b in range(w.batch):
        ref = O.ar_beam_search(model, case.req(b), w.beam, V)[-1]
        assert_topk_matches(*(ar[k][b].cpu().numpy() for k in ("codes", "scores", "count")), ref, w.beam, tol)
        ref = O.nezha_draft(head, case.req(b), w.beam, V)[-1]
        assert_topk_matches(*(dr[k][b].cpu().numpy() for k in ("codes", "scores", "count")), ref, w.beam, tol)
    assert int(ar["count"].min()) == w.beam                        # 30 000 items: every request fills its beam


def test_maximum_number_of_levels():
    """L = 8 codes per item (NEZHA_MAX_LEVELS) over codebooks of 4: seven verification levels, Eq. 4 with eight digits."""
    w = synth.scaled(synth.WORKLOADS["tiny"], L=8, T=(4,) * 8, n_items=9_000, batch=3, beam=6, n_hist=5)
    case = Case(w).prefill()
    model, head, V = case.oracle
    probe = synth.probe_keys_mix(w, case.catalog, 20_000)
    keys = case.eng.pack(torch.from_numpy(probe).cuda())
    assert np.array_equal(keys.cpu().numpy().view(np.uint64), O.pack_keys(probe, w.T))
    assert np.array_equal(case.eng.probe(keys).cpu().numpy().astype(bool), V.contains(probe))
    ar = case.eng.decode(w.beam, mode=2)
    sp = case.eng.decode(w.beam, mode=1, trace=True)
    dr = case.eng.decode(w.beam, mode=0)
    assert torch.equal(ar["codes"], sp["codes"]) and torch.equal(ar["count"], sp["count"])
    assert 1 <= sp["stats"].rounds <= w.L - 1
    beams, scores = sp["trace"]["beams"].cpu().numpy(), sp["trace"]["beam_scores"].cpu().numpy()
    for b in range(w.batch):
        check_levels(case, b, beams[:, b], scores[:, b], w.beam)
        ref = O.ar_beam_search(model, case.req(b), w.beam, V)[-1]
        assert_topk_matches(*(ar[k][b].cpu().numpy() for k in ("codes", "scores", "count")), ref, w.beam, tolerance(w))
        ref = O.nezha_draft(head, case.req(b), w.beam, V)[-1]
        assert_topk_matches(*(dr[k][b].cpu().numpy() for k in ("codes", "scores", "count")), ref, w.beam, tolerance(w))


def test_one_item_catalogue_and_beam_wider_than_it():
    """A catalogue of one item under a beam that keeps every prefix (64 beams over 8 x 8 x 8 codes): every mode returns
    that item alone (count 1, the other beam slots -1).  Under a narrow beam the item's prefix may be pruned before the
    last level, where alone validity is checked, so the result may be empty: it must equal the oracle's.  A single level
    L = 1 has no prefix to verify at all."""
    catalog = np.array([[3, 1, 4]], dtype=np.int32)
    for beam in (64, 3):
        w = synth.scaled(synth.WORKLOADS["tiny"], T=(8, 8, 8), n_items=1, batch=2, beam=beam)
        hist = np.tile(catalog[None], (w.batch, 5, 1)).astype(np.int32)
        case = Case(w, catalog=catalog, hist=hist).prefill()
        model, head, V = case.oracle
        assert case.n_unique == 1
        for mode in (0, 1, 2):
            out = case.eng.decode(w.beam, mode=mode)
            codes, count = out["codes"].cpu().numpy(), out["count"].cpu().numpy()
            for b in range(w.batch):
                ref = (O.nezha_draft(head, case.req(b), beam, V) if mode == 0 else O.ar_beam_search(model, case.req(b), beam, V))[-1]
                assert count[b] == len(ref) and (beam == 3 or count[b] == 1)
                assert np.all(codes[b, : count[b]] == catalog[0]) and np.all(codes[b, count[b]:] == -1)
    w1 = synth.scaled(synth.WORKLOADS["tiny"], L=1, T=(32,), n_items=20, batch=2, beam=5)
    c1 = Case(w1).prefill()
    model, head, V = c1.oracle
    for mode in (0, 1, 2):
        out = c1.eng.decode(w1.beam, mode=mode)
        for b in range(w1.batch):
            ref = (O.nezha_draft(head, c1.req(b), w1.beam, V) if mode == 0 else O.ar_beam_search(model, c1.req(b), w1.beam, V))[-1]
            assert_topk_matches(*(out[k][b].cpu().numpy() for k in ("codes", "scores", "count")), ref, w1.beam, tolerance(w1))


# ---------------------------------------------------------------------------------------- the last-level mask from the prefix map
@pytest.mark.parametrize("name", ["tiny", "small_cut", "t512", "t1024", "one_level"])
def test_final_mask_from_prefix_map_equals_hash_probes(name):
    """NEZHA_OPT_FINAL_MASK = 1 (the default) answers Eq. 5 from the (prefix -> bit set of last codes) table instead of the hash set:
    every mode must return the same bits as with the hash probes, whatever the codebook size (1, 2, 8 or 16 words of bits)."""
    w = {"tiny": synth.WORKLOADS["tiny"],
         "small_cut": synth.scaled(synth.WORKLOADS["small"], n_layers=2, n_items=100_000, batch=4, n_hist=20),
         "t512": synth.scaled(synth.WORKLOADS["paper"], n_layers=1, batch=3),
         "t1024": synth.scaled(synth.WORKLOADS["tiny"], L=2, T=(1024, 1024), n_items=30_000, batch=2, beam=16, n_hist=6),
         "one_level": synth.scaled(synth.WORKLOADS["tiny"], L=1, T=(32,), n_items=20, batch=2, beam=5)}[name]
    case = Case(w).prefill()
    case.eng.set_option(3, 0)
    base = {m: case.eng.decode(w.beam, mode=m) for m in (0, 1, 2)}
    case.eng.set_option(3, 1)
    for m in (0, 1, 2):
        got = case.eng.decode(w.beam, mode=m)
        for k in ("codes", "scores", "count"):
            assert torch.equal(got[k], base[m][k]), (name, m, k)
    V = case.oracle[2]
    codes, count = base[1]["codes"].cpu().numpy(), base[1]["count"].cpu().numpy()
    live = np.arange(w.beam)[None, :] < count[:, None]
    assert V.contains(codes[live]).all()
    case.eng.set_option(3, 0)
    again = case.eng.decode(w.beam, mode=1)
    assert torch.equal(again["codes"], base[1]["codes"])


# ---------------------------------------------------------------------------------------- validity at every level
@pytest.mark.parametrize("name", ["tiny", "small_cut", "t512", "sparse"])
def test_validity_filter_at_every_level(name):
    """NEZHA_OPT_LEVEL_FILTER = 1: a partial ID survives a level only if some valid ID begins with it.  Every mode against
    the oracle with the same switch; every beam of every level is the beginning of a catalogue item; modes 1 and 2 agree;
    and a search that wastes no beam on dead prefixes returns at least as many items as the default."""
    w = {"tiny": synth.WORKLOADS["tiny"],
         "small_cut": synth.scaled(synth.WORKLOADS["small"], n_layers=2, n_items=100_000, batch=4, n_hist=20),
         "t512": synth.scaled(synth.WORKLOADS["paper"], n_layers=1, batch=3),
         # a catalogue so thin that most first codes begin no item
         "sparse": synth.scaled(synth.WORKLOADS["tiny"], n_items=12, batch=3, beam=6)}[name]
    case = Case(w).prefill()
    model, head, V = case.oracle
    base = {m: case.eng.decode(w.beam, mode=m) for m in (0, 1, 2)}
    case.eng.set_option(4, 1)
    out = case.eng.decode(w.beam, mode=1, trace=True)
    ar = case.eng.decode(w.beam, mode=2)
    dr = case.eng.decode(w.beam, mode=0)
    assert torch.equal(out["codes"], ar["codes"]) and torch.equal(out["count"], ar["count"])
    beams, scores = out["trace"]["beams"].cpu().numpy(), out["trace"]["beam_scores"].cpu().numpy()
    dcodes, dscores, dcount = (dr[k].cpu().numpy() for k in ("codes", "scores", "count"))
    for b in range(w.batch):
        check_levels(case, b, beams[:, b], scores[:, b], w.beam, every_level=True,
                     tol=wide_tolerance(w) if name == "t512" else None)      # d = 2048: see wide_tolerance
        for n in range(w.L):
            cnt = int((beams[n, b, :, 0] >= 0).sum())
            assert V.contains_prefix(beams[n, b, :cnt, : n + 1]).all()
        ref = O.nezha_draft(head, case.req(b), w.beam, V, every_level=True)[-1]
        assert_topk_matches(dcodes[b], dscores[b], dcount[b], ref, w.beam, tolerance(w))
    check_walk_against_trace(out, w.batch, w.L)
    for m, got in ((0, dr), (1, out), (2, ar)):
        assert bool((got["count"] >= base[m]["count"]).all()), (name, m)
    print(f"{name}: requests with fewer than K items, last-level filter only -> every level: "
          f"{int((base[2]['count'] < w.beam).sum())} -> {int((ar['count'] < w.beam).sum())} of {w.batch} (primary), "
          f"{int((base[0]['count'] < w.beam).sum())} -> {int((dr['count'] < w.beam).sum())} (draft head)")
    case.eng.set_option(4, 0)
    again = case.eng.decode(w.beam, mode=1)
    assert torch.equal(again["codes"], base[1]["codes"])


@pytest.mark.parametrize("name", ["tiny", "small_cut"])
def test_adaptive_drafting(name):
    """NEZHA_OPT_ADAPTIVE_DRAFT = 1: a request stops drafting after a round that gained nothing.  Same items as without it
    and as plain decoding; rounds, tokens and accepted lengths as the oracle's with the same policy (tiny: natural drafts
    and seeded corrupted drafts); never more tokens than without it; the walk replayed from the trace."""
    w = {"tiny": synth.WORKLOADS["tiny"],
         "small_cut": synth.scaled(synth.WORKLOADS["small"], n_layers=2, n_items=100_000, batch=6, n_hist=20)}[name]
    case = Case(w).prefill()
    model, head, V = case.oracle
    K = w.beam
    plain = case.eng.decode(K, mode=1, trace=True)
    ar = case.eng.decode(K, mode=2, trace=True)
    case.eng.set_option(5, 1)
    out = case.eng.decode(K, mode=1, trace=True)
    assert torch.equal(out["codes"], ar["codes"]) and torch.equal(out["count"], ar["count"])
    assert out["stats"].primary_tokens <= plain["stats"].primary_tokens
    check_walk_against_trace(out, w.batch, w.L)
    tr = {k: v.cpu().numpy() for k, v in out["trace"].items()}
    # the policy itself, from the trace: a round drafts (the draft head's tree has nodes) iff every earlier round of the
    # request settled at least two levels
    for b in range(w.batch):
        spec, m = True, 1
        for r in range(w.L - 1):
            reached = int(tr["level_reached"][r, b])
            if reached < 0:
                break
            drafted = bool((tr["tree_count"][r, :, b] > 0).any())
            if not spec:
                assert not drafted and int(tr["n_draft"][r, b]) == 0, (b, r)
            spec = spec and (reached - m >= 2)
            m = reached
    if name == "tiny":
        tot = 0
        for b in range(w.batch):
            sets, st = O.speculative_decode(model, head, case.req(b), K, V, adaptive=True)
            for r in range(st.rounds):
                n = len(st.accepted_len[r])
                assert int(tr["n_draft"][r, b]) == n and list(tr["accepted_len"][r, b, :n]) == st.accepted_len[r]
                assert int(tr["level_reached"][r, b]) == st.reject_level[r]
            tot += st.primary_tokens
        assert out["stats"].primary_tokens == tot
        ar_codes = ar["codes"].cpu().numpy()
        rng = np.random.default_rng(11)
        drafts = ar_codes.copy()
        n_draft = ar["count"].cpu().numpy().copy()
        for b in range(w.batch):
            for k in range(n_draft[b]):
                if rng.random() < 0.6:
                    lvl = int(rng.integers(0, w.L))
                    drafts[b, k, lvl] = (drafts[b, k, lvl] + 1 + rng.integers(0, w.T[lvl] - 1)) % w.T[lvl]
        got = case.eng.decode_with_drafts(K, torch.from_numpy(drafts).cuda(), torch.from_numpy(n_draft).cuda(), trace=True)
        assert torch.equal(got["codes"], ar["codes"])
        tot = 0
        for b in range(w.batch):
            D = [tuple(int(c) for c in drafts[b, k]) for k in range(n_draft[b])]
            sets, st = O.speculative_decode(model, head, case.req(b), K, V, drafts_round1=D, adaptive=True)
            assert [int(x) for x in got["trace"]["level_reached"][: st.rounds, b].cpu()] == st.reject_level
            tot += st.primary_tokens
        assert got["stats"].primary_tokens == tot
    case.eng.set_option(5, 0)
    again = case.eng.decode(K, mode=1)
    assert again["stats"].primary_tokens == plain["stats"].primary_tokens


def test_select_stage_with_prefix_filter(tiny):
    """One level of beam search on caller-supplied logits with the filter at an earlier level (level 1 of 3)."""
    w = tiny.w
    V = tiny.oracle[2]
    rng = np.random.default_rng(3)
    nb, K, level = 4, w.beam, 1
    logits = rng.standard_normal((w.batch, nb, w.T[level])).astype(np.float32)
    bscore = -rng.random((w.batch, nb)).astype(np.float32)
    bcodes = np.stack([rng.permutation(w.T[0])[:nb] for _ in range(w.batch)])[:, :, None].astype(np.int32)
    n_live = np.full((w.batch,), nb, dtype=np.int32)
    for per_beam in (w.T[level], 3):
        parent, code, score, count = (x.cpu().numpy() for x in tiny.eng.select(
            torch.from_numpy(logits).cuda(), torch.from_numpy(bscore).cuda(), torch.from_numpy(bcodes).cuda(),
            torch.from_numpy(n_live).cuda(), K, level, per_beam, True))
        for b in range(w.batch):
            beams = [O.Beam((int(bcodes[b, r, 0]),), np.float32(bscore[b, r])) for r in range(nb)]
            ref = O.expand_level(beams, [logits[b, r].astype(np.float64) for r in range(nb)], K, per_beam, V)
            got = [(int(bcodes[b, parent[b, k], 0]), int(code[b, k])) for k in range(count[b])]
            assert got == [x.codes for x in ref]
            assert np.allclose(score[b, : count[b]], [float(x.score) for x in ref], atol=2e-6)


def test_nearly_full_tables():
    """Load factor 0.95: long probe walks in the hash set and in the prefix map; membership stays exact, and both
    last-level masks still agree with each other and with the oracle's set."""
    w = synth.scaled(synth.WORKLOADS["small"], n_layers=1, n_items=200_000, batch=3, n_hist=10, load_factor=0.95)
    case = Case(w).prefill()
    V = case.oracle[2]
    assert case.n_unique == w.n_items
    probe = synth.probe_keys_mix(w, case.catalog, 300_000)
    keys = case.eng.pack(torch.from_numpy(probe).cuda())
    assert np.array_equal(case.eng.probe(keys).cpu().numpy().astype(bool), V.contains(probe))
    outs = {}
    for mask in (0, 1):
        case.eng.set_option(3, mask)
        outs[mask] = case.eng.decode(w.beam, mode=2)
    for k in ("codes", "scores", "count"):
        assert torch.equal(outs[0][k], outs[1][k])
    codes, count = outs[1]["codes"].cpu().numpy(), outs[1]["count"].cpu().numpy()
    live = np.arange(w.beam)[None, :] < count[:, None]
    assert V.contains(codes[live]).all()
