"""GPU parity on the bf16 'small' workload (full size: 1M-item Zipf catalogue, batch 64, beam 10).

bf16 storage puts the GPU's logits within 2e-2 of the fp64 oracle, so beam sets are compared level by level
with the tie rule: the oracle re-expands the GPU's own beams of level n-1 and the GPU's level-n set must be a
valid top-K of that expansion up to score differences below the tolerance."""
import numpy as np
import pytest
import torch

from oracle import nezha_oracle as O
from paper_2511_18793_b200 import synth
from gpu_helpers import Case, assert_topk_matches, check_levels, check_walk_against_trace, tolerance, wide_tolerance

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def small():
    return Case(synth.WORKLOADS["small"]).prefill()


def test_small_hashset_full_catalogue(small):
    w = small.w
    V = small.oracle[2]
    assert small.n_unique == w.n_items == len(V)
    probe = synth.probe_keys_mix(w, small.catalog, 1_000_000)
    keys = small.eng.pack(torch.from_numpy(probe).cuda())
    assert np.array_equal(keys.cpu().numpy().view(np.uint64), O.pack_keys(probe, w.T))
    found = small.eng.probe(keys).cpu().numpy().astype(bool)
    assert np.array_equal(found, V.contains(probe))
    assert 0.45 < found.mean() < 0.56


def test_small_hidden_and_logits_within_bf16_tolerance(small):
    w = small.w
    model, head, _ = small.oracle
    h = small.eng.get_hidden().cpu().numpy()
    rows = [0, w.batch // 2, w.batch - 1]
    for b in rows:
        assert np.abs(h[b] - small.req(b).h).max() < 3e-2          # unit-RMS vectors stored through bf16 stages
    rng = np.random.default_rng(7)
    for level in range(w.L):
        nb = w.beam
        pre = np.stack([rng.integers(0, w.T[l], size=(w.batch, nb)) for l in range(level)], axis=2).astype(np.int32) \
            if level else None
        pt = None if pre is None else torch.from_numpy(pre).cuda()
        got = small.eng.primary_logits(nb, level, pt).cpu().numpy()
        gotd = small.eng.draft_logits(nb, level, pt).cpu().numpy()
        for b in rows:
            req = small.req(b)
            ref = model.next_level_logits_many(req, [tuple(pre[b, r]) if level else () for r in range(nb)])
            assert np.abs(got[b] - np.stack(ref)).max() < tolerance(w)
            for r in range(nb):
                st = O.teacher_forced_state(head, req, tuple(pre[b, r]) if level else ())
                assert np.abs(gotd[b, r] - head.logits(level, req.h[level + 1], st)).max() < tolerance(w)


def test_small_verified_decode_all_rows(small):
    w = small.w
    V = small.oracle[2]
    out = small.eng.decode(w.beam, mode=1, trace=True)
    ar = small.eng.decode(w.beam, mode=2)
    # GPU-internal invariants on all rows: zero sacrifice and zero hallucinations
    assert torch.equal(out["codes"], ar["codes"]) and torch.equal(out["count"], ar["count"])
    codes, count = out["codes"].cpu().numpy(), out["count"].cpu().numpy()
    # (with an untrained model most level-(L-1) beams have no valid completion: count < beam is expected)
    live = np.arange(w.beam)[None, :] < count[:, None]
    assert V.contains(codes[live]).all() and np.all(codes[~live] == -1)
    assert 1 <= out["stats"].rounds <= w.L - 1
    beams = out["trace"]["beams"].cpu().numpy()
    scores = out["trace"]["beam_scores"].cpu().numpy()
    for b in range(w.batch):
        check_levels(small, b, beams[:, b], scores[:, b], w.beam)
        assert np.array_equal(beams[w.L - 1, b], codes[b])
    check_walk_against_trace(out, w.batch, w.L)


def test_small_accept_and_roll_back_bookkeeping(small):
    """Accepted lengths, rejection levels, rounds and token counts at beam 10, four levels, 64 requests: replayed with the
    oracle's integer rules from the GPU's own beam sets and draft trees -- for the head's own drafts, for seeded
    corruptions of the true tuples, and for the true beam sets themselves (one round, nothing beyond plain decoding's
    tokens)."""
    w = small.w
    K, L = w.beam, w.L
    art = small.eng.decode(K, mode=2, trace=True)
    ar_codes = art["codes"].cpu().numpy()
    rng = np.random.default_rng(17)
    for rho in (0.0, 0.3, 1.0):
        drafts = np.maximum(ar_codes, 0)
        n_draft = art["count"].cpu().numpy().copy()
        for b in range(w.batch):
            for k in range(n_draft[b]):
                if rng.random() < rho:
                    lvl = int(rng.integers(0, L))
                    drafts[b, k, lvl] = (drafts[b, k, lvl] + 1 + rng.integers(0, w.T[lvl] - 1)) % w.T[lvl]
        out = small.eng.decode_with_drafts(K, torch.from_numpy(drafts).cuda(), torch.from_numpy(n_draft).cuda(), trace=True)
        assert torch.equal(out["codes"], art["codes"]) and torch.allclose(out["scores"], art["scores"], atol=1e-4)
        check_walk_against_trace(out, w.batch, L)
        tr_tree = out["trace"]["tree_count"].cpu().numpy()
        for b in range(w.batch):
            D = [tuple(int(c) for c in drafts[b, k]) for k in range(n_draft[b])]
            assert list(tr_tree[0, :, b]) == [len(x) for x in O.tree_from_tuples(D, L)]
    beams = art["trace"]["beams"]
    counts = (beams[:, :, :, 0] >= 0).sum(dim=2).to(torch.int32)
    out = small.eng.decode_with_draft_tree(K, beams, counts, trace=True)
    assert torch.equal(out["codes"], art["codes"]) and torch.allclose(out["scores"], art["scores"], atol=1e-4)
    assert out["stats"].rounds == 1 and out["stats"].primary_tokens == int(counts[: L - 1].sum())
    acc = out["trace"]["accepted_len"].cpu().numpy()
    for b in range(w.batch):
        n = int(counts[L - 1, b])
        assert np.all(acc[0, b, :n] == L)
    check_walk_against_trace(out, w.batch, L)
    check_walk_against_trace(art, w.batch, L)                      # plain decoding: empty trees, L - 1 rounds
    assert art["stats"].rounds == L - 1


def test_small_draft_mode(small):
    w = small.w
    _, head, V = small.oracle
    out = small.eng.decode(w.beam, mode=0)
    codes, scores, count = [out[k].cpu().numpy() for k in ("codes", "scores", "count")]
    n_valid = 0
    for b in range(w.batch):
        n_valid += int(count[b])
        if count[b]:
            assert V.contains(codes[b, : count[b]]).all()
        ref = O.nezha_draft(head, small.req(b), w.beam, V)[-1]
        assert_topk_matches(codes[b], scores[b], count[b], ref, w.beam, tolerance(w))
        for k in range(count[b]):                                   # scores are the head's joint log-probabilities
            lp = O.joint_logprob_draft(head, small.req(b), tuple(int(c) for c in codes[b, k]))
            assert abs(lp - scores[b, k]) < w.L * tolerance(w)
    assert n_valid >= 0


# ---------------------------------------------------------------------------------------- other bf16 shapes
SHAPES = {
    "hd128_gqa2": dict(d_model=512, n_q_heads=4, n_kv_heads=2, d_ffn=1024),      # head_dim 128, groups of 2
    "hd64_gqa7": dict(d_model=448, n_q_heads=7, n_kv_heads=1, d_ffn=896),        # head_dim 64, 7 query heads on 1 KV head
    "hd128_mha": dict(d_model=256, n_q_heads=2, n_kv_heads=2, d_ffn=512),
}


@pytest.mark.parametrize("shape", sorted(SHAPES))
def test_bf16_shapes_ragged_histories(shape):
    w = synth.scaled(synth.WORKLOADS["small"], n_layers=2, n_items=50_000, batch=5, beam=7, n_hist=40, seed=11,
                     **SHAPES[shape])
    case = Case(w)
    lens = [40, 1, 17, 0, 33]
    case.eng.prefill(case.hist_dev, torch.tensor(lens, dtype=torch.int32, device="cuda"))
    model, head, V = case.oracle
    reqs = [model.prefill(case.hist[b, :n]) for b, n in enumerate(lens)]
    case._reqs = {(b, None): r for b, r in enumerate(reqs)}
    h = case.eng.get_hidden().cpu().numpy()
    for b in range(w.batch):
        assert np.abs(h[b] - reqs[b].h).max() < 3e-2
    rng = np.random.default_rng(1)
    for level in (1, 3):
        pre = np.stack([rng.integers(0, w.T[l], size=(w.batch, w.beam)) for l in range(level)], axis=2).astype(np.int32)
        got = case.eng.primary_logits(w.beam, level, torch.from_numpy(pre).cuda()).cpu().numpy()
        for b in range(w.batch):
            ref = model.next_level_logits_many(reqs[b], [tuple(pre[b, r]) for r in range(w.beam)])
            assert np.abs(got[b] - np.stack(ref)).max() < tolerance(w)
    out = case.eng.decode(w.beam, mode=1, trace=True)
    ar = case.eng.decode(w.beam, mode=2)
    assert torch.equal(out["codes"], ar["codes"])
    beams = out["trace"]["beams"].cpu().numpy()
    scores = out["trace"]["beam_scores"].cpu().numpy()
    for b in range(w.batch):
        check_levels(case, b, beams[:, b], scores[:, b], w.beam)
    check_walk_against_trace(out, w.batch, w.L)


@pytest.mark.parametrize("batch", [7, 6, 3, 1])
def test_paper_setting_three_levels_of_512_codes(batch):
    """L = 3 levels over codebooks of 512 (the paper's own setting), beam 10, short histories: every mode, all requests,
    on a two-layer cut of the 1B-sized backbone.  With 6 requests (120 rows per pass at most), 3 (60 rows) and 1 (20 rows)
    every product of the decode calls runs in the weight-streaming kernel, on its 128-, 64- and 32-row accumulator; with
    7 requests in the general kernels."""
    w = synth.scaled(synth.WORKLOADS["paper"], n_layers=2, batch=batch)
    case = Case(w).prefill()
    model, head, V = case.oracle
    assert case.n_unique == w.n_items
    out = case.eng.decode(w.beam, mode=1, trace=True)
    ar = case.eng.decode(w.beam, mode=2)
    assert torch.equal(out["codes"], ar["codes"]) and torch.equal(out["count"], ar["count"])
    beams, scores = out["trace"]["beams"].cpu().numpy(), out["trace"]["beam_scores"].cpu().numpy()
    dr = case.eng.decode(w.beam, mode=0)
    dcodes, dscores, dcount = (dr[k].cpu().numpy() for k in ("codes", "scores", "count"))
    for b in range(w.batch):
        check_levels(case, b, beams[:, b], scores[:, b], w.beam, tol=wide_tolerance(w))     # d = 2048, two layers
        ref = O.nezha_draft(head, case.req(b), w.beam, V)[-1]
        assert_topk_matches(dcodes[b], dscores[b], dcount[b], ref, w.beam, tolerance(w))
    codes, count = out["codes"].cpu().numpy(), out["count"].cpu().numpy()
    live = np.arange(w.beam)[None, :] < count[:, None]
    assert V.contains(codes[live]).all()
    check_walk_against_trace(out, w.batch, w.L)
    # the true beam sets as the draft tree: one round, the tokens of plain decoding, every tuple accepted in full
    tb = out["trace"]["beams"]
    counts = (tb[:, :, :, 0] >= 0).sum(dim=2).to(torch.int32)
    pt = case.eng.decode_with_draft_tree(w.beam, tb, counts, trace=True)
    assert torch.equal(pt["codes"], ar["codes"]) and torch.equal(pt["count"], ar["count"])
    live_t = torch.from_numpy(live).cuda()                  # (one pass over all levels rounds differently from one per level)
    assert (pt["scores"][live_t] - ar["scores"][live_t]).abs().max().item() <= tolerance(w) if live.any() else True
    assert pt["stats"].rounds == 1 and pt["stats"].primary_tokens == int(counts[: w.L - 1].sum())
    check_walk_against_trace(pt, w.batch, w.L)


@pytest.mark.parametrize("name", ["tiny", "small", "paper_batch1"])
def test_graph_replay_equals_eager_launches(name):
    """On a stream of its own the library captures every round of a decode call into a CUDA graph after one eager
    run and replays it afterwards.  Eager, capturing and replaying calls must give the same bits as an engine on the
    default stream (which never captures), in every mode, with and without trace outputs and with injected drafts.
    (paper_batch1: one request of the paper's setting on a two-layer cut, whose products are cluster launches of the
    weight-streaming kernel: those are captured and replayed too, and the drafts of the last part are the result
    itself, so that call ends in one round.)"""
    w = synth.scaled(synth.WORKLOADS["paper"], n_layers=2, batch=1) if name == "paper_batch1" else synth.WORKLOADS[name]
    ref = Case(w).prefill()
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        cap = Case(w, weights=ref.weights, catalog=ref.catalog, hist=ref.hist, stream=st).prefill()
        for mode in (1, 0, 2):
            want = ref.eng.decode(w.beam, mode=mode, trace=(mode == 1))
            out = cap.eng.alloc_outputs(w.batch, w.beam, trace=(mode == 1))
            for call in range(4):                                   # eager, capture, replay, replay
                got = cap.eng.decode(w.beam, mode=mode, out=out)
                st.synchronize()
                for k in ("codes", "scores", "count"):
                    assert torch.equal(got[k], want[k]), (mode, call, k)
                assert got["stats"].rounds == want["stats"].rounds
                assert got["stats"].primary_tokens == want["stats"].primary_tokens
                if mode == 1:
                    for k, v in want["trace"].items():
                        assert torch.equal(got["trace"][k], v), (call, k)
        drafts = want["codes"].clone().clamp_(min=0)
        nd = want["count"].clone()
        w1 = ref.eng.decode_with_drafts(w.beam, drafts, nd)
        out = cap.eng.alloc_outputs(w.batch, w.beam)
        for call in range(3):
            g1 = cap.eng.decode_with_drafts(w.beam, drafts, nd, out=out)
            st.synchronize()
            assert torch.equal(g1["codes"], w1["codes"]) and torch.equal(g1["scores"], w1["scores"])
            assert g1["stats"].rounds == w1["stats"].rounds
    torch.cuda.synchronize()
