"""GPU parity at the full sizes of the three LLM-shaped workloads (0.5B / 1.5B / 7B shapes; 10M and 100M-item
catalogues), in the launch configuration bench.py times.

All requests: GPU-internal invariants (verified decode == plain autoregressive decode item for item; every emitted
tuple is in the exact valid set; counts and padding).  A fixed subset of requests: the oracle recomputes every
beam level from the GPU's own beams (tie rule), the prefill hidden states and the draft head's first-level logits.  The hash set is probed with a
hit/miss mix and with sibling keys and compared bit for bit with the exact set."""
import numpy as np
import pytest
import torch

from oracle import nezha_oracle as O
from paper_2511_18793_b200 import synth
from gpu_helpers import Case, wide_tolerance, check_levels, check_walk_against_trace, e2e_tolerance, hidden_rms_bound, hidden_tolerance, stage_tolerance

pytestmark = pytest.mark.gpu

PLAN = {                       # workload -> (requests checked by the oracle, oracle arithmetic)
    "0.5b": ([0, 128, 255, 77], np.float64),
    "1.5b": ([0, 127], np.float64),
    "7b": ([0, 31], np.float32),   # 5.7e9 parameters x 2005 tokens: fp32 BLAS keeps the check to about a minute per request
}


@pytest.mark.parametrize("name", ["0.5b", "1.5b", "7b"])
def test_full_size_workload(name):
    w = synth.WORKLOADS[name]
    rows, odt = PLAN[name]
    # the launch configuration bench.py times: a stream of the engine's own, on which the library replays every round of a
    # decode call as a CUDA graph from the third call on (first call eager, second captured)
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        _full_size_checks(name, w, rows, odt, st)
    torch.cuda.synchronize()


def _full_size_checks(name, w, rows, odt, st):
    case = Case(w, oracle_dtype=odt, stream=st).prefill()
    V = O.ValidSet(case.catalog, w.T)
    assert case.n_unique == w.n_items == len(V)
    # ---- hash set, bit exact
    probe = synth.probe_keys_mix(w, case.catalog, 2_000_000)
    keys = case.eng.pack(torch.from_numpy(probe).cuda())
    assert np.array_equal(keys.cpu().numpy().view(np.uint64), O.pack_keys(probe, w.T))
    assert np.array_equal(case.eng.probe(keys).cpu().numpy().astype(bool), V.contains(probe))
    pre = case.catalog[np.random.default_rng(0).integers(0, len(case.catalog), 2000)]
    sib = np.repeat(pre, w.T[-1], axis=0)
    sib[:, -1] = np.tile(np.arange(w.T[-1]), len(pre))
    got = case.eng.probe(case.eng.pack(torch.from_numpy(sib.astype(np.int32)).cuda())).cpu().numpy().astype(bool)
    assert np.array_equal(got, V.contains(sib))
    # ---- decode: invariants on every request (eager, captured and replayed calls must agree bit for bit)
    outs = case.eng.alloc_outputs(w.batch, w.beam, trace=True)
    first = {k: v.clone() for k, v in case.eng.decode(w.beam, mode=1, out=outs).items() if k in ("codes", "scores", "count")}
    for call in range(4):       # the tiling follows the token counts of the call before: eager again, captured, replayed twice
        out = case.eng.decode(w.beam, mode=1, out=outs)
        st.synchronize()
        for k, v in first.items():
            assert torch.equal(out[k], v), (call, k)
    ar_out = case.eng.alloc_outputs(w.batch, w.beam)
    for call in range(4):
        ar = case.eng.decode(w.beam, mode=2, out=ar_out)
    st.synchronize()
    assert torch.equal(out["codes"], ar["codes"]) and torch.equal(out["count"], ar["count"])
    assert torch.allclose(out["scores"], ar["scores"], atol=1e-4)
    codes, count = out["codes"].cpu().numpy(), out["count"].cpu().numpy()
    live = np.arange(w.beam)[None, :] < count[:, None]
    assert V.contains(codes[live]).all() and np.all(codes[~live] == -1)
    assert 1 <= out["stats"].rounds <= w.L - 1
    # accept / roll-back bookkeeping of every request, replayed from the GPU's own beams and draft trees (integers only)
    check_walk_against_trace(out, w.batch, w.L)
    beams_dev = out["trace"]["beams"]
    counts = (beams_dev[:, :, :, 0] >= 0).sum(dim=2).to(torch.int32)
    perfect = case.eng.decode_with_draft_tree(w.beam, beams_dev.clone(), counts, trace=True)
    assert torch.equal(perfect["codes"], ar["codes"]) and torch.allclose(perfect["scores"], ar["scores"], atol=1e-4)
    assert perfect["stats"].rounds == 1 and perfect["stats"].primary_tokens == int(counts[: w.L - 1].sum())
    check_walk_against_trace(perfect, w.batch, w.L)
    dr = case.eng.decode(w.beam, mode=0)
    dcodes, dcount = dr["codes"].cpu().numpy(), dr["count"].cpu().numpy()
    dlive = np.arange(w.beam)[None, :] < dcount[:, None]
    assert V.contains(dcodes[dlive]).all()
    # ---- oracle on a subset of requests
    case._oracle = None
    model, head, _ = case.oracle
    h = case.eng.get_hidden().cpu().numpy()
    beams = out["trace"]["beams"].cpu().numpy()
    scores = out["trace"]["beam_scores"].cpu().numpy()
    swaps = []
    for b in rows:
        dh = h[b] - case.req(b).h
        assert np.abs(dh).max() < hidden_tolerance(w) and np.sqrt((dh ** 2).mean()) < hidden_rms_bound(w)
        check_levels(case, b, beams[:, b], scores[:, b], w.beam, tol=e2e_tolerance(w), swaps=swaps)
    # members that were not the oracle's own choice (all of them near-ties at the K-th place): a minority at every level
    print(f"{name}: tie-rule members per (request, level): {swaps}")
    assert max(swaps) <= w.beam // 2
    # draft head, stage-wise: the oracle's Eq. 1-2 on the hidden states the GPU's prefill produced (float64 copies of
    # the same numbers), so that the 2e-2 budget is spent by the draft head alone and not by 24-32 layers of bf16
    # activations upstream; end to end (oracle hidden states) the same logits stay within the depth-scaled bound
    # (h_l + s_1 carries two hidden-state errors, hence the factor)
    gotd = case.eng.draft_logits(w.beam, 0, None).cpu().numpy()
    for b in rows:
        hg = h[b].astype(np.float64)
        w_std = float(np.hypot(0.02, w.draft_noise))
        tol = stage_tolerance(w, w_std, float(np.sqrt(((hg[1] + hg[0]) ** 2).mean())))
        assert np.abs(gotd[b, 0] - head.logits(0, hg[1], hg[0])).max() < tol
        assert np.abs(gotd[b, 0] - head.logits(0, case.req(b).h[1], case.req(b).h[0])).max() < \
            tol + 1.5 * e2e_tolerance(w, std=w_std)


@pytest.mark.parametrize("name", ["0.5b", "1.5b", "7b"])
def test_two_layer_cut_at_full_width(name):
    """The three LLM shapes cut to two layers: full width, head dimension, grouped-query ratio, context length and beam
    (so the CTA-pair GEMM, both tcgen05 attention shapes and the 20- / 50-beam selection all run), without 24-32 layers
    of accumulated bf16 rounding between the GPU and the fp64 oracle.  Every request, every stage:
      * prefill hidden states within the two-layer bound; teacher-forced primary logits of every level within 2e-2 in rms
        at every width, and their largest element (of 5 k to 13 k per request and level) within five standard deviations
        of the rounding model: the measured hidden-state error of bf16 activations (0.0074 rms after one layer, 0.0105
        after two, whatever the width) seen through an LM-head row of norm 0.02 * sqrt(d) is 0.0063 / 0.0082 / 0.0134 rms
        per logit at d = 896 / 1536 / 4096;
      * every beam level of the verified decode against the oracle's expansion of the GPU's own beams;
      * verified == plain autoregressive decode, zero hallucinations, the accept / roll-back walk replayed."""
    w = synth.scaled(synth.WORKLOADS[name], n_layers=2, batch=4, n_items=200_000)
    case = Case(w).prefill()
    model, head, V = case.oracle
    tol = wide_tolerance(w)
    h = case.eng.get_hidden().cpu().numpy()
    for b in range(w.batch):
        dh = h[b] - case.req(b).h
        assert np.abs(dh).max() < hidden_tolerance(w) and np.sqrt((dh ** 2).mean()) < hidden_rms_bound(w)
    rng = np.random.default_rng(3)
    for level in range(w.L):
        pre = np.stack([rng.integers(0, w.T[l], size=(w.batch, w.beam)) for l in range(level)], axis=2).astype(np.int32) \
            if level else None
        pt = None if pre is None else torch.from_numpy(pre).cuda()
        got = case.eng.primary_logits(w.beam, level, pt).cpu().numpy()
        for b in range(w.batch):
            ref = model.next_level_logits_many(case.req(b), [tuple(pre[b, r]) if level else () for r in range(w.beam)])
            err = got[b] - np.stack(ref)
            assert np.abs(err).max() < tol and np.sqrt((err ** 2).mean()) < 2e-2, (level, b, np.abs(err).max())
    out = case.eng.decode(w.beam, mode=1, trace=True)
    ar = case.eng.decode(w.beam, mode=2)
    assert torch.equal(out["codes"], ar["codes"]) and torch.equal(out["count"], ar["count"])
    codes, count = out["codes"].cpu().numpy(), out["count"].cpu().numpy()
    live = np.arange(w.beam)[None, :] < count[:, None]
    assert V.contains(codes[live]).all() and np.all(codes[~live] == -1)
    beams, scores = out["trace"]["beams"].cpu().numpy(), out["trace"]["beam_scores"].cpu().numpy()
    swaps = []
    for b in range(w.batch):
        check_levels(case, b, beams[:, b], scores[:, b], w.beam, tol=max(tol, e2e_tolerance(w)), swaps=swaps)
    print(f"{name} (2 layers): tie-rule members per (request, level): {swaps}")
    assert max(swaps) <= w.beam // 2
    check_walk_against_trace(out, w.batch, w.L)
