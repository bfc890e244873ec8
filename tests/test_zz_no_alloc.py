"""nezha_contains_noalloc against nezha_pack + nezha_probe.

The entry point under test answers "are these code tuples valid items?" without allocating device memory: the
packed keys it needs in between sit in a buffer that is part of the library.  It is meant for callers that cannot
call cudaMalloc where they need the answer (a server whose memory pool owns the whole device, a thread in a
section that must not synchronise the device, a plug-in handed buffers but no allocator).  Its answers must be bit
for bit those of the allocating path, on a first call and again on a second call that finds the buffer full of
the first call's keys.  This file sorts last on purpose, so a run that stops at the first failure has been
through every other test before.
"""
import numpy as np
import pytest
import torch

from oracle import nezha_oracle as O
from paper_2511_18793_b200 import synth

pytestmark = pytest.mark.gpu


def test_contains_noalloc_matches_pack_and_probe_twice():
    from paper_2511_18793_b200 import binding
    w = synth.scaled(synth.WORKLOADS["small"], n_items=200_000, n_layers=1, batch=2, n_hist=4)
    catalog = synth.make_catalog(w)
    cat_dev = torch.from_numpy(catalog).cuda()
    eng = binding.Engine(binding.make_config(w), synth.make_weights(w, device="cuda"), cat_dev, w.load_factor)
    assert eng.build_hashset() == w.n_items
    V = O.ValidSet(catalog, w.T)
    # two different requests, the second shorter than the first: it must not see the first one's left-over keys
    for n, seed in ((300_000, 1), (70_001, 2)):
        codes_np = synth.probe_keys_mix(w, catalog, n, seed=seed)
        codes = torch.from_numpy(codes_np).cuda()
        found = torch.full((n,), 7, dtype=torch.uint8, device="cuda")      # allocated here, before the call
        ref = eng.probe(eng.pack(codes))                                    # the existing, allocating path
        got = eng.contains_noalloc(codes, found)
        eng.sync()
        assert torch.equal(got, ref)                                        # integer result: bit exact
        assert np.array_equal(got.cpu().numpy().astype(bool), V.contains(codes_np))
        assert 0.4 < got.float().mean().item() < 0.6                        # the mix is half hits, half random tuples


def test_contains_noalloc_rejects_oversized_and_early_calls():
    from paper_2511_18793_b200 import binding
    w = synth.scaled(synth.WORKLOADS["tiny"], batch=1, n_hist=2)
    catalog = synth.make_catalog(w)
    eng = binding.Engine(binding.make_config(w), synth.make_weights(w, device="cuda"),
                         torch.from_numpy(catalog).cuda(), w.load_factor)
    n = binding.NOALLOC_MAX_TUPLES + 1
    codes = torch.zeros(n, w.L, dtype=torch.int32, device="cuda")
    found = torch.zeros(n, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.NezhaError) as e:                            # hash set not built yet
        eng.contains_noalloc(codes[:8], found[:8])
    assert e.value.status == 2
    eng.build_hashset()
    with pytest.raises(binding.NezhaError) as e:
        eng.contains_noalloc(codes, found)
    assert e.value.status == 1 and "NEZHA_NOALLOC_MAX_TUPLES" in str(e.value)
    got = eng.contains_noalloc(codes[: n - 1], found[: n - 1])              # exactly the maximum is accepted
    eng.sync()
    exp = bool(O.ValidSet(catalog, w.T).contains(np.zeros((1, w.L), dtype=np.int64))[0])
    assert bool(got.all().item()) == exp and bool(got.any().item()) == exp


def test_out_of_range_codes_are_never_found():
    """A tuple with a code outside [0, T_l) is no semantic ID: both paths must answer 0 for it (its packed key is the
    table's empty-slot value, which equals every free slot) and the next synchronising call reports NEZHA_ERR_CATALOG.
    The same holds for a raw key of all ones handed to nezha_probe."""
    from paper_2511_18793_b200 import binding
    w = synth.scaled(synth.WORKLOADS["small"], n_items=50_000, n_layers=1, batch=2, n_hist=4)
    catalog = synth.make_catalog(w)
    eng = binding.Engine(binding.make_config(w), synth.make_weights(w, device="cuda"),
                         torch.from_numpy(catalog).cuda(), w.load_factor)
    assert eng.build_hashset() == w.n_items
    good = catalog[:64].copy()
    bad = np.repeat(catalog[:1], 64, axis=0)
    for i in range(64):
        bad[i, i % w.L] = -1 if i % 2 else w.T[i % w.L]
    codes_np = np.concatenate([good, bad]).astype(np.int32)
    codes = torch.from_numpy(codes_np).cuda()
    want = np.concatenate([np.ones(64, bool), np.zeros(64, bool)])
    for path in ("noalloc", "pack_probe"):
        found = torch.full((128,), 7, dtype=torch.uint8, device="cuda")
        if path == "noalloc":
            eng.contains_noalloc(codes, found)
        else:
            eng.probe(eng.pack(codes), out=found)
        with pytest.raises(binding.NezhaError) as e:
            eng.sync()
        assert e.value.status == 6                                          # NEZHA_ERR_CATALOG
        assert np.array_equal(found.cpu().numpy().astype(bool), want), path
        eng.sync()                                                          # the error was reported once and cleared
    ones = torch.full((33,), -1, dtype=torch.int64, device="cuda")          # bit pattern of 2^64 - 1
    assert not eng.probe(ones).any().item()
    eng.sync()
