"""Seeded synthetic workloads: shapes, random-init weights, item catalogues, user histories.

This module is the only code shared by the CUDA path's tests/benchmarks and the CPU oracle.  It holds
no arithmetic of the decoding method: it only draws random inputs of the right shape and distribution.

The five workloads take the shapes of the paper's setting (semantic IDs of L codes over per-level
codebooks, short histories of items flattened into code tokens, beam search of width K; Section 4.1
"Implementation Details" and Table 2) scaled up to LLM backbones of 0.5B-7B parameters.  They stand in
for the public datasets (Yelp, Amazon Beauty, Amazon Games) and the production data the paper measures
on, none of which is available here.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                 # "fp32" | "bf16": storage type of weights, activations and KV cache
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    d_ffn: int
    L: int                     # codes per semantic ID
    T: Tuple[int, ...]         # codebook size per level
    n_items: int               # catalogue size (valid tuples)
    catalog: str               # "uniform" | "zipf"
    n_hist: int                # history items per request
    batch: int
    beam: int
    seed: int
    draft_noise: float = 0.0   # std of extra N(0, .) noise on the draft-head matrices
    load_factor: float = 0.5
    rope_theta: float = 10000.0
    rms_eps: float = 1e-6

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_q_heads

    @property
    def vocab(self) -> int:
        # level codes, then L placeholder tokens, then BOS
        return int(sum(self.T)) + self.L + 1

    @property
    def ctx_tokens(self) -> int:
        # BOS + flattened history
        return 1 + self.n_hist * self.L


WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", "fp32", 2, 64, 4, 4, 256, 3, (32, 32, 32), 5_000, "uniform", 20, 4, 5, 0),
    "small": Workload("small", "bf16", 4, 512, 8, 8, 2048, 4, (256,) * 4, 1_000_000, "zipf", 50, 64, 10, 1),
    "0.5b": Workload("0.5b", "bf16", 24, 896, 14, 2, 4864, 4, (256,) * 4, 10_000_000, "zipf", 100, 256, 20, 2),
    "1.5b": Workload("1.5b", "bf16", 28, 1536, 12, 2, 8960, 4, (256,) * 4, 100_000_000, "zipf", 200, 128, 50, 3),
    "7b": Workload("7b", "bf16", 32, 4096, 32, 8, 11008, 4, (256,) * 4, 100_000_000, "zipf", 500, 32, 20, 4,
                   draft_noise=0.05),
    # The setting of the paper's own public-data experiments (Section 4.1, Tables 2 and 3): semantic IDs of L = 3 codes
    # over codebooks of 512, beam 10, histories of about a dozen items, tens of thousands of items, a backbone of the
    # size of the 1B-parameter model it names (16 layers, d = 2048, 32 query / 8 KV heads, FFN 8192).
    "paper": Workload("paper", "bf16", 16, 2048, 32, 8, 8192, 3, (512,) * 3, 57_000, "zipf", 12, 64, 10, 5),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (reduced batch, catalogue, history... for tests)."""
    return replace(w, **kw)


def torch_dtype(w: Workload) -> torch.dtype:
    return torch.float32 if w.dtype == "fp32" else torch.bfloat16


# ----------------------------------------------------------------------------------------------------
# weights
# ----------------------------------------------------------------------------------------------------

def make_weights(w: Workload, device: str = "cpu", std: float = 0.02) -> Dict[str, object]:
    """Random-init weights, all matrices row-major [out_features, in_features].

    Matrices ~ N(0, std^2); norm gains ~ 1 + 0.1*N(0,1) and the draft bias ~ N(0, std^2) so that a test
    notices a dropped gain or bias.  Values are drawn in fp32 and rounded once to the storage type; those
    rounded values are the ground truth for every consumer.  The draft-head matrices get extra
    N(0, draft_noise^2) noise (the low-acceptance workload).
    """
    g = torch.Generator(device=device)
    g.manual_seed(1_000_003 * (w.seed + 1))
    dt = torch_dtype(w)
    d, hd = w.d_model, w.head_dim

    def mat(rows, cols, s=std):
        return (torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * s).to(dt)

    def gain(n):
        return (1.0 + 0.1 * torch.randn(n, generator=g, device=device, dtype=torch.float32)).to(dt)

    out: Dict[str, object] = {
        "embed": mat(w.vocab, d),
        "lm_head": mat(w.vocab, d),
        "final_norm": gain(d),
    }
    per_layer = {k: [] for k in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")}
    for _ in range(w.n_layers):
        per_layer["attn_norm"].append(gain(d))
        per_layer["wq"].append(mat(w.n_q_heads * hd, d))
        per_layer["wk"].append(mat(w.n_kv_heads * hd, d))
        per_layer["wv"].append(mat(w.n_kv_heads * hd, d))
        per_layer["wo"].append(mat(d, w.n_q_heads * hd))
        per_layer["mlp_norm"].append(gain(d))
        per_layer["w_gate"].append(mat(w.d_ffn, d))
        per_layer["w_up"].append(mat(w.d_ffn, d))
        per_layer["w_down"].append(mat(d, w.d_ffn))
    out.update(per_layer)
    ds = float(np.sqrt(std * std + w.draft_noise * w.draft_noise))
    out["draft_logit"] = [mat(w.T[l], d, ds) for l in range(w.L)]
    out["draft_ws"] = mat(d, d, ds)
    out["draft_we"] = mat(d, d, ds)
    out["draft_b"] = mat(1, d, ds).reshape(d)
    return out


def weights_to_numpy(weights: Dict[str, object]) -> Dict[str, object]:
    """Host float32 copies (exact for both storage types) for consumers that work in numpy."""
    def cv(t):
        return t.detach().to("cpu", torch.float32).numpy()
    return {k: ([cv(t) for t in v] if isinstance(v, list) else cv(v)) for k, v in weights.items()}


# ----------------------------------------------------------------------------------------------------
# catalogue
# ----------------------------------------------------------------------------------------------------

def _zipf_quotas(n_items: int, n_prefix: int, cap: int, s: float) -> np.ndarray:
    """q_r = min(cap, floor(c * r^-s)) for ranks r = 1..n_prefix with c chosen so that sum(q) == n_items."""
    assert n_items <= n_prefix * cap
    n_prefix = min(n_prefix, n_items)      # quotas are non-increasing and sum to n_items: later ranks get 0
    r = np.arange(1, n_prefix + 1, dtype=np.float64) ** (-s)
    lo, hi = 0.0, float(cap) * float(n_prefix) ** s + 1.0

    def total(c):
        return int(np.minimum(np.floor(c * r), cap).sum())

    for _ in range(40):                      # a shortfall left by the finite bisection goes to `rem` below
        mid = 0.5 * (lo + hi)
        if total(mid) <= n_items:
            lo = mid
        else:
            hi = mid
    q = np.minimum(np.floor(lo * r), cap).astype(np.int64)
    rem = n_items - int(q.sum())
    assert rem >= 0
    if rem:
        free = np.flatnonzero(q < cap)
        # one extra item to the first unsaturated ranks, round-robin if the remainder is larger
        while rem > 0:
            take = free[: min(rem, free.size)]
            q[take] += 1
            rem -= take.size
            free = np.flatnonzero(q < cap)
    return q


def make_catalog(w: Workload) -> np.ndarray:
    """Distinct valid code tuples, int32 [n_items, L], in a seeded order.

    "uniform": n distinct tuples uniform over the whole code space.
    "zipf":    the prod(T[:-1]) prefixes get Zipf(1.1) quotas of last-level codes (clustered prefixes; the
               head saturates at T_L items per prefix), rank -> prefix by a seeded permutation, and each
               prefix's last codes are an arithmetic progression with a seeded start and odd stride.
    Catalogue order: popular prefixes first, which is what the Zipf history sampler relies on.
    """
    rng = np.random.default_rng(7_000_001 * (w.seed + 1))
    T = np.asarray(w.T, dtype=np.int64)
    if w.catalog == "uniform":
        space = int(np.prod(T))
        flat = rng.choice(space, size=w.n_items, replace=False)
        codes = np.stack(np.unravel_index(flat, tuple(int(t) for t in T)), axis=1)
        return np.ascontiguousarray(codes.astype(np.int32))
    n_prefix = int(np.prod(T[:-1]))
    cap = int(T[-1])
    q = _zipf_quotas(w.n_items, n_prefix, cap, 1.1)
    used = int(np.flatnonzero(q).max()) + 1
    q = q[:used]
    # seeded bijection rank -> prefix id over the whole prefix space: odd multiplier + offset modulo a
    # power of two when the space is one, else a random permutation
    if n_prefix & (n_prefix - 1) == 0:
        a = int(rng.integers(0, n_prefix // 2)) * 2 + 1
        b = int(rng.integers(0, n_prefix))
        prefix_id = (np.arange(used, dtype=np.int64) * a + b) & (n_prefix - 1)
    else:
        prefix_id = rng.permutation(n_prefix)[:used].astype(np.int64)
    start = rng.integers(0, cap, size=used, dtype=np.int64)
    if cap & (cap - 1) == 0:
        stride = rng.integers(0, cap // 2, size=used, dtype=np.int64) * 2 + 1
    else:
        stride = np.ones(used, dtype=np.int64)
    owner = np.repeat(np.arange(used, dtype=np.int64), q)            # prefix rank of every item
    first = np.cumsum(q) - q
    within = np.arange(w.n_items, dtype=np.int64) - first[owner]     # 0..q_r-1
    last = (start[owner] + stride[owner] * within) % cap
    pre = np.stack(np.unravel_index(prefix_id[owner], tuple(int(t) for t in T[:-1])), axis=1)
    codes = np.concatenate([pre.astype(np.int32), last.astype(np.int32)[:, None]], axis=1)
    return np.ascontiguousarray(codes)


# ----------------------------------------------------------------------------------------------------
# histories
# ----------------------------------------------------------------------------------------------------

def make_histories(w: Workload, catalog: Optional[np.ndarray], batch: Optional[int] = None) -> np.ndarray:
    """User histories, int32 [batch, n_hist, L].

    "uniform" workloads: every code uniform over its codebook.  "zipf" workloads: items drawn from a
    continuous power law (exponent 1.1) over catalogue order, their L codes appended.
    """
    B = w.batch if batch is None else batch
    rng = np.random.default_rng(9_000_011 * (w.seed + 1))
    if w.catalog == "uniform" or catalog is None:
        cols = [rng.integers(0, w.T[l], size=(B, w.n_hist), dtype=np.int64) for l in range(w.L)]
        return np.ascontiguousarray(np.stack(cols, axis=2).astype(np.int32))
    n = catalog.shape[0]
    u = rng.random(size=(B, w.n_hist))
    a = 0.1                                        # exponent - 1
    r = ((float(n) ** (-a) - 1.0) * u + 1.0) ** (-1.0 / a)
    idx = np.clip(np.floor(r).astype(np.int64) - 1, 0, n - 1)
    return np.ascontiguousarray(catalog[idx].astype(np.int32))


def probe_keys_mix(w: Workload, catalog: np.ndarray, n: int, seed: int = 0) -> np.ndarray:
    """Code tuples for stand-alone probe tests: half drawn from the catalogue, half uniform over the space."""
    rng = np.random.default_rng(11_000_027 * (w.seed + 1) + seed)
    hit = catalog[rng.integers(0, catalog.shape[0], size=n // 2)]
    cols = [rng.integers(0, w.T[l], size=n - n // 2, dtype=np.int64) for l in range(w.L)]
    rnd = np.stack(cols, axis=1).astype(np.int32)
    out = np.concatenate([hit, rnd], axis=0)
    return np.ascontiguousarray(out[rng.permutation(n)])
