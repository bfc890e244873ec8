"""Helpers shared by the tests: build oracle objects from a synthetic workload."""
import numpy as np

from oracle import nezha_oracle as O
from paper_2511_18793_b200 import synth


def oracle_shape(w):
    return O.ModelShape(w.n_layers, w.d_model, w.n_q_heads, w.n_kv_heads, w.d_ffn, w.L, tuple(w.T),
                        w.rope_theta, w.rms_eps)


def oracle_bundle(w, weights_np, catalog, cache_f64=True, dtype=np.float64):
    shape = oracle_shape(w)
    return (O.PrimaryModel(shape, weights_np, cache_f64=cache_f64, dtype=dtype), O.DraftHead(shape, weights_np),
            O.ValidSet(catalog, w.T))


MICRO = synth.Workload("micro", "fp32", 1, 16, 2, 1, 32, 3, (4, 4, 4), 40, "uniform", 3, 2, 16, 5)


def codes_of(beams):
    return [b.codes for b in beams]


def scores_of(beams):
    return np.asarray([b.score for b in beams], dtype=np.float32)
