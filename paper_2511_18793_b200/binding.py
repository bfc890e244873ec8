"""ctypes binding of libnezha.so: the same entry points as include/nezha.h, argument marshalling only.

PyTorch supplies device memory and the CUDA stream; every computation runs inside the library.  Importing
this module fails loudly when the library has not been built (there is no fallback path).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnezha.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_18793_b200.build`")
lib = C.CDLL(LIB_PATH)

MAX_LEVELS = 8
MODE_DRAFT, MODE_VERIFIED, MODE_AR = 0, 1, 2
OPT_DRAFT_TRANSITION, OPT_DRAFT_INPUTS, OPT_DRAFT_FILTER, OPT_FINAL_MASK, OPT_LEVEL_FILTER, OPT_ADAPTIVE_DRAFT = 0, 1, 2, 3, 4, 5
STATUS_NAMES = ["OK", "ERR_ARG", "ERR_STATE", "ERR_ARENA_TOO_SMALL", "ERR_CUDA", "ERR_HASH_FULL", "ERR_CATALOG",
                "ERR_UNSUPPORTED"]


class NezhaConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("d_ffn", C.c_int32), ("L", C.c_int32), ("T", C.c_int32 * MAX_LEVELS), ("dtype", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("max_batch", C.c_int32), ("max_beam", C.c_int32),
                ("max_hist_items", C.c_int32)]


_PP = C.POINTER(C.c_void_p)


class NezhaWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", _PP), ("wq", _PP), ("wk", _PP), ("wv", _PP), ("wo", _PP), ("mlp_norm", _PP),
                ("w_gate", _PP), ("w_up", _PP), ("w_down", _PP), ("draft_logit", _PP),
                ("draft_ws", C.c_void_p), ("draft_we", C.c_void_p), ("draft_b", C.c_void_p)]


class NezhaDecodeStats(C.Structure):
    _fields_ = [("rounds", C.c_int32), ("primary_tokens", C.c_int64), ("drafted", C.c_int64),
                ("accepted_levels", C.c_int64)]


class NezhaTrace(C.Structure):
    _fields_ = [("drafts", C.c_void_p), ("n_draft", C.c_void_p), ("accepted_len", C.c_void_p),
                ("level_reached", C.c_void_p), ("beams", C.c_void_p), ("beam_scores", C.c_void_p),
                ("tree_codes", C.c_void_p), ("tree_count", C.c_void_p)]


_vp, _i32, _sz = C.c_void_p, C.c_int32, C.c_size_t
lib.nezha_arena_bytes.restype = _sz
lib.nezha_arena_bytes.argtypes = [C.POINTER(NezhaConfig), _sz, C.c_double]
lib.nezha_create.restype = C.c_int
lib.nezha_create.argtypes = [C.POINTER(NezhaConfig), C.POINTER(NezhaWeights), _vp, _sz, C.c_double, _vp, _sz, _vp,
                             C.POINTER(_vp)]
lib.nezha_build_hashset.restype = C.c_int
lib.nezha_build_hashset.argtypes = [_vp, C.POINTER(C.c_uint64)]
lib.nezha_pack.restype = C.c_int
lib.nezha_pack.argtypes = [_vp, _vp, _sz, _vp]
lib.nezha_probe.restype = C.c_int
lib.nezha_probe.argtypes = [_vp, _vp, _sz, _vp]
lib.nezha_contains_noalloc.restype = C.c_int
lib.nezha_contains_noalloc.argtypes = [_vp, _vp, _sz, _vp]
lib.nezha_prefill.restype = C.c_int
lib.nezha_prefill.argtypes = [_vp, _vp, _vp, _i32, _i32]
lib.nezha_decode.restype = C.c_int
lib.nezha_decode.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp, _vp, C.POINTER(NezhaDecodeStats), C.POINTER(NezhaTrace)]
lib.nezha_decode_with_drafts.restype = C.c_int
lib.nezha_decode_with_drafts.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, C.POINTER(NezhaDecodeStats),
                                         C.POINTER(NezhaTrace)]
lib.nezha_decode_with_draft_tree.restype = C.c_int
lib.nezha_decode_with_draft_tree.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, C.POINTER(NezhaDecodeStats),
                                             C.POINTER(NezhaTrace)]
lib.nezha_set_option.restype = C.c_int
lib.nezha_set_option.argtypes = [_vp, _i32, _i32]
lib.nezha_get_hidden.restype = C.c_int
lib.nezha_get_hidden.argtypes = [_vp, _vp]
lib.nezha_primary_logits.restype = C.c_int
lib.nezha_primary_logits.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp]
lib.nezha_draft_logits.restype = C.c_int
lib.nezha_draft_logits.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp]
lib.nezha_select.restype = C.c_int
lib.nezha_select.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
class NezhaProfile(C.Structure):
    _fields_ = [("launches", C.c_int64 * 16), ("ms", C.c_double * 16)]


PROFILE_CLASSES = ["gemm", "attention", "select", "norm", "rope_append", "embed", "swiglu", "draft_glue", "nodes",
                   "accept", "hash", "misc"]
lib.nezha_gemm.restype = C.c_int
lib.nezha_gemm.argtypes = [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _vp, _i32]
lib.nezha_launch_count.restype = C.c_uint64
lib.nezha_launch_count.argtypes = []
lib.nezha_profile_enable.restype = C.c_int
lib.nezha_profile_enable.argtypes = [_vp, _i32]
lib.nezha_profile_read.restype = C.c_int
lib.nezha_profile_read.argtypes = [_vp, C.POINTER(NezhaProfile)]
lib.nezha_sync.restype = C.c_int
lib.nezha_sync.argtypes = [_vp]
lib.nezha_last_error.restype = C.c_char_p
lib.nezha_last_error.argtypes = [_vp]
lib.nezha_destroy.restype = None
lib.nezha_destroy.argtypes = [_vp]

NOALLOC_MAX_TUPLES = 1 << 20
EXPORTS = ["nezha_arena_bytes", "nezha_create", "nezha_build_hashset", "nezha_pack", "nezha_probe",
           "nezha_contains_noalloc", "nezha_prefill",
           "nezha_decode", "nezha_decode_with_drafts", "nezha_decode_with_draft_tree", "nezha_set_option", "nezha_get_hidden", "nezha_primary_logits",
           "nezha_draft_logits", "nezha_select", "nezha_gemm", "nezha_launch_count", "nezha_profile_enable",
           "nezha_profile_read", "nezha_sync", "nezha_last_error", "nezha_destroy"]


class NezhaError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"NEZHA_{STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}: {msg}")
        self.status = status


def make_config(w, max_batch: Optional[int] = None, max_beam: Optional[int] = None,
                max_hist_items: Optional[int] = None) -> NezhaConfig:
    """nezha_config from a synth.Workload-like object (fields only; no arithmetic)."""
    cfg = NezhaConfig()
    cfg.n_layers, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.d_ffn = (w.n_layers, w.d_model, w.n_q_heads,
                                                                             w.n_kv_heads, w.d_ffn)
    cfg.L = w.L
    for l in range(w.L):
        cfg.T[l] = w.T[l]
    cfg.dtype = 0 if w.dtype == "fp32" else 1
    cfg.rope_theta, cfg.rms_eps = w.rope_theta, w.rms_eps
    cfg.max_batch = w.batch if max_batch is None else max_batch
    cfg.max_beam = w.beam if max_beam is None else max_beam
    cfg.max_hist_items = w.n_hist if max_hist_items is None else max_hist_items
    return cfg


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


def _ptr_array(ts: Sequence[torch.Tensor]):
    arr = (C.c_void_p * len(ts))(*[_ptr(t) for t in ts])
    return C.cast(arr, _PP), arr


class Engine:
    """One nezha_ctx plus the device buffers it borrows (arena, catalogue).  Thin: each method is one C call."""

    def __init__(self, cfg: NezhaConfig, weights: Dict[str, object], catalog: torch.Tensor, load_factor: float = 0.5,
                 stream: Optional[torch.cuda.Stream] = None, arena_slack: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("libnezha needs a CUDA device; there is no CPU path")
        self.cfg = cfg
        self.L = cfg.L
        self.T = [cfg.T[l] for l in range(cfg.L)]
        self.stream = stream
        self.catalog = catalog.contiguous()
        assert self.catalog.dtype == torch.int32 and self.catalog.is_cuda
        n_items = int(self.catalog.shape[0])
        need = lib.nezha_arena_bytes(C.byref(cfg), n_items, load_factor)
        if need == 0:
            raise NezhaError(1, "nezha_arena_bytes rejected the configuration")
        self.arena_bytes = need + arena_slack
        self.arena = torch.empty(self.arena_bytes, dtype=torch.uint8, device=self.catalog.device)
        assert self.arena.data_ptr() % 256 == 0
        w = NezhaWeights()
        keep = []
        w.embed, w.lm_head, w.final_norm = _ptr(weights["embed"]), _ptr(weights["lm_head"]), _ptr(weights["final_norm"])
        for name in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down", "draft_logit"):
            p, arr = _ptr_array(weights[name])
            setattr(w, name, p)
            keep.append(arr)
        w.draft_ws, w.draft_we, w.draft_b = _ptr(weights["draft_ws"]), _ptr(weights["draft_we"]), _ptr(weights["draft_b"])
        self._h = C.c_void_p()
        st = lib.nezha_create(C.byref(cfg), C.byref(w), _ptr(self.catalog), n_items, load_factor, _ptr(self.arena),
                              self.arena_bytes, self._stream_ptr(), C.byref(self._h))
        if st != 0:
            raise NezhaError(st, "nezha_create failed")
        self.batch = 0

    def _stream_ptr(self):
        return None if self.stream is None else self.stream.cuda_stream

    def _check(self, st: int):
        if st != 0:
            raise NezhaError(st, lib.nezha_last_error(self._h).decode())

    def close(self):
        if self._h:
            lib.nezha_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- one method per entry point -------------------------------------------------------------------
    def build_hashset(self) -> int:
        n = C.c_uint64(0)
        self._check(lib.nezha_build_hashset(self._h, C.byref(n)))
        return int(n.value)

    def pack(self, codes: torch.Tensor) -> torch.Tensor:
        assert codes.dtype == torch.int32 and codes.dim() == 2 and codes.shape[1] == self.L
        assert codes.device == self.arena.device
        codes = codes.contiguous()
        keys = torch.empty(codes.shape[0], dtype=torch.int64, device=codes.device)   # bit pattern of uint64
        self._check(lib.nezha_pack(self._h, _ptr(codes), codes.shape[0], _ptr(keys)))
        return keys

    def probe(self, keys: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        found = out if out is not None else torch.empty(keys.shape[0], dtype=torch.uint8, device=keys.device)
        self._check(lib.nezha_probe(self._h, _ptr(keys), keys.shape[0], _ptr(found)))
        return found

    def contains_noalloc(self, codes: torch.Tensor, found: torch.Tensor) -> torch.Tensor:
        """nezha_contains_noalloc: validity of code tuples with no allocation anywhere; `codes` (int32 [n, L],
        contiguous) and `found` (uint8 [n]) are the caller's, and this method creates no tensor either."""
        assert codes.dtype == torch.int32 and found.dtype == torch.uint8 and found.shape[0] == codes.shape[0]
        assert codes.dim() == 2 and codes.shape[1] == self.L and codes.is_contiguous() and found.is_contiguous()
        assert codes.device == self.arena.device and found.device == self.arena.device
        self._check(lib.nezha_contains_noalloc(self._h, _ptr(codes), codes.shape[0], _ptr(found)))
        return found

    def prefill(self, hist_codes: torch.Tensor, n_hist: torch.Tensor):
        hist_codes, n_hist = hist_codes.contiguous(), n_hist.contiguous()
        batch, max_n = int(hist_codes.shape[0]), int(hist_codes.shape[1])
        self._check(lib.nezha_prefill(self._h, _ptr(hist_codes), _ptr(n_hist), batch, max_n))
        self.batch = batch

    def alloc_outputs(self, batch: int, beam: int, trace: bool = False):
        dev = self.arena.device
        out = {"codes": torch.empty(batch, beam, self.L, dtype=torch.int32, device=dev),
               "scores": torch.empty(batch, beam, dtype=torch.float32, device=dev),
               "count": torch.empty(batch, dtype=torch.int32, device=dev)}
        if trace:
            R = max(self.L - 1, 1)
            out["trace"] = {"drafts": torch.empty(R, batch, beam, self.L, dtype=torch.int32, device=dev),
                            "n_draft": torch.empty(R, batch, dtype=torch.int32, device=dev),
                            "accepted_len": torch.empty(R, batch, beam, dtype=torch.int32, device=dev),
                            "level_reached": torch.empty(R, batch, dtype=torch.int32, device=dev),
                            "beams": torch.empty(self.L, batch, beam, self.L, dtype=torch.int32, device=dev),
                            "beam_scores": torch.empty(self.L, batch, beam, dtype=torch.float32, device=dev),
                            "tree_codes": torch.empty(R, self.L, batch, beam, self.L, dtype=torch.int32, device=dev),
                            "tree_count": torch.empty(R, self.L, batch, dtype=torch.int32, device=dev)}
        return out

    @staticmethod
    def _trace_struct(out) -> Optional[NezhaTrace]:
        if "trace" not in out:
            return None
        t = out["trace"]
        return NezhaTrace(_ptr(t["drafts"]), _ptr(t["n_draft"]), _ptr(t["accepted_len"]), _ptr(t["level_reached"]),
                          _ptr(t["beams"]), _ptr(t["beam_scores"]), _ptr(t.get("tree_codes")), _ptr(t.get("tree_count")))

    def decode(self, beam: int, mode: int = MODE_VERIFIED, out=None, trace: bool = False, want_stats: bool = True):
        out = out if out is not None else self.alloc_outputs(self.batch, beam, trace)
        stats = NezhaDecodeStats()
        tr = self._trace_struct(out)
        self._check(lib.nezha_decode(self._h, self.batch, beam, mode, _ptr(out["codes"]), _ptr(out["scores"]),
                                     _ptr(out["count"]), C.byref(stats) if want_stats else None,
                                     C.byref(tr) if tr is not None else None))
        out["stats"] = stats
        return out

    def decode_with_drafts(self, beam: int, drafts: torch.Tensor, n_draft: torch.Tensor, out=None, trace: bool = False):
        out = out if out is not None else self.alloc_outputs(self.batch, beam, trace)
        stats = NezhaDecodeStats()
        tr = self._trace_struct(out)
        drafts, n_draft = drafts.contiguous(), n_draft.contiguous()
        self._check(lib.nezha_decode_with_drafts(self._h, self.batch, beam, _ptr(drafts), _ptr(n_draft),
                                                 _ptr(out["codes"]), _ptr(out["scores"]), _ptr(out["count"]),
                                                 C.byref(stats), C.byref(tr) if tr is not None else None))
        out["stats"] = stats
        return out

    def decode_with_draft_tree(self, beam: int, tree_codes: torch.Tensor, tree_count: torch.Tensor, out=None,
                               trace: bool = False):
        """tree_codes int32 [L, batch, beam, L], tree_count int32 [L, batch] (the layout of the trace's `beams`)."""
        out = out if out is not None else self.alloc_outputs(self.batch, beam, trace)
        stats = NezhaDecodeStats()
        tr = self._trace_struct(out)
        assert tuple(tree_codes.shape) == (self.L, self.batch, beam, self.L) and tree_codes.dtype == torch.int32
        assert tuple(tree_count.shape) == (self.L, self.batch) and tree_count.dtype == torch.int32
        tree_codes, tree_count = tree_codes.contiguous(), tree_count.contiguous()
        self._check(lib.nezha_decode_with_draft_tree(self._h, self.batch, beam, _ptr(tree_codes), _ptr(tree_count),
                                                     _ptr(out["codes"]), _ptr(out["scores"]), _ptr(out["count"]),
                                                     C.byref(stats), C.byref(tr) if tr is not None else None))
        out["stats"] = stats
        return out

    def set_option(self, option: int, value: int):
        self._check(lib.nezha_set_option(self._h, option, value))

    def get_hidden(self) -> torch.Tensor:
        h = torch.empty(self.batch, self.L + 1, self.cfg.d_model, dtype=torch.float32, device=self.arena.device)
        self._check(lib.nezha_get_hidden(self._h, _ptr(h)))
        return h

    def _stage_logits(self, fn, n_beams: int, level: int, prefixes: Optional[torch.Tensor]) -> torch.Tensor:
        out = torch.empty(self.batch, n_beams, self.T[level], dtype=torch.float32, device=self.arena.device)
        p = None if prefixes is None else prefixes.contiguous()
        self._check(fn(self._h, self.batch, n_beams, level, _ptr(p), _ptr(out)))
        return out

    def primary_logits(self, n_beams: int, level: int, prefixes: Optional[torch.Tensor] = None) -> torch.Tensor:
        return self._stage_logits(lib.nezha_primary_logits, n_beams, level, prefixes)

    def draft_logits(self, n_beams: int, level: int, prefixes: Optional[torch.Tensor] = None) -> torch.Tensor:
        return self._stage_logits(lib.nezha_draft_logits, n_beams, level, prefixes)

    def select(self, logits: torch.Tensor, beam_scores: torch.Tensor, beam_codes: Optional[torch.Tensor],
               n_live: torch.Tensor, beam: int, level: int, per_beam: int, filter: bool):
        batch, n_beams = int(logits.shape[0]), int(logits.shape[1])
        dev = logits.device
        parent = torch.empty(batch, beam, dtype=torch.int32, device=dev)
        code = torch.empty(batch, beam, dtype=torch.int32, device=dev)
        score = torch.empty(batch, beam, dtype=torch.float32, device=dev)
        count = torch.empty(batch, dtype=torch.int32, device=dev)
        bc = None if beam_codes is None else beam_codes.contiguous()
        self._check(lib.nezha_select(self._h, batch, n_beams, beam, level, per_beam, 1 if filter else 0,
                                     _ptr(logits.contiguous()), _ptr(beam_scores.contiguous()), _ptr(bc),
                                     _ptr(n_live.contiguous()), _ptr(parent), _ptr(code), _ptr(score), _ptr(count)))
        return parent, code, score, count

    def gemm(self, A: torch.Tensor, W: torch.Tensor, C_out: torch.Tensor, epilogue: int = 0,
             bias: Optional[torch.Tensor] = None, path: int = 0):
        M, K = A.shape
        N = W.shape[0]
        assert W.shape[1] == K and tuple(C_out.shape) == (M, N)
        self._check(lib.nezha_gemm(self._h, _ptr(A), _ptr(W), _ptr(C_out), M, N, K, epilogue, _ptr(bias), path))
        return C_out

    def profile_enable(self, on: bool):
        self._check(lib.nezha_profile_enable(self._h, 1 if on else 0))

    def profile_read(self) -> Dict[str, Dict[str, float]]:
        p = NezhaProfile()
        self._check(lib.nezha_profile_read(self._h, C.byref(p)))
        return {name: {"launches": int(p.launches[i]), "ms": float(p.ms[i])} for i, name in enumerate(PROFILE_CLASSES)}

    def sync(self):
        self._check(lib.nezha_sync(self._h))
