"""ctypes front end of the CPU oracle (oracle/spd_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU-baseline leg of
the benchmark.  It never imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, List, Sequence

import numpy as np
import torch

from . import build as _build

MAX_K = 16
MAX_ORD = 8


class OrcConfig(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("d_ffn", C.c_int32),
        ("vocab", C.c_int32), ("max_pos", C.c_int32),
        ("rms_eps", C.c_double), ("rope_theta", C.c_double),
        ("k", C.c_int32), ("n_min", C.c_int32), ("n_max", C.c_int32),
        ("lam", C.c_double * MAX_ORD),
        ("alpha", C.c_double), ("tau", C.c_double), ("delta", C.c_double),
        ("kv_dtype", C.c_int32), ("pad_", C.c_int32),
    ]


_PP = C.POINTER(C.c_void_p)


class OrcWeights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + [
        (n, _PP) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "wgate", "wup", "wdown")]


class OrcNgram(C.Structure):
    _fields_ = [("n", C.c_int32), ("pad_", C.c_int32), ("n_entries", C.c_int64),
                ("keys", C.c_void_p), ("counts", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        L = _lib
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(OrcConfig), C.POINTER(OrcWeights), C.POINTER(OrcNgram), C.c_int]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_step_forward.argtypes = [C.c_void_p]
        L.orc_step_score.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_step_commit.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_feed_token.argtypes = [C.c_void_p, C.c_int32]
        L.orc_set_logP.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_follow_cache.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_double, C.c_void_p, C.c_void_p]
        L.orc_follow_need.argtypes = [C.c_void_p]
        L.orc_follow_need.restype = C.c_double
        for name in ("orc_logits", "orc_trace", "orc_logP", "orc_gamma_now", "orc_cand_tok", "orc_cand_lp",
                     "orc_scores", "orc_png_last", "orc_cnt_last", "orc_tot_last", "orc_sel_last", "orc_drafts",
                     "orc_kcache", "orc_vcache"):
            getattr(L, name).restype = C.c_void_p
            getattr(L, name).argtypes = [C.c_void_p]
        L.orc_len.argtypes = [C.c_void_p]
        L.orc_T.argtypes = [C.c_void_p]
        L.orc_round_bf16.restype = C.c_float
        L.orc_round_bf16.argtypes = [C.c_float]
        L.orc_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_double, C.c_void_p]
        L.orc_rope.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_double]
        L.orc_attention_head.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
        L.orc_topk_logprob.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_double, C.c_void_p, C.c_void_p]
        L.orc_gamma.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
        L.orc_nucleus.restype = C.c_int32
        L.orc_nucleus.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_double, C.c_double, C.c_void_p]
        L.orc_ngram_counts.argtypes = [C.POINTER(OrcNgram), C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.orc_png.restype = C.c_double
        L.orc_png.argtypes = [C.POINTER(OrcConfig), C.POINTER(OrcNgram), C.c_int, C.c_void_p, C.c_int, C.c_int32,
                              C.c_void_p, C.c_void_p]
        L.orc_score_stage.argtypes = [C.POINTER(OrcConfig), C.POINTER(OrcNgram), C.c_int, C.c_void_p, C.c_int, C.c_int,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    return _lib


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """uint16 bit patterns of a bf16 tensor, as a host array."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def make_config(shape, k: int, orders: Sequence[int], lam: Sequence[float], alpha: float, tau: float, delta: float,
                max_pos: int, kv_dtype: str = "bf16", rms_eps: float = 1e-5, rope_theta: float = 10000.0) -> OrcConfig:
    c = OrcConfig()
    c.n_layers, c.d_model, c.n_heads, c.d_ffn, c.vocab = (shape.n_layers, shape.d_model, shape.n_heads, shape.d_ffn,
                                                           shape.vocab)
    c.max_pos, c.rms_eps, c.rope_theta = max_pos, rms_eps, rope_theta
    c.k = k
    c.n_min, c.n_max = (min(orders), max(orders)) if len(orders) else (2, 1)
    for i in range(MAX_ORD):
        c.lam[i] = float(lam[i]) if i < len(lam) else 0.0
    c.alpha, c.tau, c.delta = alpha, tau, delta
    c.kv_dtype = {"f32": 0, "bf16": 1}[kv_dtype]
    return c


class NgramTables:
    """Host copies of the frequency tables in the oracle's layout."""

    def __init__(self, tables: Sequence[Dict[str, object]]):
        self._keep: List[np.ndarray] = []
        self.n = len(tables)
        self.arr = (OrcNgram * max(1, self.n))()
        for i, t in enumerate(tables):
            keys = np.ascontiguousarray(np.asarray(t["keys"], dtype=np.int32))
            counts = np.ascontiguousarray(np.asarray(t["counts"], dtype=np.int64))
            self._keep += [keys, counts]
            self.arr[i].n = int(t["n"])
            self.arr[i].n_entries = counts.shape[0]
            self.arr[i].keys = _ptr(keys)
            self.arr[i].counts = _ptr(counts)


class Oracle:
    """One SPD decoding context on the CPU."""

    def __init__(self, cfg: OrcConfig, weights: Dict[str, object], tables: Sequence[Dict[str, object]]):
        self.cfg = cfg
        self.k = cfg.k
        self._keep: List[object] = []
        w = OrcWeights()
        for name in ("tok_emb", "final_norm", "lm_head"):
            a = bf16_bits(weights[name])
            self._keep.append(a)
            setattr(w, name, _ptr(a))
        for name in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "wgate", "wup", "wdown"):
            arrs = [bf16_bits(t) for t in weights[name]]
            ptrs = (C.c_void_p * len(arrs))(*[_ptr(a) for a in arrs])
            self._keep += [arrs, ptrs]
            setattr(w, name, C.cast(ptrs, _PP))
        self._w = w
        self.tables = NgramTables(tables)
        self.h = lib().orc_create(C.byref(cfg), C.byref(w), self.tables.arr, self.tables.n)
        if not self.h:
            raise ValueError("orc_create rejected the configuration")

    def close(self) -> None:
        if self.h:
            lib().orc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- procedure ----
    def prefill(self, ids: Sequence[int]):
        a = np.asarray(ids, dtype=np.int32)
        out = np.zeros(self.k, np.int32)
        g = np.zeros(self.k, np.float64)
        if lib().orc_prefill(self.h, _ptr(a), len(a), _ptr(out), _ptr(g)):
            raise ValueError("orc_prefill: bad arguments")
        return out, g

    def reset(self, draft: int):
        """Section 5.3: generation restarts from one draft.  By definition: the first timestep on the prefix
        followed by that draft's tokens, everything recomputed from scratch."""
        return self.prefill(self.drafts()[int(draft)].tolist())

    def step(self):
        ids = np.zeros(self.k, np.int32)
        par = np.zeros(self.k, np.int32)
        g = np.zeros(self.k, np.float64)
        if lib().orc_step(self.h, _ptr(ids), _ptr(par), _ptr(g)):
            raise ValueError("orc_step: out of positions")
        return ids, par, g

    def generate(self, max_steps: int, eos_id: int = -1) -> int:
        """Algorithm 1's loop, "until max generation length or stop token": steps until max_steps are taken or the
        most probable draft (drafts are ordered by probability) has just emitted eos_id.  The paper does not say
        which draft's token counts; the most probable one is this implementation's reading.  Returns the steps taken."""
        for n in range(max_steps):
            ids, _, _ = self.step()
            if eos_id >= 0 and int(ids[0]) == eos_id:
                return n + 1
        return max_steps

    def step_forward(self) -> None:
        if lib().orc_step_forward(self.h):
            raise ValueError("orc_step_forward: out of positions")

    def step_score(self):
        nl = np.zeros(self.k, np.float64)
        ng = np.zeros(self.k, np.float64)
        lib().orc_step_score(self.h, _ptr(nl), _ptr(ng))
        return self.sel().copy(), nl, ng

    def step_commit(self, sel: Sequence[int], new_logP: Sequence[float]) -> None:
        s = np.asarray(sel, dtype=np.int32)
        nl = np.asarray(new_logP, dtype=np.float64)
        lib().orc_step_commit(self.h, _ptr(s), _ptr(nl))

    def set_logP(self, logP) -> None:
        a = np.ascontiguousarray(logP, dtype=np.float64)
        lib().orc_set_logP(self.h, _ptr(a))

    def follow_cache(self, k=None, v=None, slack: float = 0.0):
        """Follow the given cache contents (float32 [L, T, d]) in later passes; returns (adopted, refused)
        counts accumulated since the previous call.  slack = absolute float error allowed for the other side.
        `follow_need` then holds the largest slack any adopted value needed over that period."""
        flips, bad = C.c_int64(), C.c_int64()
        self.follow_need = float(lib().orc_follow_need(self.h))
        if k is None:
            self._fk = self._fv = None
            lib().orc_follow_cache(self.h, None, None, 0, 0.0, C.byref(flips), C.byref(bad))
        else:
            self._fk = np.ascontiguousarray(k, dtype=np.float32)
            self._fv = np.ascontiguousarray(v, dtype=np.float32)
            lib().orc_follow_cache(self.h, _ptr(self._fk), _ptr(self._fv), self._fk.shape[1], float(slack), C.byref(flips),
                                   C.byref(bad))
        return flips.value, bad.value

    def feed_token(self, tok: int) -> None:
        if lib().orc_feed_token(self.h, int(tok)):
            raise ValueError("orc_feed_token: bad token or out of positions")

    # ---- read-outs ----
    def _view(self, fn: str, dtype, count: int) -> np.ndarray:
        p = getattr(lib(), fn)(self.h)
        return np.ctypeslib.as_array(C.cast(p, C.POINTER(np.ctypeslib.as_ctypes_type(dtype))), shape=(count,))

    def logits(self) -> np.ndarray:
        return self._view("orc_logits", np.float64, self.cfg.vocab).copy()

    def trace(self) -> np.ndarray:
        return self._view("orc_trace", np.float64, self.cfg.n_layers * 2 * self.cfg.d_model).reshape(
            self.cfg.n_layers, 2, self.cfg.d_model).copy()

    def logP(self) -> np.ndarray:
        return self._view("orc_logP", np.float64, MAX_K)[: self.k].copy()

    def gamma(self) -> np.ndarray:
        return self._view("orc_gamma_now", np.float64, MAX_K)[: self.k].copy()

    def cand_tok(self) -> np.ndarray:
        return self._view("orc_cand_tok", np.int32, MAX_K)[: self.k].copy()

    def cand_lp(self) -> np.ndarray:
        return self._view("orc_cand_lp", np.float64, MAX_K)[: self.k].copy()

    def scores(self) -> np.ndarray:
        return self._view("orc_scores", np.float64, MAX_K * MAX_K)[: self.k * self.k].copy()

    def png(self) -> np.ndarray:
        return self._view("orc_png_last", np.float64, MAX_K * MAX_K)[: self.k * self.k].copy()

    def counts(self) -> np.ndarray:
        """[k*k, n_tables] n-gram counts used by the last scoring stage (-1 = order skipped)."""
        a = self._view("orc_cnt_last", np.int64, MAX_K * MAX_K * MAX_ORD).reshape(MAX_K * MAX_K, MAX_ORD)
        return a[: self.k * self.k, : self.tables.n].copy()

    def totals(self) -> np.ndarray:
        """[k, n_tables] context totals used by the last scoring stage."""
        a = self._view("orc_tot_last", np.int64, MAX_K * MAX_ORD).reshape(MAX_K, MAX_ORD)
        return a[: self.k, : self.tables.n].copy()

    def sel(self) -> np.ndarray:
        return self._view("orc_sel_last", np.int32, MAX_K)[: self.k]

    def length(self) -> int:
        return lib().orc_len(self.h)

    def T(self) -> int:
        return lib().orc_T(self.h)

    def drafts(self) -> np.ndarray:
        a = self._view("orc_drafts", np.int32, self.k * self.cfg.max_pos).reshape(self.k, self.cfg.max_pos)
        return a[:, : self.length()].copy()

    def kv_cache(self):
        n = self.cfg.n_layers * self.cfg.max_pos * self.cfg.d_model
        shp = (self.cfg.n_layers, self.cfg.max_pos, self.cfg.d_model)
        return (self._view("orc_kcache", np.float32, n).reshape(shp), self._view("orc_vcache", np.float32, n).reshape(shp))


# ---- stand-alone stages (pure functions of their arguments) ----

def score_stage(cfg: OrcConfig, tables: NgramTables, hist: np.ndarray, logP, cand_tok, cand_lp):
    """Scoring stage on explicit inputs.  hist: int32 [k, hist_len].  Returns a dict of all outputs."""
    k = cfg.k
    hist = np.ascontiguousarray(hist, dtype=np.int32)
    logP = np.ascontiguousarray(logP, dtype=np.float64)
    cand_tok = np.ascontiguousarray(cand_tok, dtype=np.int32)
    cand_lp = np.ascontiguousarray(cand_lp, dtype=np.float64)
    png = np.zeros(k * k)
    score = np.zeros(k * k)
    cnt = np.zeros((k * k, MAX_ORD), np.int64)
    tot = np.zeros((k, MAX_ORD), np.int64)
    sel = np.zeros(k, np.int32)
    nl = np.zeros(k)
    ng = np.zeros(k)
    lib().orc_score_stage(C.byref(cfg), tables.arr, tables.n, _ptr(hist), hist.shape[1], hist.shape[1], _ptr(logP),
                          _ptr(cand_tok), _ptr(cand_lp), _ptr(png), _ptr(score), _ptr(cnt), _ptr(tot), _ptr(sel),
                          _ptr(nl), _ptr(ng))
    return {"png": png, "score": score, "cnt": cnt[:, : tables.n], "tot": tot[:, : tables.n], "sel": sel,
            "logP": nl, "gamma": ng}


def topk_logprob(z: np.ndarray, k: int, tau: float):
    z = np.ascontiguousarray(z, dtype=np.float64)
    tok = np.zeros(k, np.int32)
    lp = np.zeros(k, np.float64)
    lib().orc_topk_logprob(_ptr(z), z.shape[0], k, tau, _ptr(tok), _ptr(lp))
    return tok, lp


def nucleus(z: np.ndarray, temperature: float, p: float, u: float):
    """Nucleus sampling of one token from logits z: (token, {size, mass, gap_cut, gap_draw})."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    info = np.zeros(4, np.float64)
    tok = lib().orc_nucleus(_ptr(z), z.shape[0], float(temperature), float(p), float(u), _ptr(info))
    return int(tok), {"size": int(info[0]), "mass": float(info[1]), "gap_cut": float(info[2]), "gap_draw": float(info[3])}


def max_threads() -> int:
    return lib().orc_max_threads()
