"""ctypes binding of include/spd.h.  Names follow the C ABI; no arithmetic of the method lives here."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import build as _build

MAX_K = 16
MAX_ORDERS = 8

DBG = {name: i for i, name in enumerate(
    ["LOGITS", "CAND_TOK", "CAND_LP", "LOGP_IN", "SCORE", "PNG", "CNT", "TOT", "SEL", "LOGP", "HIST_IN", "TRACE",
     "HIDDEN", "KCACHE", "VCACHE"])}

_STATUS = {0: "SPD_OK", -1: "SPD_EINVAL", -2: "SPD_ESTATE", -3: "SPD_ERANGE", -4: "SPD_ENOMEM", -5: "SPD_ECUDA",
           -6: "SPD_ETABLE", -7: "SPD_ETIMEOUT"}


def status_name(rc: int) -> str:
    return _STATUS.get(rc, "SPD_E?(%d)" % rc)


class SpdError(RuntimeError):
    def __init__(self, rc: int, what: str):
        lib = load_library()
        msg = "%s: %s (%s)" % (what, status_name(rc), lib.spd_strerror(rc).decode())
        if rc == -5:
            msg += ": " + lib.spd_last_cuda_error().decode()
        super().__init__(msg)
        self.status = rc


class SpdConfig(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("d_ffn", C.c_int32),
        ("vocab", C.c_int32), ("max_pos", C.c_int32),
        ("rms_eps", C.c_float), ("rope_theta", C.c_float),
        ("k", C.c_int32), ("n_min", C.c_int32), ("n_max", C.c_int32),
        ("lam", C.c_float * MAX_ORDERS),
        ("alpha", C.c_float), ("tau", C.c_float), ("delta", C.c_float),
        ("eos_id", C.c_int32), ("kv_dtype", C.c_int32),
        ("stream", C.c_void_p),
    ]


_PP = C.POINTER(C.c_void_p)


class _Weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + [
        (n, _PP) for n in ("attn_norm", "wqkv", "wo", "ffn_norm", "wgate_up", "wdown")] + [("lm_head_img", C.c_void_p)] + [
        (n, _PP) for n in ("wqkv_img", "wo_img", "wgate_up_img")]


class _Table(C.Structure):
    _fields_ = [("n", C.c_int32), ("reserved", C.c_int32), ("ngram_slots", C.c_uint64), ("ctx_slots", C.c_uint64),
                ("ngram", C.c_void_p), ("ctx", C.c_void_p)]


_lib: Optional[C.CDLL] = None

EXPORTS = ["spd_workspace_bytes", "spd_create", "spd_prefill", "spd_step", "spd_generate", "spd_generate_async",
           "spd_sync", "spd_destroy", "spd_strerror", "spd_last_cuda_error", "spd_ngram_plan", "spd_ngram_build",
           "spd_debug_read", "spd_debug_score", "spd_launch_count", "spd_set_ring", "spd_score_static", "spd_reset",
           "spd_sample", "spd_debug_nucleus", "spd_debug_expire", "spd_debug_expire_products", "spd_debug_trace", "spd_finished", "spd_batch_generate", "spd_batch_step", "spd_pack_image", "spd_ring_plan"]


def load_library() -> C.CDLL:
    """Loads libspd.so, building it first when its sources are newer (the environment variable
    SPD_LIBRARY names another build of the library to load instead).  Raises if neither is possible."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("SPD_LIBRARY", "")
    if not path:
        path = _build.LIB
        try:
            path = _build.build()
        except Exception as exc:  # no compiler on this machine: the prebuilt library must be there
            if not os.path.exists(path):
                raise RuntimeError("libspd.so is missing and could not be built: %s" % exc) from exc
    L = C.CDLL(path)
    L.spd_workspace_bytes.argtypes = [C.POINTER(SpdConfig), C.POINTER(C.c_size_t)]
    L.spd_create.argtypes = [C.POINTER(SpdConfig), C.POINTER(_Weights), C.POINTER(_Table), C.c_int32, C.c_void_p,
                             C.c_size_t, C.POINTER(C.c_void_p)]
    L.spd_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    L.spd_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    L.spd_reset.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    L.spd_sample.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    L.spd_generate.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    L.spd_generate_async.argtypes = [C.c_void_p, C.c_int32]
    L.spd_sync.argtypes = [C.c_void_p]
    L.spd_destroy.argtypes = [C.c_void_p]
    L.spd_strerror.restype = C.c_char_p
    L.spd_strerror.argtypes = [C.c_int]
    L.spd_last_cuda_error.restype = C.c_char_p
    L.spd_ngram_plan.argtypes = [C.c_int32, C.c_int64, C.c_void_p, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    L.spd_ngram_build.argtypes = [C.c_int32, C.c_int64, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64,
                                  C.c_void_p]
    L.spd_debug_read.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_size_t]
    L.spd_debug_score.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    L.spd_debug_nucleus.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_float, C.c_float, C.c_void_p]
    L.spd_debug_expire.argtypes = [C.c_void_p]
    L.spd_debug_trace.argtypes = [C.c_void_p, C.c_int]
    L.spd_finished.argtypes = [C.c_void_p]
    L.spd_batch_generate.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
    L.spd_batch_step.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    L.spd_debug_expire_products.argtypes = [C.c_void_p]
    L.spd_pack_image.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    L.spd_ring_plan.argtypes = [C.POINTER(SpdConfig), C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    L.spd_launch_count.restype = C.c_int64
    L.spd_launch_count.argtypes = [C.c_void_p]
    L.spd_set_ring.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
    L.spd_score_static.argtypes = [C.POINTER(SpdConfig), C.POINTER(_Table), C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    _lib = L
    return L


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise SpdError(rc, what)


def spd_ngram_build_host(table: Dict[str, object]):
    """spd_ngram_plan + spd_ngram_build for one frequency table {'n', 'keys' [N,n], 'counts' [N]}.
    Returns (ngram_slots, ctx_slots, ngram image uint8 tensor, ctx image uint8 tensor) on the host."""
    L = load_library()
    n = int(table["n"])
    keys = np.ascontiguousarray(np.asarray(table["keys"], dtype=np.int32))
    counts = np.ascontiguousarray(np.asarray(table["counts"], dtype=np.int64))
    ne = counts.shape[0]
    ns, cs = C.c_uint64(), C.c_uint64()
    _check(L.spd_ngram_plan(n, ne, keys.ctypes.data, C.byref(ns), C.byref(cs)), "spd_ngram_plan")
    ng = torch.empty(ns.value * 16, dtype=torch.uint8)
    cx = torch.empty(cs.value * 16, dtype=torch.uint8)
    _check(L.spd_ngram_build(n, ne, keys.ctypes.data, counts.ctypes.data, ns.value, ng.data_ptr(), cs.value,
                             cx.data_ptr()), "spd_ngram_build")
    return ns.value, cs.value, ng, cx


def build_ngram_tables(tables: Sequence[Dict[str, object]], device: str | torch.device = "cuda:0") -> List[Dict[str, object]]:
    """Hash-table images of the given frequency tables, uploaded to `device` (ascending order n)."""
    out = []
    for t in sorted(tables, key=lambda t: int(t["n"])):
        ns, cs, ng, cx = spd_ngram_build_host(t)
        out.append({"n": int(t["n"]), "ngram_slots": ns, "ctx_slots": cs, "ngram": ng.to(device), "ctx": cx.to(device)})
    return out


def _image(t: torch.Tensor) -> Optional[torch.Tensor]:
    """Fragment-order image of a bf16 matrix (spd_pack_image), or None when its shape does not divide."""
    rows, cols = t.shape
    if rows % 8 or cols % 32 or t.dtype != torch.bfloat16:
        return None
    out = torch.empty_like(t)
    with torch.cuda.device(t.device):
        _check(load_library().spd_pack_image(t.data_ptr(), rows, cols, out.data_ptr(), torch.cuda.current_stream(t.device).cuda_stream),
               "spd_pack_image")
    return out


def pack_weights(weights: Dict[str, object], device: str | torch.device = "cuda:0", consume: bool = False,
                 images: bool = True) -> Dict[str, object]:
    """Lays the decoder's tensors out as spd_weights wants them, on `device`: wqkv = rows of W_q, W_k,
    W_v stacked; wgate_up = gate and up rows interleaved.  With consume=True the per-layer inputs are
    dropped from `weights` as they are packed (halves peak memory).  images=True adds the fragment-order
    images of lm_head, wqkv, wo and wgate_up that let the decode timesteps use the tensor cores (all four or
    none: shapes that do not divide leave them out)."""
    dev = torch.device(device)
    out: Dict[str, object] = {k: weights[k].to(dev).contiguous() for k in ("tok_emb", "final_norm", "lm_head")}
    for k in ("attn_norm", "wqkv", "wo", "ffn_norm", "wgate_up", "wdown"):
        out[k] = []
    n_layers = len(weights["wq"])
    for l in range(n_layers):
        out["attn_norm"].append(weights["attn_norm"][l].to(dev).contiguous())
        out["ffn_norm"].append(weights["ffn_norm"][l].to(dev).contiguous())
        out["wqkv"].append(torch.cat([weights["wq"][l].to(dev), weights["wk"][l].to(dev), weights["wv"][l].to(dev)], 0).contiguous())
        out["wo"].append(weights["wo"][l].to(dev).contiguous())
        g, u = weights["wgate"][l].to(dev), weights["wup"][l].to(dev)
        out["wgate_up"].append(torch.stack([g, u], 1).reshape(2 * g.shape[0], g.shape[1]).contiguous())
        out["wdown"].append(weights["wdown"][l].to(dev).contiguous())
        if consume:
            for k in ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown"):
                weights[k][l] = None
    if images and dev.type == "cuda":
        img: Dict[str, object] = {"lm_head_img": _image(out["lm_head"])}
        for k in ("wqkv", "wo", "wgate_up"):
            img[k + "_img"] = [_image(t) for t in out[k]]
        if img["lm_head_img"] is not None and all(t is not None for k in ("wqkv", "wo", "wgate_up") for t in img[k + "_img"]):
            out.update(img)
    return out


class SpdContext:
    """One decoding context (spd_create ... spd_destroy).  `packed` comes from pack_weights, `tables`
    from build_ngram_tables; both must live on the context's device."""

    def __init__(self, shape, packed: Dict[str, object], tables: Sequence[Dict[str, object]], k: int,
                 orders: Sequence[int], lam: Sequence[float], alpha: float, tau: float, delta: float, max_pos: int,
                 kv_dtype: str = "bf16", rms_eps: float = 1e-5, rope_theta: float = 10000.0,
                 stream: Optional[torch.cuda.Stream] = None, eos_id: int = -1):
        L = load_library()
        self.lib = L
        self.k = k
        self.shape = shape
        self.device = packed["tok_emb"].device
        if self.device.type != "cuda":
            raise RuntimeError("SpdContext needs CUDA tensors; there is no CPU path")
        cfg = SpdConfig()
        cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.d_ffn, cfg.vocab = (shape.n_layers, shape.d_model, shape.n_heads,
                                                                        shape.d_ffn, shape.vocab)
        cfg.max_pos, cfg.rms_eps, cfg.rope_theta, cfg.k = max_pos, rms_eps, rope_theta, k
        cfg.n_min, cfg.n_max = (min(orders), max(orders)) if len(orders) else (2, 2)
        for i in range(MAX_ORDERS):
            cfg.lam[i] = float(lam[i]) if i < len(lam) else 0.0
        cfg.alpha, cfg.tau, cfg.delta, cfg.eos_id = alpha, tau, delta, eos_id
        cfg.kv_dtype = {"f32": 0, "bf16": 1}[kv_dtype]
        self.stream = stream
        cfg.stream = stream.cuda_stream if stream is not None else None
        self.cfg = cfg
        self._keep: List[object] = [packed, tables]
        w = _Weights()
        for name in ("tok_emb", "final_norm", "lm_head"):
            setattr(w, name, packed[name].data_ptr())
        for name in ("attn_norm", "wqkv", "wo", "ffn_norm", "wgate_up", "wdown"):
            arr = (C.c_void_p * shape.n_layers)(*[t.data_ptr() for t in packed[name]])
            self._keep.append(arr)
            setattr(w, name, C.cast(arr, _PP))
        if "lm_head_img" in packed:
            w.lm_head_img = packed["lm_head_img"].data_ptr()
            for name in ("wqkv_img", "wo_img", "wgate_up_img"):
                arr = (C.c_void_p * shape.n_layers)(*[t.data_ptr() for t in packed[name]])
                self._keep.append(arr)
                setattr(w, name, C.cast(arr, _PP))
        tabs = (_Table * max(1, len(tables)))()
        for i, t in enumerate(tables):
            tabs[i].n, tabs[i].ngram_slots, tabs[i].ctx_slots = t["n"], t["ngram_slots"], t["ctx_slots"]
            tabs[i].ngram, tabs[i].ctx = t["ngram"].data_ptr(), t["ctx"].data_ptr()
        nbytes = C.c_size_t()
        _check(L.spd_workspace_bytes(C.byref(cfg), C.byref(nbytes)), "spd_workspace_bytes")
        self.workspace = torch.empty(nbytes.value, dtype=torch.uint8, device=self.device)
        self.h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(L.spd_create(C.byref(cfg), C.byref(w), tabs, len(tables), self.workspace.data_ptr(), nbytes.value,
                                C.byref(self.h)), "spd_create")

    def close(self) -> None:
        if getattr(self, "h", None):
            self.lib.spd_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def spd_prefill(self, prefix_ids: Sequence[int]):
        a = np.ascontiguousarray(np.asarray(prefix_ids, dtype=np.int32))
        ids = np.zeros(self.k, np.int32)
        g = np.zeros(self.k, np.float32)
        _check(self.lib.spd_prefill(self.h, a.ctypes.data, a.shape[0], ids.ctypes.data, g.ctypes.data), "spd_prefill")
        return ids, g

    def spd_reset(self, draft: int):
        ids = np.zeros(self.k, np.int32)
        g = np.zeros(self.k, np.float32)
        _check(self.lib.spd_reset(self.h, int(draft), ids.ctypes.data, g.ctypes.data), "spd_reset")
        return ids, g

    def spd_debug_trace(self, on: bool) -> None:
        _check(self.lib.spd_debug_trace(self.h, 1 if on else 0), "spd_debug_trace")

    def spd_debug_expire(self) -> int:
        """Status the device recorded when one block withheld its barrier arrival (SPD_ETIMEOUT = -7)."""
        return int(self.lib.spd_debug_expire(self.h))

    def spd_debug_expire_products(self) -> int:
        """Status the device recorded when a stage of the long-prefix products never arrived (SPD_ETIMEOUT = -7)."""
        return int(self.lib.spd_debug_expire_products(self.h))

    def spd_debug_nucleus(self, logits, top_p: float, temperature: float, u: float) -> int:
        z = np.ascontiguousarray(logits, dtype=np.float32)
        assert z.shape == (self.shape.vocab,)
        tok = C.c_int32(-1)
        _check(self.lib.spd_debug_nucleus(self.h, z.ctypes.data, float(top_p), float(temperature), float(u), C.byref(tok)),
               "spd_debug_nucleus")
        return int(tok.value)

    def spd_sample(self, uniforms, top_p: float, temperature: float):
        """Extends the prefix by len(uniforms) nucleus-sampled tokens, then the first timestep: (new ids, ids, gamma)."""
        u = np.ascontiguousarray(uniforms, dtype=np.float32)
        new = np.zeros(u.shape[0], np.int32)
        ids = np.zeros(self.k, np.int32)
        g = np.zeros(self.k, np.float32)
        _check(self.lib.spd_sample(self.h, int(u.shape[0]), float(top_p), float(temperature), u.ctypes.data,
                                   new.ctypes.data, ids.ctypes.data, g.ctypes.data), "spd_sample")
        return new, ids, g

    def spd_step(self):
        ids = np.zeros(self.k, np.int32)
        par = np.zeros(self.k, np.int32)
        g = np.zeros(self.k, np.float32)
        _check(self.lib.spd_step(self.h, ids.ctypes.data, par.ctypes.data, g.ctypes.data), "spd_step")
        return ids, par, g

    def spd_generate(self, n_steps: int, total_len: int):
        """total_len = tokens per draft after the call (tokens so far + n_steps); fewer come back when the stop
        token ended the run early."""
        toks = np.zeros(self.k * total_len, np.int32)
        ln = C.c_int32()
        lp = np.zeros(self.k, np.float32)
        g = np.zeros(self.k, np.float32)
        _check(self.lib.spd_generate(self.h, n_steps, toks.ctypes.data, C.byref(ln), lp.ctypes.data, g.ctypes.data),
               "spd_generate")
        assert ln.value == total_len or (self.cfg.eos_id >= 0 and ln.value < total_len), (ln.value, total_len)
        return toks[: self.k * ln.value].reshape(self.k, ln.value).copy(), lp, g

    def spd_finished(self) -> bool:
        return bool(self.lib.spd_finished(self.h))

    def spd_generate_async(self, n_steps: int) -> None:
        _check(self.lib.spd_generate_async(self.h, n_steps), "spd_generate_async")

    def spd_sync(self) -> None:
        _check(self.lib.spd_sync(self.h), "spd_sync")

    def spd_set_ring(self, stage_bytes: int, n_stages: int) -> None:
        _check(self.lib.spd_set_ring(self.h, stage_bytes, n_stages), "spd_set_ring")

    def spd_launch_count(self) -> int:
        return int(self.lib.spd_launch_count(self.h))

    def spd_debug_read(self, what: str, positions: int = 0) -> np.ndarray:
        """`positions` (KCACHE / VCACHE only) = cached positions so far: prefix length + tokens generated - 1."""
        k, c = self.k, self.cfg
        shapes = {"LOGITS": (np.float32, (c.vocab,)), "CAND_TOK": (np.int32, (k,)), "CAND_LP": (np.float32, (k,)),
                  "LOGP_IN": (np.float32, (k,)), "SCORE": (np.float32, (k * k,)), "PNG": (np.float32, (k * k,)),
                  "CNT": (np.uint32, (k * k, 8)), "TOT": (np.uint32, (k, 8)), "SEL": (np.int32, (k,)),
                  "LOGP": (np.float32, (k,)), "HIST_IN": (np.int32, (k, 8)),
                  "TRACE": (np.float32, (c.n_layers, 2, c.d_model)), "HIDDEN": (np.float32, (c.d_model,))}
        if what in ("KCACHE", "VCACHE"):
            shapes[what] = (np.float32, (c.n_layers, int(positions), c.d_model))
        dt, shp = shapes[what]
        out = np.zeros(shp, dt)
        _check(self.lib.spd_debug_read(self.h, DBG[what], out.ctypes.data, out.nbytes), "spd_debug_read")
        if what in ("CNT", "TOT"):      # unsigned 32-bit on the device, 0xffffffff = order skipped: as int64 with -1
            wide = out.astype(np.int64)
            wide[out == np.uint32(0xffffffff)] = -1
            return wide
        return out

    def spd_debug_score(self, hist: np.ndarray, logp, cand_tok, cand_lp) -> None:
        hist = np.ascontiguousarray(hist, dtype=np.int32)
        logp = np.ascontiguousarray(logp, dtype=np.float32)
        cand_tok = np.ascontiguousarray(cand_tok, dtype=np.int32)
        cand_lp = np.ascontiguousarray(cand_lp, dtype=np.float32)
        _check(self.lib.spd_debug_score(self.h, hist.ctypes.data, hist.shape[1], logp.ctypes.data, cand_tok.ctypes.data,
                                        cand_lp.ctypes.data), "spd_debug_score")


def _ctx_array(ctxs: Sequence["SpdContext"]):
    return (C.c_void_p * len(ctxs))(*[c.h for c in ctxs])


def spd_batch_generate(ctxs: Sequence["SpdContext"], n_steps: int) -> None:
    """n_steps timesteps of all the contexts together, one pass over the weights per timestep."""
    _check(load_library().spd_batch_generate(_ctx_array(ctxs), len(ctxs), n_steps), "spd_batch_generate")


def spd_batch_step(ctxs: Sequence["SpdContext"]):
    """One timestep of all the contexts together.  Returns per context (ids, parents, gamma) as spd_step does."""
    n = len(ctxs)
    ids = np.zeros((n, MAX_K), np.int32)
    par = np.zeros((n, MAX_K), np.int32)
    g = np.zeros((n, MAX_K), np.float32)
    _check(load_library().spd_batch_step(_ctx_array(ctxs), n, ids.ctypes.data, par.ctypes.data, g.ctypes.data), "spd_batch_step")
    return [(ids[r, : c.k].copy(), par[r, : c.k].copy(), g[r, : c.k].copy()) for r, c in enumerate(ctxs)]


def spd_score_static(k: int, vocab: int, orders: Sequence[int], lam: Sequence[float], alpha: float, delta: float,
                     tables: Sequence[Dict[str, object]], hist: np.ndarray, logp, cand_tok, cand_lp,
                     stream: Optional[torch.cuda.Stream] = None):
    """Scoring stage through the entry point that allocates nothing on the device (for callers that
    have device pointers but no allocator to obtain a workspace from).  `tables` come from
    build_ngram_tables and live on the current CUDA device.  Returns (sel, logp, gamma, score)."""
    L = load_library()
    cfg = SpdConfig()
    cfg.k, cfg.vocab = k, vocab
    cfg.n_min, cfg.n_max = (min(orders), max(orders)) if len(orders) else (2, 2)
    for i in range(MAX_ORDERS):
        cfg.lam[i] = float(lam[i]) if i < len(lam) else 0.0
    cfg.alpha, cfg.delta = alpha, delta
    cfg.stream = stream.cuda_stream if stream is not None else None
    tabs = (_Table * max(1, len(tables)))()
    for i, t in enumerate(tables):
        tabs[i].n, tabs[i].ngram_slots, tabs[i].ctx_slots = t["n"], t["ngram_slots"], t["ctx_slots"]
        tabs[i].ngram, tabs[i].ctx = t["ngram"].data_ptr(), t["ctx"].data_ptr()
    hist = np.ascontiguousarray(hist, dtype=np.int32)
    logp = np.ascontiguousarray(logp, dtype=np.float32)
    cand_tok = np.ascontiguousarray(cand_tok, dtype=np.int32)
    cand_lp = np.ascontiguousarray(cand_lp, dtype=np.float32)
    kk = max(1, min(k, MAX_K))
    sel = np.zeros(kk, np.int32)
    out_lp = np.zeros(kk, np.float32)
    gamma = np.zeros(kk, np.float32)
    score = np.zeros(kk * kk, np.float32)
    _check(L.spd_score_static(C.byref(cfg), tabs, len(tables), hist.ctypes.data, hist.shape[1], logp.ctypes.data,
                              cand_tok.ctypes.data, cand_lp.ctypes.data, sel.ctypes.data, out_lp.ctypes.data,
                              gamma.ctypes.data, score.ctypes.data), "spd_score_static")
    return sel, out_lp, gamma, score
