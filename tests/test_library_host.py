"""Host-side checks of the CUDA library that need no GPU: exported symbols, argument checks, table images."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import spd_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import paper_2405_18400_b200 as P
    return P.load_library()


def test_library_exports_every_declared_symbol(lib):
    hdr = open(os.path.join(ROOT, "include", "spd.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(spd_[a-z_0-9]+)\s*\(", hdr))
    assert {"spd_create", "spd_prefill", "spd_step", "spd_generate", "spd_workspace_bytes", "spd_destroy"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), n


def _cfg(**kw):
    from paper_2405_18400_b200 import SpdConfig
    c = SpdConfig()
    c.n_layers, c.d_model, c.n_heads, c.d_ffn, c.vocab, c.max_pos = 2, 256, 4, 688, 4096, 64
    c.rms_eps, c.rope_theta, c.k, c.n_min, c.n_max = 1e-5, 10000.0, 3, 2, 4
    c.alpha, c.tau, c.delta, c.eos_id, c.kv_dtype = 0.5, 0.1, 0.01, -1, 1
    for k, v in kw.items():
        setattr(c, k, v)
    return c


def test_workspace_bytes_and_config_checks(lib):
    n = C.c_size_t()
    assert lib.spd_workspace_bytes(C.byref(_cfg()), C.byref(n)) == 0
    kv = 2 * 2 * 64 * 256 * 2
    assert kv < n.value < kv + (4 << 20)
    n32 = C.c_size_t()
    assert lib.spd_workspace_bytes(C.byref(_cfg(kv_dtype=0)), C.byref(n32)) == 0 and n32.value - n.value == kv
    bad = [dict(k=0), dict(k=17), dict(vocab=70000), dict(d_model=250), dict(n_heads=3), dict(n_heads=16),
           dict(n_min=1), dict(n_max=7), dict(tau=0.0), dict(delta=0.0), dict(delta=1.5), dict(alpha=1.5),
           dict(eos_id=-2), dict(eos_id=4096), dict(kv_dtype=2), dict(max_pos=1), dict(d_ffn=20000)]
    for kw in bad:
        assert lib.spd_workspace_bytes(C.byref(_cfg(**kw)), C.byref(n)) == -1, kw
    assert lib.spd_workspace_bytes(None, C.byref(n)) == -1
    assert lib.spd_strerror(-7) == b"bounded device wait expired" and lib.spd_strerror(0) == b"ok"


def _unpack(img):
    a = img.numpy().view(np.uint32).reshape(-1, 4)
    used = a[a[:, 3] > 0]
    toks = np.stack([used[:, 0] & 0xffff, used[:, 0] >> 16, used[:, 1] & 0xffff, used[:, 1] >> 16,
                     used[:, 2] & 0xffff, used[:, 2] >> 16], 1)
    return toks, used[:, 3]


def test_ngram_images_hold_every_entry_and_every_context_total(tiny_inputs):
    from paper_2405_18400_b200.binding import spd_ngram_build_host
    wl, weights, tables, prefix = tiny_inputs
    for t in tables:
        n = int(t["n"])
        ns, cs, ng, cx = spd_ngram_build_host(t)
        assert ns >= 2 * 20000 and ns & (ns - 1) == 0 and cs & (cs - 1) == 0
        toks, cnt = _unpack(ng)
        assert np.all(toks[:, n:] == 0)
        got = {tuple(r[:n]): int(c) for r, c in zip(toks.tolist(), cnt.tolist())}
        want = {tuple(r): int(c) for r, c in zip(t["keys"].tolist(), t["counts"].tolist())}
        assert got == want
        totals = {}
        for key, c in want.items():
            totals[key[:-1]] = totals.get(key[:-1], 0) + c
        toks, cnt = _unpack(cx)
        assert {tuple(r[: n - 1]): int(c) for r, c in zip(toks.tolist(), cnt.tolist())} == totals
        assert cs >= 2 * len(totals)


def test_ngram_build_rejects_bad_input(lib):
    ns, cs = C.c_uint64(), C.c_uint64()
    keys = np.array([[1, 2], [1, 2]], np.int32)
    assert lib.spd_ngram_plan(2, 2, keys.ctypes.data, C.byref(ns), C.byref(cs)) == -1       # not strictly increasing
    keys = np.array([[1, 3], [1, 2]], np.int32)
    assert lib.spd_ngram_plan(2, 2, keys.ctypes.data, C.byref(ns), C.byref(cs)) == -1
    keys = np.array([[1, 70000]], np.int32)
    assert lib.spd_ngram_plan(2, 1, keys.ctypes.data, C.byref(ns), C.byref(cs)) == -3       # token id above 65535
    assert lib.spd_ngram_plan(7, 0, None, C.byref(ns), C.byref(cs)) == -1
    keys = np.array([[1, 2], [1, 5], [2, 0]], np.int32)
    cnt = np.array([3, 1 << 33, 1], np.int64)
    assert lib.spd_ngram_plan(2, 3, keys.ctypes.data, C.byref(ns), C.byref(cs)) == 0 and (ns.value, cs.value) == (16, 16)
    buf = np.zeros(16 * 16, np.uint8)
    buf2 = np.zeros(16 * 16, np.uint8)
    assert lib.spd_ngram_build(2, 3, keys.ctypes.data, cnt.ctypes.data, 16, buf.ctypes.data, 16, buf2.ctypes.data) == -3
    cnt[1] = 4
    assert lib.spd_ngram_build(2, 3, keys.ctypes.data, cnt.ctypes.data, 8, buf.ctypes.data, 16, buf2.ctypes.data) == -4
    assert lib.spd_ngram_build(2, 3, keys.ctypes.data, cnt.ctypes.data, 16, buf.ctypes.data, 16, buf2.ctypes.data) == 0
    assert sorted(buf2.view(np.uint32).reshape(-1, 4)[:, 3].tolist())[-2:] == [1, 7]


def test_no_cpu_path():
    import torch
    import paper_2405_18400_b200 as P
    wl = si.get_workload("tiny")
    fake = {"tok_emb": torch.zeros(2, 2)}
    with pytest.raises(RuntimeError):
        P.SpdContext(wl.shape, fake, [], 3, wl.orders, wl.lambdas(), 0.5, 0.1, 0.01, 64)


def test_ring_plan(lib):
    """The decode kernel's default ring: two of the longest rows per stage when four such stages fit, else one row;
    the fragments of x (192 bytes per 32 columns of d_model) come out of the ring's room when there are images."""
    def plan(images, **kw):
        sb, ns = C.c_int32(), C.c_int32()
        assert lib.spd_ring_plan(C.byref(_cfg(**kw)), 1 if images else 0, C.byref(sb), C.byref(ns)) == 0
        return sb.value, ns.value
    big = dict(n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000, max_pos=4096)
    assert plan(True, **big) == (44032, 4) and plan(False, **big) == (44032, 4)           # 2 x 22016 bytes (a multiple of 1 KB)
    wide = dict(n_layers=40, d_model=5120, n_heads=40, d_ffn=13824, vocab=32000, max_pos=4096)
    assert plan(True, **wide) == (27648, 6) and plan(False, **wide) == (27648, 7)         # four two-row stages do not fit
    assert plan(True)[0] == 32768 and plan(False)[0] == 32768                             # short rows: 32 KB stages
    for images in (False, True):
        sb, ns = plan(images, **big)
        assert sb * ns + 20480 + (4096 // 32 * 192 if images else 0) + 4096 <= 232448     # within the 227 KB of a block
    assert lib.spd_ring_plan(C.byref(_cfg(k=0)), 0, C.byref(C.c_int32()), C.byref(C.c_int32())) == -1
