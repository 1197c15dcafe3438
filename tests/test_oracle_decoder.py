"""Pins for the oracle's decoder: closed forms, and an independent dense float64 decoder."""
import ctypes as C
import math

import numpy as np
import pytest
import torch

import spd_inputs as si
from oracle import spd_oracle as so
from tests.ref_decoder import dense_forward, f64


def _bits(vals):
    return so.bf16_bits(torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16))


def test_round_bf16_matches_library_rounding():
    rng = np.random.default_rng(0)
    xs = np.concatenate([rng.standard_normal(2000).astype(np.float32) * 3,
                         np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38, 1e-40], np.float32)])
    want = torch.from_numpy(xs).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([so.lib().orc_round_bf16(float(x)) for x in xs], np.float32)
    assert np.array_equal(got, want)
    # exact ties go to the even mantissa: 1 + 2^-8 -> 1, 1 + 3*2^-8 -> 1 + 2^-6
    assert got[2000] == 1.0 and got[2001] == 1.015625


def test_rmsnorm_closed_forms():
    d = 8
    y = np.zeros(d)
    g = _bits([0.5, 1, 2, 1, 1, 1, 1, 1])
    x = np.full(d, -3.0)
    so.lib().orc_rmsnorm(x.ctypes.data, g.ctypes.data, d, 0.0, y.ctypes.data)
    assert np.allclose(y, -np.array([0.5, 1, 2, 1, 1, 1, 1, 1]), atol=1e-15)      # constant vector -> sign * gain
    x = np.array([3.0, 4.0, 0, 0, 0, 0, 0, 0])
    so.lib().orc_rmsnorm(x.ctypes.data, g.ctypes.data, d, 0.0, y.ctypes.data)
    assert np.allclose(y[:2], [0.5 * 3 / math.sqrt(25 / 8), 4 / math.sqrt(25 / 8)], atol=1e-15)
    so.lib().orc_rmsnorm(x.ctypes.data, g.ctypes.data, d, 1.0, y.ctypes.data)
    assert np.allclose(y[1], 4 / math.sqrt(25 / 8 + 1.0), atol=1e-15)               # eps sits inside the root


def test_rope_closed_forms():
    hd = 8
    x0 = np.arange(1.0, hd + 1)
    x = x0.copy()
    so.lib().orc_rope(x.ctypes.data, hd, 0, 10000.0)
    assert np.array_equal(x, x0)                                                    # position 0 is the identity
    x = x0.copy()
    so.lib().orc_rope(x.ctypes.data, hd, 3, 10000.0)
    assert np.allclose(x[0::2] ** 2 + x[1::2] ** 2, x0[0::2] ** 2 + x0[1::2] ** 2)  # a rotation per pair
    # pair 0 turns by pos radians, pair i by pos * theta^(-2i/hd); counter-clockwise
    assert np.allclose(x[:2], [1 * math.cos(3) - 2 * math.sin(3), 1 * math.sin(3) + 2 * math.cos(3)])
    a = 3 * 10000.0 ** (-2 * 2 / 8)
    assert np.allclose(x[4:6], [5 * math.cos(a) - 6 * math.sin(a), 5 * math.sin(a) + 6 * math.cos(a)])
    # relative property: <rope(q,p), rope(k,s)> depends on p - s only
    q, k = np.random.default_rng(1).standard_normal((2, hd))
    def dot(p, s):
        a_, b_ = q.copy(), k.copy()
        so.lib().orc_rope(a_.ctypes.data, hd, p, 10000.0)
        so.lib().orc_rope(b_.ctypes.data, hd, s, 10000.0)
        return float(a_ @ b_)
    assert abs(dot(7, 4) - dot(13, 10)) < 1e-12 and abs(dot(7, 4) - dot(8, 4)) > 1e-6


def test_attention_closed_forms():
    hd, T, stride = 4, 3, 8
    K = np.zeros((T, stride), np.float32)
    V = np.zeros((T, stride), np.float32)
    V[:, :hd] = [[1, 2, 3, 4], [5, 6, 7, 8], [-1, 0, 1, 2]]
    q = np.array([0.3, -0.2, 0.1, 0.9])
    o = np.zeros(hd)
    so.lib().orc_attention_head(q.ctypes.data, K.ctypes.data, V.ctypes.data, 1, hd, stride, o.ctypes.data)
    assert np.array_equal(o, V[0, :hd])                                             # one position: output = v
    so.lib().orc_attention_head(q.ctypes.data, K.ctypes.data, V.ctypes.data, 3, hd, stride, o.ctypes.data)
    assert np.allclose(o, V[:, :hd].mean(0))                                        # equal scores: plain mean
    K[1, :hd] = q * 2
    so.lib().orc_attention_head(q.ctypes.data, K.ctypes.data, V.ctypes.data, 3, hd, stride, o.ctypes.data)
    s = float(q @ (q * 2)) / math.sqrt(hd)                                          # scale is 1/sqrt(hd)
    w = np.array([1.0, math.exp(s), 1.0])
    assert np.allclose(o, (w[:, None] * V[:, :hd]).sum(0) / w.sum())


@pytest.mark.parametrize("kv_dtype,tol", [("f32", 2e-6), ("bf16", 2e-3)])
def test_prefill_logits_match_independent_dense_decoder(tiny_inputs, kv_dtype, tol):
    wl, weights, tables, prefix = tiny_inputs
    cfg = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, kv_dtype)
    o = so.Oracle(cfg, weights, tables)
    o.prefill(prefix)
    X = f64(weights["tok_emb"])[torch.tensor(prefix)]
    logits, trace = dense_forward(weights, wl.shape, X, kv_dtype)
    assert np.abs(o.logits() - logits[-1].numpy()).max() < tol
    tr = o.trace()
    for l in range(wl.shape.n_layers):
        assert np.abs(tr[l, 0] - trace[2 * l][-1].numpy()).max() < tol
        assert np.abs(tr[l, 1] - trace[2 * l + 1][-1].numpy()).max() < tol


def test_cached_superposed_steps_match_dense_pass_over_all_input_rows(tiny_inputs):
    """Eq. 3 + the shared cache: step logits equal a cache-free dense pass whose input rows are the
    prefix embeddings followed by the superposed embeddings sum_i gamma_i E[token_i]."""
    wl, weights, tables, prefix = tiny_inputs
    cfg = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, "f32")
    o = so.Oracle(cfg, weights, tables)
    E = f64(weights["tok_emb"])
    rows = [E[t] for t in prefix]
    ids, g = o.prefill(prefix)
    for _ in range(4):
        assert abs(g.sum() - 1) < 1e-12
        rows.append(sum(float(g[i]) * E[int(ids[i])] for i in range(3)))
        ids, par, g = o.step()
        logits, _ = dense_forward(weights, wl.shape, torch.stack(rows), "f32")
        assert np.abs(o.logits() - logits[-1].numpy()).max() < 2e-6


def test_dense_prefill_equals_token_by_token_decoding(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    for kv in ("f32", "bf16"):
        cfg = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, kv)
        a = so.Oracle(cfg, weights, tables)
        b = so.Oracle(cfg, weights, tables)
        a.prefill(prefix)
        for t in prefix:
            b.feed_token(t)
        assert a.T() == b.T() == len(prefix)
        assert np.abs(a.logits() - b.logits()).max() < 1e-12
        ka, va = a.kv_cache()
        kb, vb = b.kv_cache()
        assert np.array_equal(ka, kb) and np.array_equal(va, vb)


def test_bf16_cache_holds_bf16_values(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    cfg = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, "bf16")
    o = so.Oracle(cfg, weights, tables)
    o.prefill(prefix)
    k, v = o.kv_cache()
    for a in (k[:, :16], v[:, :16]):
        t = torch.from_numpy(np.ascontiguousarray(a))
        assert torch.equal(t.to(torch.bfloat16).to(torch.float32), t) and t.abs().max() > 0
    assert np.all(k[:, 16:] == 0)


def _bf16_step(a, up):
    """The bf16 value next to each (bf16-representable, non-zero) float32 value, upwards or downwards."""
    bits = a.astype(np.float32).view(np.uint32).astype(np.int64)
    away = (a > 0) == up
    return (bits + np.where(away, 1 << 16, -(1 << 16))).astype(np.uint32).view(np.float32)


def test_cache_following_adopts_only_valid_roundings(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    cfg = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, "bf16")
    a = so.Oracle(cfg, weights, tables)
    a.prefill(prefix)
    k, v = (x[:, :16].copy() for x in a.kv_cache())
    z0 = a.logits()
    b = so.Oracle(cfg, weights, tables)
    b.follow_cache(k, v)
    b.prefill(prefix)
    assert b.follow_cache(None) == (0, 0) and np.array_equal(b.logits(), z0)      # its own values: nothing to adopt
    # the exact layer-0 keys (layer 0 does not depend on the cache type): a float32 cache keeps them to 2^-24
    cfg32 = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, "f32")
    e = so.Oracle(cfg32, weights, tables)
    e.prefill(prefix)
    x = e.kv_cache()[0][0, :16].astype(np.float64)
    own = k[0].astype(np.float64)
    assert np.all(own != 0)
    toward = _bf16_step(k[0], x > own)        # the exact value's other neighbour
    beyond = _bf16_step(k[0], x <= own)       # the neighbour on the far side of the cache value
    mid_dist = np.abs(0.5 * (own + toward.astype(np.float64)) - x)   # distance of x from the rounding boundary
    # (1) without slack no neighbour is a rounding of x (exact midpoints aside: none here)
    k2 = k.copy()
    k2[0] = toward
    c = so.Oracle(cfg, weights, tables)
    c.follow_cache(k2, v, slack=0.0)
    c.prefill(prefix)
    assert np.array_equal(c.kv_cache()[0][0, :16], k[0])
    assert c.follow_cache(None)[1] >= k[0].size
    # (2) with slack s exactly the values within s of the boundary flip: half a spacing plus s, not a whole spacing
    s_ = float(np.median(mid_dist))
    clear = np.abs(mid_dist - s_) > 1e-6 * np.abs(x)
    c = so.Oracle(cfg, weights, tables)
    c.follow_cache(k2, v, slack=s_)
    c.prefill(prefix)
    got = c.kv_cache()[0][0, :16]
    assert np.array_equal((got == toward)[clear], (mid_dist <= s_)[clear])
    assert np.array_equal(got[mid_dist > s_ + 1e-6 * np.abs(x)], k[0][mid_dist > s_ + 1e-6 * np.abs(x)])
    flips, bad = c.follow_cache(None)
    assert flips > 0.3 * k[0].size and bad > 0.3 * k[0].size and 0 < c.follow_need <= s_
    # (3) the far-side neighbour is never a rounding of x, even with a slack of half a spacing
    k3 = k.copy()
    k3[0] = beyond
    c = so.Oracle(cfg, weights, tables)
    c.follow_cache(k3, v, slack=float(np.min(np.abs(toward.astype(np.float64) - own))) * 0.49)
    c.prefill(prefix)
    assert np.array_equal(c.kv_cache()[0][0, :16], k[0]) and c.follow_cache(None)[0] == 0
    # (4) values that are no rounding of the exact ones are refused and counted
    k4 = k.copy()
    k4[1, 3, :7] += 1.0
    d = so.Oracle(cfg, weights, tables)
    d.follow_cache(k4, v, slack=1e-6)
    d.prefill(prefix)
    assert d.follow_cache(None) == (0, 7) and np.array_equal(d.logits(), z0)


def test_cache_following_slack_covers_values_near_zero(tiny_inputs):
    """Near zero the spacing of bf16 is far below any float error: there the slack, not the spacing, decides.  A value
    moved by less than the slack (many bf16 steps near zero) is adopted with the slack and refused without it."""
    wl, weights, tables, prefix = tiny_inputs
    cfg = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, "bf16")
    a = so.Oracle(cfg, weights, tables)
    a.prefill(prefix)
    k, v = (x[:, :16].copy() for x in a.kv_cache())
    small = np.argsort(np.abs(k[0]).ravel())[:8]           # the layer-0 keys closest to zero: |value| < 2e-3,
    slack = 2e-4                                           # bf16 spacing there <= 8e-6, far below this slack
    assert np.abs(k[0].ravel()[small]).max() < 2e-3
    moved = k.copy()
    flat = moved[0].reshape(-1)
    t = torch.from_numpy(flat[small] + np.float32(0.5 * slack)).to(torch.bfloat16).to(torch.float32).numpy()
    changed = t != flat[small]
    assert changed.all()                                   # half a slack crosses many bf16 steps for these
    flat[small] = t
    for s_, adopted in ((slack, True), (0.0, False)):
        c = so.Oracle(cfg, weights, tables)
        c.follow_cache(moved, v, slack=s_)
        c.prefill(prefix)
        got = c.kv_cache()[0][0, :16].reshape(-1)[small]
        flips, bad = c.follow_cache(None)
        if adopted:
            assert np.array_equal(got, t) and bad == 0 and flips >= changed.sum()
        else:
            assert np.array_equal(got[changed], k[0].reshape(-1)[small][changed]) and bad >= changed.sum()
