"""Pins for the oracle's SPD procedure (Sections 3-3.2, Algorithm 1): special cases, invariants and a
brute-force enumeration of the k*k options in the linear domain."""
import itertools
import math

import numpy as np
import pytest
import torch

import spd_inputs as si
from oracle import spd_oracle as so
from tests.ref_decoder import dense_forward, f64


def _cfg(wl, k=3, kv="f32", alpha=None, delta=None, tau=None, max_pos=64, lam=None, orders=None):
    orders = wl.orders if orders is None else orders
    return so.make_config(wl.shape, k, orders, wl.lambdas() if lam is None else lam,
                          wl.alpha if alpha is None else alpha, wl.tau if tau is None else tau,
                          wl.delta if delta is None else delta, max_pos, kv)


def _dicts(tables):
    return {int(t["n"]): {tuple(r): int(c) for r, c in zip(t["keys"].tolist(), t["counts"].tolist())} for t in tables}


def _brute_png(dicts, lam, hist, tok):
    """Eq. 5 with dictionary counts: p_n = count(ctx + tok) / sum_x count(ctx + x)."""
    p = 0.0
    for n, d in dicts.items():
        if len(hist) < n - 1:
            continue
        ctx = tuple(hist[len(hist) - (n - 1):])
        tot = sum(c for key, c in d.items() if key[:-1] == ctx)
        if tot > 0:
            p += lam[n - 2] * d.get(ctx + (tok,), 0) / tot
    return p


def _hit_case(tables, rng, k, vocab):
    """Draft histories and kept tokens chosen so that n-gram lookups hit: histories end in stored
    contexts, kept tokens mix stored continuations with random tokens."""
    big = tables[-1]
    n = int(big["n"])
    keys = big["keys"].numpy()
    rows = keys[rng.integers(0, keys.shape[0], size=k)]
    hist = np.concatenate([rng.integers(0, vocab, size=(k, 3)), rows[:, : n - 1]], axis=1).astype(np.int32)
    cand = [int(rows[0, n - 1]), int(rows[1 % k, n - 1])]
    while len(cand) < k:
        t = int(rng.integers(0, vocab))
        if t not in cand:
            cand.append(t)
    cand = list(dict.fromkeys(cand))
    while len(cand) < k:
        cand.append(int(rng.integers(0, vocab)))
    return hist, np.array(cand[:k], np.int32)


def test_first_timestep_is_topk_of_the_prefix_distribution(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    o = so.Oracle(_cfg(wl, k=4), weights, tables)
    ids, g = o.prefill(prefix)
    z, _ = dense_forward(weights, wl.shape, f64(weights["tok_emb"])[torch.tensor(prefix)], "f32")
    lp = torch.log_softmax(z[-1] / wl.tau, dim=0)
    order = torch.argsort(z[-1].float(), descending=True, stable=True)[:4]
    assert ids.tolist() == order.tolist()                          # draft i gets the i-th most probable token
    assert np.allclose(o.logP(), lp[order].numpy(), atol=1e-9)     # p_i = p_theta(token | M): no n-gram term (Eq. 1)
    p = torch.exp(lp[order]).numpy()
    assert np.allclose(g, p / p.sum(), atol=1e-12)                 # Eq. 4
    d = o.drafts()
    assert d.shape == (4, len(prefix) + 1) and (d[:, :-1] == np.array(prefix)).all()


def test_topk_logprob_against_library_and_ties():
    rng = np.random.default_rng(3)
    z = rng.standard_normal(500) * 4
    z[[7, 300]] = z.max() + 1.0                                    # an exact tie for first place
    tok, lp = so.topk_logprob(z, 5, 0.06)
    assert tok[0] == 7 and tok[1] == 300                           # ties go to the lower id
    want = torch.log_softmax(torch.from_numpy(z) / 0.06, 0)
    assert np.allclose(lp, want[torch.from_numpy(tok.astype(np.int64))].numpy(), atol=1e-10)
    assert sorted(tok[2:].tolist()) == sorted(np.argsort(-z)[2:5].tolist())


@pytest.mark.parametrize("alpha,delta", [(0.54, 0.01), (0.0, 1.0), (0.9, 0.5)])
def test_k1_is_greedy_decoding(tiny_inputs, alpha, delta):
    """With one draft the procedure keeps the single most probable token each step, whatever the
    n-gram settings: the sequence must equal an argmax loop over a cache-free dense decoder."""
    wl, weights, tables, prefix = tiny_inputs
    o = so.Oracle(_cfg(wl, k=1, alpha=alpha, delta=delta), weights, tables)
    ids, g = o.prefill(prefix)
    got = [int(ids[0])]
    for _ in range(5):
        ids, par, g = o.step()
        assert g[0] == 1.0 and par[0] == 0
        got.append(int(ids[0]))
    seq = list(prefix)
    want = []
    E = f64(weights["tok_emb"])
    for _ in range(6):
        z, _ = dense_forward(weights, wl.shape, E[torch.tensor(seq)], "f32")
        t = int(torch.argmax(z[-1]))
        want.append(t)
        seq.append(t)
    assert got == want


def test_gamma_sums_to_one_sorted_and_drafts_unique(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    for k in (2, 3, 5):
        o = so.Oracle(_cfg(wl, k=k, kv="bf16"), weights, tables)
        ids, g = o.prefill(prefix)
        hist = [list(prefix) + [int(t)] for t in ids]
        for _ in range(6):
            ids, par, g = o.step()
            assert abs(g.sum() - 1.0) < 1e-12 and np.all(np.diff(g) <= 0)      # Eq. 3 constraint; ordered by probability
            assert np.all(np.diff(o.logP()) <= 0)
            hist = [hist[int(par[r])] + [int(ids[r])] for r in range(k)]
            assert o.drafts().tolist() == hist                                  # parent bookkeeping
            assert len({tuple(h) for h in hist}) == k                           # k unique drafts
            p = np.exp(o.logP() - o.logP().max())
            assert np.allclose(g, p / p.sum(), atol=1e-12)


def test_score_stage_equals_bruteforce_enumeration(tiny_inputs):
    """All k*k options evaluated in the linear domain (p_i * p_theta^(1-a) * p_ngram^a, or with delta when a
    draft's n-gram distribution misses every kept token), full sort, against the oracle's log-domain stage."""
    wl, weights, tables, prefix = tiny_inputs
    dicts = _dicts(tables)
    lam = wl.lambdas()
    rng = np.random.default_rng(11)
    ot = so.NgramTables(tables)
    seen_hit = seen_miss_draft = seen_dropped = 0
    for trial in range(30):
        k = int(rng.integers(2, 6))
        cfg = _cfg(wl, k=k)
        hist, cand = _hit_case(tables, rng, k, wl.shape.vocab)
        if trial % 3 == 0:
            hist[k - 1] = rng.integers(0, wl.shape.vocab, size=hist.shape[1])   # a draft with (almost surely) no overlap
        logP = -rng.random(k) * 3
        cand_lp = np.sort(-rng.random(k) * 4)[::-1].copy()
        out = so.score_stage(cfg, ot, hist, logP, cand, cand_lp)
        joint = {}
        for i in range(k):
            pn = [_brute_png(dicts, lam, hist[i].tolist(), int(c)) for c in cand]
            assert np.allclose(out["png"][i * k:(i + 1) * k], pn, atol=1e-15)
            assert all(p <= 0.5 + 1e-12 for p in pn)                            # printed lambdas sum to 0.20 (n<=4) / 0.50
            for j in range(k):
                pt = math.exp(cand_lp[j])
                if max(pn) == 0.0:
                    pf = wl.delta * pt ** (1 - wl.alpha)                        # Eq. 7
                    seen_miss_draft += 1
                elif pn[j] > 0:
                    pf = pt ** (1 - wl.alpha) * pn[j] ** wl.alpha               # Eq. 6
                    seen_hit += 1
                else:
                    pf = 0.0                                                    # token absent from the n-gram distribution
                    seen_dropped += 1
                joint[i * k + j] = math.exp(logP[i]) * pf
        ranked = sorted(joint, key=lambda q: (-joint[q], q))[:k]
        assert out["sel"].tolist() == ranked
        pj = np.array([joint[q] for q in ranked])
        assert np.all(pj > 0)
        assert np.allclose(np.exp(out["logP"]), pj, rtol=1e-12)
        assert np.allclose(out["gamma"], pj / pj.sum(), atol=1e-12)
    assert seen_hit > 20 and seen_miss_draft > 20 and seen_dropped > 20


def test_ngram_counts_and_totals(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    dicts = _dicts(tables)
    ot = so.NgramTables(tables)
    rng = np.random.default_rng(5)
    import ctypes as C
    for ti, t in enumerate(tables):
        n = int(t["n"])
        keys = t["keys"].numpy()
        for trial in range(40):
            row = keys[rng.integers(0, keys.shape[0])].copy()
            if trial % 2:
                row[-1] = rng.integers(0, wl.shape.vocab)
            if trial % 5 == 4:
                row[0] = rng.integers(0, wl.shape.vocab)
            cnt = np.zeros(1, np.int64)
            tot = np.zeros(1, np.int64)
            ctx = np.ascontiguousarray(row[:-1].astype(np.int32))
            so.lib().orc_ngram_counts(C.byref(ot.arr[ti]), ctx.ctypes.data, int(row[-1]), cnt.ctypes.data, tot.ctypes.data)
            d = dicts[n]
            assert cnt[0] == d.get(tuple(row.tolist()), 0)
            assert tot[0] == sum(c for key, c in d.items() if key[:-1] == tuple(row[:-1].tolist()))
        # each stored context's distribution sums to one over the stored continuations
        ctx = tuple(keys[123][:-1].tolist())
        tot = sum(c for key, c in dicts[n].items() if key[:-1] == ctx)
        assert abs(sum(c / tot for key, c in dicts[n].items() if key[:-1] == ctx) - 1.0) < 1e-12


def test_alpha_zero_delta_one_ignores_the_tables(tiny_inputs):
    """'n-gram smoothing disabled' (Appendix B): with alpha = 0 and delta = 1 every finite option scores
    logP_i + lp_j, so on all-miss tables the best option is always (draft 0, token 0)."""
    wl, weights, tables, prefix = tiny_inputs
    empty = [{"n": n, "keys": np.zeros((0, n), np.int32), "counts": np.zeros(0, np.int64)} for n in wl.orders]
    o = so.Oracle(_cfg(wl, alpha=0.0, delta=1.0), weights, empty)
    o.prefill(prefix)
    for _ in range(4):
        lp0 = o.logP().copy()
        o.step_forward()
        sel, nl, ng = o.step_score()
        sc = o.scores().reshape(3, 3)
        assert np.allclose(sc, lp0[:, None] + o.cand_lp()[None, :], atol=1e-12)
        assert sel[0] == 0
        o.step_commit(sel, nl)


def test_all_miss_tables_rank_like_scaled_beam_search(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    empty = [{"n": n, "keys": np.zeros((0, n), np.int32), "counts": np.zeros(0, np.int64)} for n in wl.orders]
    o = so.Oracle(_cfg(wl), weights, empty)
    o.prefill(prefix)
    for _ in range(3):
        lp0 = o.logP().copy()
        o.step_forward()
        sel, nl, ng = o.step_score()
        want = lp0[:, None] + (1 - wl.alpha) * o.cand_lp()[None, :] + math.log(wl.delta)   # Eq. 7 for every draft
        assert np.allclose(o.scores().reshape(3, 3), want, atol=1e-12)
        flat = want.reshape(-1)
        assert sel.tolist() == sorted(range(9), key=lambda q: (-np.float32(flat[q]), q))[:3]
        o.step_commit(sel, nl)


def test_score_stage_invariances(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    rng = np.random.default_rng(21)
    ot = so.NgramTables(tables)
    k = 4
    cfg = _cfg(wl, k=k)
    hist, cand = _hit_case(tables, rng, k, wl.shape.vocab)
    logP = -rng.random(k) * 3
    cand_lp = np.sort(-rng.random(k) * 4)[::-1].copy()
    a = so.score_stage(cfg, ot, hist, logP, cand, cand_lp)
    # a common factor on p_theta (e.g. renormalising over the kept tokens) changes neither choice nor gamma
    b = so.score_stage(cfg, ot, hist, logP, cand, cand_lp + 1.2345)
    assert a["sel"].tolist() == b["sel"].tolist() and np.allclose(a["gamma"], b["gamma"], atol=1e-12)
    # so does a common factor on all draft probabilities
    c = so.score_stage(cfg, ot, hist, logP - 7.0, cand, cand_lp)
    assert a["sel"].tolist() == c["sel"].tolist() and np.allclose(a["gamma"], c["gamma"], atol=1e-12)
    # permuting the draft slots selects the same (draft, token) options
    perm = np.array([2, 0, 3, 1])
    d = so.score_stage(cfg, ot, hist[perm], logP[perm], cand, cand_lp)
    opts_a = {(int(q) // k, int(q) % k) for q in a["sel"]}
    opts_d = {(int(perm[int(q) // k]), int(q) % k) for q in d["sel"]}
    assert opts_a == opts_d and np.allclose(np.sort(a["gamma"]), np.sort(d["gamma"]), atol=1e-12)


def test_short_history_skips_long_orders(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    dicts = _dicts(tables)
    ot = so.NgramTables(tables)
    cfg = _cfg(wl, k=2)
    key = tables[0]["keys"][50].tolist()                          # a stored bigram
    hist = np.array([[key[0]], [key[0]]], np.int32)               # one-token histories: only n = 2 applies
    out = so.score_stage(cfg, ot, hist, np.zeros(2), np.array([key[1], 4095], np.int32), np.array([-0.1, -0.2]))
    assert np.all(out["cnt"][:, 1:] == -1) and np.all(out["tot"][:, 1:] == -1)
    assert np.isclose(out["png"][0], wl.lambdas()[0] * _brute_png({2: dicts[2]}, [1.0], [key[0]], key[1]))


def test_equal_last_tokens_make_the_step_an_ordinary_decode_step(tiny_inputs):
    """If every draft ends in the same token, sum_i gamma_i E[token] = E[token] (Eq. 3 with sum gamma = 1), so the LM
    pass equals ordinary decoding of that token."""
    wl, weights, tables, prefix = tiny_inputs
    cfg = _cfg(wl)
    a = so.Oracle(cfg, weights, tables)
    a.prefill(prefix)
    for _ in range(8):
        ids, par, g = a.step()
        if len(set(ids.tolist())) == 1:
            break
    assert len(set(ids.tolist())) == 1, "fixture no longer reaches a step with equal last tokens"
    n_sup = a.T() - len(prefix)
    a.step_forward()
    E = f64(weights["tok_emb"])
    b = so.Oracle(cfg, weights, tables)
    b.prefill(prefix)
    for _ in range(n_sup):
        b.step()
    b.feed_token(int(ids[0]))
    assert np.abs(a.logits() - b.logits()).max() < 1e-9


def test_generation_stops_after_the_stop_token(tiny_inputs):
    """Algorithm 1's loop condition: with a stop token the run ends with the step in which the most probable draft
    emits it and is otherwise unchanged; without one, or with one that never comes, all steps are taken."""
    wl, weights, tables, prefix = tiny_inputs
    cfg = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, "f32")
    a = so.Oracle(cfg, weights, tables)
    a.prefill(prefix)
    assert a.generate(6) == 6
    full = a.drafts()[:, len(prefix):].copy()
    tops = []                       # the most probable draft's newest token after each step
    b = so.Oracle(cfg, weights, tables)
    b.prefill(prefix)
    for _ in range(6):
        ids, _, _ = b.step()
        tops.append(int(ids[0]))
    eos = tops[3]
    first = tops.index(eos)         # it may also have come earlier
    c = so.Oracle(cfg, weights, tables)
    c.prefill(prefix)
    assert c.generate(6, eos) == first + 1
    assert c.drafts().shape[1] == len(prefix) + 1 + first + 1
    never = next(t for t in range(wl.shape.vocab) if t not in full)
    d = so.Oracle(cfg, weights, tables)
    d.prefill(prefix)
    assert d.generate(6, never) == 6 and np.array_equal(d.drafts()[:, len(prefix):], full)
