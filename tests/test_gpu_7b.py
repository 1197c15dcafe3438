"""Parity at the benchmark's full size: the 7B-shape decoder with 10 M-entry n-gram tables per order,
k = 3, 15-token prefix, in the launch configuration bench.py times (one launch of several steps)."""
import numpy as np
import pytest
import torch

import spd_inputs as si
from oracle import spd_oracle as so
from tests.gpu_common import compare_first_step, compare_step

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def big():
    import paper_2405_18400_b200 as P

    wl = si.get_workload("7b_k3")
    dev = torch.device("cuda:0")
    weights = si.make_weights(wl.shape, seed=0, device=dev)
    host = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in weights.items()}
    tables = si.make_ngram_tables(wl.shape.vocab, wl.zipf_s, wl.stream_len, wl.orders, wl.retain, seed=1, device=dev)
    prefix = si.make_prefix(wl.prefix_kind, wl.prefix_len, wl.shape.vocab, wl.zipf_s, seed=2)
    packed = P.pack_weights(weights, dev, consume=True)
    del weights
    dtabs = P.build_ngram_tables(tables, dev)
    torch.cuda.empty_cache()
    ctx = P.SpdContext(wl.shape, packed, dtabs, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, wl.kv_dtype)
    cfg = so.make_config(wl.shape, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, wl.kv_dtype)
    orc = so.Oracle(cfg, host, tables)
    yield wl, ctx, orc, tables, prefix
    ctx.close()
    orc.close()


def test_7b_steps_match_oracle(big):
    wl, ctx, orc, tables, prefix = big
    stats = []
    compare_first_step(ctx, orc, prefix, stats)
    for _ in range(3):
        compare_step(ctx, orc, stats)
    assert max(s["eps_z"] for s in stats) < 1e-3
    # the remaining steps of a 10-token draft in ONE launch, as the benchmark runs them
    margins_ok = True
    toks, lp, g = ctx.spd_generate(wl.gen_tokens - 4, wl.gen_tokens)
    for _ in range(wl.gen_tokens - 4):
        orc.step_forward()
        sel, nl, ng = orc.step_score()
        z = np.sort(orc.logits().astype(np.float32))[::-1][: wl.k + 1].astype(np.float64)
        sc = np.sort(orc.scores()[np.isfinite(orc.scores())])[::-1][: wl.k + 1]
        margins_ok &= bool(np.min(-np.diff(z)) > 1e-3 and np.min(-np.diff(sc)) > 2e-2)
        orc.step_commit(sel, nl)
    if margins_ok:
        assert np.array_equal(toks, orc.drafts()[:, len(prefix):])
        assert np.abs(g - orc.gamma()).max() < 2e-3
    z, z_o = ctx.spd_debug_read("LOGITS").astype(np.float64), orc.logits()
    assert np.abs(z - z_o).max() < 2e-2


def test_7b_tables_scoring_stage_with_hits(big):
    """Histories that end in stored 6-gram contexts of the 10 M-entry tables: counts, totals, choice."""
    wl, ctx, orc, tables, prefix = big
    rng = np.random.default_rng(5)
    keys = tables[-1]["keys"].numpy()
    k = wl.k
    hits = 0
    for trial in range(8):
        rows = keys[rng.integers(0, keys.shape[0], size=k)]
        hist = np.concatenate([rng.integers(0, wl.shape.vocab, size=(k, 3)), rows[:, :5]], axis=1).astype(np.int32)
        cand = list(dict.fromkeys([int(rows[0, 5]), int(rows[1, 5])]))
        while len(cand) < k:
            t = int(rng.integers(0, wl.shape.vocab))
            if t not in cand:
                cand.append(t)
        cand = np.array(cand, np.int32)
        logP = (-rng.random(k) * 3).astype(np.float32)
        cand_lp = np.sort((-rng.random(k) * 4).astype(np.float32))[::-1].copy()
        ctx.spd_debug_score(hist, logP, cand, cand_lp)
        want = so.score_stage(orc.cfg, orc.tables, hist, logP, cand, cand_lp)
        assert np.array_equal(ctx.spd_debug_read("CNT")[:, :5], want["cnt"])
        assert np.array_equal(ctx.spd_debug_read("TOT")[:, :5], want["tot"])
        hits += int((want["cnt"] > 0).sum())
        sc = ctx.spd_debug_read("SCORE").astype(np.float64)
        fin = np.isfinite(want["score"])
        assert np.array_equal(np.isfinite(sc), fin) and np.abs(sc[fin] - want["score"][fin]).max() < 5e-5
        srt = np.sort(want["score"][fin])[::-1][: k + 1]
        if np.min(-np.diff(srt)) > 1e-3:
            assert ctx.spd_debug_read("SEL").tolist() == want["sel"].tolist()
    assert hits >= 8
