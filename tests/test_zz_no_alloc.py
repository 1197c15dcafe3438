"""spd_score_static: the scoring stage for callers that cannot allocate device memory (they hold device
pointers to the tables but have no allocator to obtain a workspace from, so spd_create is closed to
them).  Its scratch is a fixed array inside the library, shared by all calls, so the check runs it twice in
a row on different inputs and compares each result with the workspace-based entry point and with the CPU
oracle's scoring stage, and watches the device's free memory across the calls."""
import numpy as np
import pytest
import torch

import spd_inputs as si
from oracle import spd_oracle as so

pytestmark = pytest.mark.gpu


def _case(tables, rng, k, vocab, hist_len):
    keys = tables[-1]["keys"].numpy()
    n = keys.shape[1]
    rows = keys[rng.integers(0, keys.shape[0], size=k)]
    hist = np.concatenate([rng.integers(0, vocab, size=(k, 8 - (n - 1))), rows[:, : n - 1]], axis=1).astype(np.int32)
    cand = list(dict.fromkeys(int(rows[i, n - 1]) for i in range(max(1, k // 2))))
    while len(cand) < k:
        t = int(rng.integers(0, vocab))
        if t not in cand:
            cand.append(t)
    logp = (-rng.random(k) * 3).astype(np.float32)
    cand_lp = np.sort((-rng.random(k) * 4).astype(np.float32))[::-1].copy()
    return np.ascontiguousarray(hist[:, 8 - hist_len:]), logp, np.array(cand, np.int32), cand_lp


def test_static_scratch_entry_point_matches_workspace_entry_point(tiny_inputs):
    import paper_2405_18400_b200 as P
    from paper_2405_18400_b200.binding import spd_score_static

    wl, weights, tables, prefix = tiny_inputs
    dtabs = P.build_ngram_tables(tables, "cuda:0")
    packed = P.pack_weights(weights, "cuda:0")
    rng = np.random.default_rng(2024)
    ctxs = {}
    hits = 0
    otabs = so.NgramTables(sorted(tables, key=lambda t: int(t["n"])))
    # two calls in a row (then more): a larger k first, so that the second call would see leftovers if
    # the shared array were not rewritten
    for k, hist_len in [(5, 8), (3, 8), (16, 2), (2, 5)]:
        if k not in ctxs:
            ctxs[k] = P.SpdContext(wl.shape, packed, dtabs, k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64)
        hist, logp, cand, cand_lp = _case(tables, rng, k, wl.shape.vocab, hist_len)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        sel, out_lp, gamma, score = spd_score_static(k, wl.shape.vocab, wl.orders, wl.lambdas(), wl.alpha, wl.delta,
                                                     dtabs, hist, logp, cand, cand_lp)
        assert torch.cuda.mem_get_info()[0] == free_before            # the call took no device memory
        # against the CPU oracle's scoring stage on the same inputs (Eq. 5-7, Eq. 2, Eq. 4)
        cfg = so.make_config(wl.shape, k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, "bf16")
        want = so.score_stage(cfg, otabs, hist, logp, cand, cand_lp)
        fin = np.isfinite(want["score"])
        assert np.array_equal(np.isfinite(score), fin) and np.abs(score[fin] - want["score"][fin]).max() < 2e-5
        srt = np.sort(want["score"][fin])[::-1][: k + 1]
        if np.min(-np.diff(srt)) > 1e-4:
            assert sel.tolist() == want["sel"].tolist()
            assert np.abs(out_lp - want["logP"]).max() < 2e-5 and np.abs(gamma - want["gamma"]).max() < 1e-4
        ctx = ctxs[k]
        ctx.spd_debug_score(hist, logp, cand, cand_lp)
        want_score = ctx.spd_debug_read("SCORE")
        assert np.array_equal(score, want_score)                      # same kernel code, same inputs: bit-identical
        assert np.array_equal(sel, ctx.spd_debug_read("SEL"))
        assert np.array_equal(out_lp, ctx.spd_debug_read("LOGP"))
        assert abs(float(gamma.sum()) - 1.0) < 1e-5 and np.all(np.diff(gamma) <= 0)
        hits += int((ctx.spd_debug_read("CNT") > 0).sum())
    assert hits > 0
    for c in ctxs.values():
        c.close()


def test_static_scratch_entry_point_refuses_oversized_requests(tiny_inputs):
    import paper_2405_18400_b200 as P
    from paper_2405_18400_b200.binding import spd_score_static

    wl, weights, tables, prefix = tiny_inputs
    dtabs = P.build_ngram_tables(tables, "cuda:0")
    z = np.zeros(17, np.float32)
    with pytest.raises(P.SpdError) as e:
        spd_score_static(17, wl.shape.vocab, wl.orders, wl.lambdas(), wl.alpha, wl.delta, dtabs,
                         np.zeros((17, 8), np.int32), z, np.arange(17, dtype=np.int32), z)
    assert e.value.status == -3
    with pytest.raises(P.SpdError) as e:
        spd_score_static(3, wl.shape.vocab, wl.orders, wl.lambdas(), wl.alpha, wl.delta, dtabs,
                         np.zeros((3, 9), np.int32), z[:3], np.arange(3, dtype=np.int32), z[:3])
    assert e.value.status == -3
    with pytest.raises(P.SpdError) as e:      # more tables than the fixed scratch was laid out for
        spd_score_static(3, wl.shape.vocab, wl.orders, wl.lambdas(), wl.alpha, wl.delta, [dtabs[0]] * 9,
                         np.zeros((3, 8), np.int32), z[:3], np.arange(3, dtype=np.int32), z[:3])
    assert e.value.status == -3
