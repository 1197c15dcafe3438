"""Batched timesteps: B requests, each a context of its own over shared weights, stepped together with one pass over
the weights per timestep, every request compared element by element with its own CPU oracle (B independent
oracles: a request's step does not depend on the batch it runs in)."""
import numpy as np
import pytest
import torch

import spd_inputs as si
from oracle import spd_oracle as so
from tests.gpu_common import compare_first_step, compare_step

pytestmark = pytest.mark.gpu


def _requests(P, shape, packed, dtabs, host, tables, n, k, orders, lam, alpha, tau, delta, max_pos, kv_dtype, prefix_len, zipf_s):
    out = []
    otabs = sorted(tables, key=lambda t: int(t["n"]))
    for r in range(n):
        ctx = P.SpdContext(shape, packed, dtabs, k, orders, lam, alpha, tau, delta, max_pos, kv_dtype)
        cfg = so.make_config(shape, k, orders, lam, alpha, tau, delta, max_pos, kv_dtype)
        orc = so.Oracle(cfg, host, otabs)
        prefix = si.make_prefix("zipf", prefix_len + (r % 5), shape.vocab, zipf_s, seed=700 + r)   # own prefix, own length
        out.append((ctx, orc, prefix))
    return out


# up to 16, 32 and 64 requests take the small-batch product with token boxes of that many rows; more take the
# long-prefix path's 128-token tiles
@pytest.mark.parametrize("n,kv_dtype", [(2, "bf16"), (8, "f32"), (32, "bf16"), (48, "bf16"), (70, "f32")])
def test_batched_steps_tiny(tiny_inputs, n, kv_dtype):
    import paper_2405_18400_b200 as P

    wl, weights, tables, _ = tiny_inputs
    packed = P.pack_weights(weights, "cuda:0")
    dtabs = P.build_ngram_tables(tables, "cuda:0")
    reqs = _requests(P, wl.shape, packed, dtabs, weights, tables, n, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta,
                     256, kv_dtype, 12, wl.zipf_s)
    for ctx, orc, prefix in reqs:
        compare_first_step(ctx, orc, prefix)
    ctxs = [r[0] for r in reqs]
    before = ctxs[0].spd_launch_count()
    for step in range(3):
        res = P.spd_batch_step(ctxs)
        for (ctx, orc, _), got in zip(reqs, res):
            ids, par, g = compare_step(ctx, orc, None, stepped=got, path="prefill")
            assert abs(float(g.sum()) - 1.0) < 1e-5 and np.all(np.diff(g) <= 0)
    # a timestep of the batch is 9 launches per layer and three around them, whatever the number of requests
    assert ctxs[0].spd_launch_count() - before == 3 * (9 * wl.shape.n_layers + 3)
    # requests leave the batch and carry on alone, or in another batch, from where they are
    compare_step(reqs[0][0], reqs[0][1])
    if n > 2:
        sub = reqs[1: n // 2 + 1]
        res = P.spd_batch_step([r[0] for r in sub])
        for (ctx, orc, _), got in zip(sub, res):
            compare_step(ctx, orc, None, stepped=got, path="prefill")
    # several timesteps in one call equal the same number of single calls
    a = reqs[-1][0]
    b_ctx = P.SpdContext(wl.shape, packed, dtabs, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 256, kv_dtype)
    pf = reqs[-1][2]
    b_ctx.spd_prefill(pf)
    P.spd_batch_generate([b_ctx], 3)
    c_ctx = P.SpdContext(wl.shape, packed, dtabs, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 256, kv_dtype)
    c_ctx.spd_prefill(pf)
    for _ in range(3):
        P.spd_batch_step([c_ctx])
    assert np.array_equal(b_ctx.spd_debug_read("LOGITS"), c_ctx.spd_debug_read("LOGITS"))
    assert np.array_equal(b_ctx.spd_debug_read("LOGP"), c_ctx.spd_debug_read("LOGP"))
    for ctx, orc, _ in reqs:
        ctx.close(); orc.close()
    b_ctx.close(); c_ctx.close()


def test_batched_steps_7b_width():
    """Eight requests at the 7B shape's width (two layers): rows of 4096 and 11008 columns through the batched
    products, head size 128, five n-gram orders."""
    import paper_2405_18400_b200 as P

    shape = si.ModelShape("w7b", 2, 4096, 32, 11008, 2000)
    dev = torch.device("cuda:0")
    weights = si.make_weights(shape, seed=51, device=dev)
    host = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in weights.items()}
    tables = si.make_ngram_tables(shape.vocab, 1.1, 100_000, (2, 3, 4, 5, 6), 5000, seed=52)
    lam = [0.01, 0.04, 0.15, 0.18, 0.12, 0.0, 0.0, 0.0]
    packed = P.pack_weights(weights, dev, consume=True)
    del weights
    dtabs = P.build_ngram_tables(tables, dev)
    reqs = _requests(P, shape, packed, dtabs, host, tables, 8, 3, (2, 3, 4, 5, 6), lam, 0.54, 0.06, 0.01, 192, "bf16", 15, 1.1)
    stats = []
    for ctx, orc, prefix in reqs:
        compare_first_step(ctx, orc, prefix, stats)
    ctxs = [r[0] for r in reqs]
    for step in range(2):
        res = P.spd_batch_step(ctxs)
        for (ctx, orc, _), got in zip(reqs, res):
            compare_step(ctx, orc, stats, stepped=got, path="prefill")
    assert max(s["eps_z"] for s in stats if "eps_z" in s) < 2e-3
    for ctx, orc, _ in reqs:
        ctx.close(); orc.close()


def test_batch_argument_checks(tiny_inputs):
    import paper_2405_18400_b200 as P

    wl, weights, tables, prefix = tiny_inputs
    packed = P.pack_weights(weights, "cuda:0")
    dtabs = P.build_ngram_tables(tables, "cuda:0")
    mk = lambda max_pos=256, **kw: P.SpdContext(wl.shape, packed, dtabs, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta,
                                                max_pos, "bf16", **kw)
    a, b, small, stopper = mk(), mk(), mk(64), mk(eos_id=5)
    for c in (a, small, stopper):
        c.spd_prefill(prefix)

    def status(ctxs, steps=1):
        with pytest.raises(P.SpdError) as e:
            P.spd_batch_generate(ctxs, steps)
        return e.value.status

    assert status([a, b]) == -2                 # b was not prefilled
    b.spd_prefill(prefix)
    assert status([a, a]) == -1                 # a request twice
    assert status([small, a]) == -3             # the leading context has no long-prefix buffers to lend
    assert status([a, stopper]) == -1           # stop tokens are a single-request feature
    assert status([a, b], 0) == -3 and status([a, b], 1000) == -3
    P.spd_batch_generate([a, small], 2)         # only the leading context needs the buffers
    assert a.spd_debug_read("CAND_TOK").tolist() == small.spd_debug_read("CAND_TOK").tolist()
    for c in (a, b, small, stopper):
        c.close()
