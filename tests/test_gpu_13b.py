"""Parity at 13B-shape (40 layers, d_model 5120, d_ffn 13824, k = 5): rows of 10 KB (three per ring chunk)
and 27 KB, five drafts, bf16 cache; a short prefix keeps the CPU oracle's dense pass to a few seconds."""
import numpy as np
import pytest
import torch

import spd_inputs as si
from oracle import spd_oracle as so
from tests.gpu_common import compare_first_step, compare_step

pytestmark = pytest.mark.gpu


def test_13b_steps_match_oracle():
    import paper_2405_18400_b200 as P

    wl = si.get_workload("13b_k5")
    dev = torch.device("cuda:0")
    weights = si.make_weights(wl.shape, seed=0, device=dev)
    host = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in weights.items()}
    tables = si.make_ngram_tables(wl.shape.vocab, wl.zipf_s, 2_000_000, wl.orders, 200_000, seed=1, device=dev)
    prefix = si.make_prefix(wl.prefix_kind, 8, wl.shape.vocab, wl.zipf_s, seed=2)
    packed = P.pack_weights(weights, dev, consume=True)
    del weights
    dtabs = P.build_ngram_tables(tables, dev)
    torch.cuda.empty_cache()
    ctx = P.SpdContext(wl.shape, packed, dtabs, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 32, wl.kv_dtype)
    cfg = so.make_config(wl.shape, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 32, wl.kv_dtype)
    orc = so.Oracle(cfg, host, tables)
    stats = []
    compare_first_step(ctx, orc, prefix, stats)
    for _ in range(3):
        ids, par, g = compare_step(ctx, orc, stats)
        assert abs(float(g.sum()) - 1.0) < 1e-5
    errs = [s for s in stats if "eps_z" in s]
    assert max(s["eps_z"] for s in errs) < 2e-3
    print("13B parity: max logit error %.3g" % max(s["eps_z"] for s in errs))
    ctx.close()
    orc.close()
