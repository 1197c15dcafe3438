"""Pins for the seeded input generators (no method arithmetic lives there)."""
import collections

import numpy as np
import torch

import spd_inputs as si
from spd_inputs.rng import hash_u64, stream_base, splitmix64_scalar, uniform01


def test_splitmix64_known_answers():
    # First outputs of the published SplitMix64 generator started from state 0.
    g = 0x9E3779B97F4A7C15
    assert splitmix64_scalar(0) == 0xE220A8397B1DCDAF
    assert splitmix64_scalar(g) == 0x6E789E6AA1B965F4
    assert splitmix64_scalar((2 * g) & ((1 << 64) - 1)) == 0x06C45D188009454F


def test_tensor_hash_matches_scalar():
    idx = torch.tensor([0, 1, 2, 12345, 2**40 + 7], dtype=torch.int64)
    got = hash_u64(3, 9, idx)
    base = stream_base(3, 9)
    for i, v in zip(idx.tolist(), got.tolist()):
        want = splitmix64_scalar((i * 0x9E3779B97F4A7C15 + base) & ((1 << 64) - 1))
        assert (v & ((1 << 64) - 1)) == want
    u = uniform01(got)
    assert ((u > 0) & (u < 1)).all()


def test_weights_are_deterministic_and_shaped():
    sh = si.SHAPES["tiny"]
    a = si.make_weights(sh, seed=0)
    b = si.make_weights(sh, seed=0)
    c = si.make_weights(sh, seed=1)
    assert a["wq"][1].dtype == torch.bfloat16 and a["wdown"][0].shape == (sh.d_model, sh.d_ffn)
    assert torch.equal(a["wgate"][1], b["wgate"][1]) and not torch.equal(a["wgate"][1], c["wgate"][1])
    assert not torch.equal(a["wq"][0], a["wk"][0])
    assert abs(a["lm_head"].float().std().item() - 0.02) < 5e-4
    assert abs(a["lm_head"].float().mean().item()) < 2e-4
    assert abs(a["final_norm"].float().mean().item() - 1.0) < 0.03
    assert sh.n_params == 2 * (4 * 256 * 256 + 3 * 256 * 688) + 4096 * 256
    assert si.SHAPES["7b"].step_weight_bytes == 13_214_154_752
    assert si.SHAPES["13b"].step_weight_bytes == 25_703_219_200


def test_zipf_stream_follows_power_law():
    toks = si.zipf_tokens(1, 0, 400_000, 1000, 1.1)
    assert toks.min() >= 0 and toks.max() < 1000
    cnt = torch.bincount(toks, minlength=1000).double()
    want = np.arange(1, 1001, dtype=np.float64) ** -1.1
    want = want / want.sum() * 400_000
    for r in (0, 1, 4, 19):
        assert abs(cnt[r].item() - want[r]) < 5 * np.sqrt(want[r])


def test_ngram_counts_match_naive_scan():
    toks = si.zipf_tokens(5, 0, 3000, 50, 1.1)
    lst = toks.tolist()
    for n in (1, 2, 3, 4, 5, 6):
        naive = collections.Counter(tuple(lst[i:i + n]) for i in range(len(lst) - n + 1))
        t = si.count_ngrams(toks, n)
        keys = [tuple(r) for r in t["keys"].tolist()]
        assert keys == sorted(naive.keys())
        assert t["counts"].tolist() == [naive[k] for k in keys]


def test_ngram_retention_keeps_most_frequent_then_smallest_key():
    toks = si.zipf_tokens(6, 0, 5000, 40, 1.1)
    lst = toks.tolist()
    for n in (2, 4, 6):
        naive = collections.Counter(tuple(lst[i:i + n]) for i in range(len(lst) - n + 1))
        ranked = sorted(naive.items(), key=lambda kv: (-kv[1], kv[0]))[:100]
        t = si.count_ngrams(toks, n, retain=100)
        keys = [tuple(r) for r in t["keys"].tolist()]
        assert keys == sorted(k for k, _ in ranked)
        assert t["counts"].tolist() == [naive[k] for k in keys]


def test_workload_constants_are_the_papers():
    gold = {}
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "hyperparams.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                p = line.split()
                gold[p[0]] = [float(x) for x in p[1:]]
    w = si.get_workload("7b_k3")
    assert [w.alpha] == gold["alpha_n2_6"] and [w.tau] == gold["tau_n2_6"]
    assert list(w.lam) == gold["lambda_n2_6"]
    assert w.lambdas()[:5] == gold["lambda_n2_6"] and w.lambdas()[5:] == [0.0] * 3
    assert [w.prefix_len] == gold["prefix_len"] and [w.k] == gold["k"] and [w.gen_tokens] == gold["draft_tokens"]
    assert [min(w.orders)] == gold["n_min"] and [max(w.orders)] == gold["n_max"]
    t = si.get_workload("tiny")
    assert [t.alpha] == gold["alpha_n2_4"] and [t.tau] == gold["tau_n2_4"]
    assert t.lambdas()[:3] == gold["lambda_n2_6"][:3] and t.lambdas()[3:] == [0.0] * 5
