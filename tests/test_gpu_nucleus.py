"""GPU parity of nucleus sampling and of the splice of Superposed Decoding onto a sampled prefix (Section 4.5).

The draw is an integer decided by floating point, so both sides decide from the same numbers: the oracle's
sampler gets the device's float32 logits (the logits themselves are compared with the usual tolerance).  The
device sums exp() values in fixed point with float32 exp arguments, the oracle in float64: a draw closer than
`EPS` (relative) to a boundary of the cumulative distribution may legitimately fall on either side, so the
device's token must be among the oracle's tokens for p and u moved by +-EPS; away from boundaries that set has
one element."""
import numpy as np
import pytest
import torch

import spd_inputs as si
from oracle import spd_oracle as so
from tests.gpu_common import LOGIT_TOL, compare_first_step, compare_step, make_tiny_pair

pytestmark = pytest.mark.gpu

EPS = 1e-5


def accepted(z, temperature, p, u):
    """(token of the unperturbed decision, set of tokens within EPS of it).  p and the temperature reach the
    device as float32."""
    z = np.asarray(z, dtype=np.float64)
    p, temperature = float(np.float32(p)), float(np.float32(temperature))
    tok, info = so.nucleus(z, temperature, p, u)
    ok = {tok}
    if info["gap_cut"] < EPS or info["gap_draw"] < EPS * 2:
        for dp in (-EPS, 0.0, EPS):
            for du in (-2 * EPS, 0.0, 2 * EPS):
                ok.add(so.nucleus(z, temperature, min(1.0, max(1e-9, p + dp)), min(max(u + du, 0.0), 1 - 1e-9))[0])
    return tok, ok


def uniforms(n, seed):
    u = si.uniform01(si.hash_u64(seed, 77, torch.arange(n))).numpy().astype(np.float32)
    return np.minimum(u, np.float32(1.0 - 2.0 ** -24))


@pytest.mark.parametrize("top_p,temperature", [(0.9, 1.0), (0.95, 0.05), (1.0, 0.7), (0.3, 0.02)])
def test_sampler_alone_matches_the_oracle(tiny_inputs, top_p, temperature):
    ctx, _ = make_tiny_pair(tiny_inputs)
    rng = np.random.default_rng(5)
    v = ctx.shape.vocab
    exact = 0
    us = uniforms(40, 3)
    for i, u in enumerate(us):
        z = (rng.normal(0, 0.3, v) + (rng.random(v) < 0.01) * rng.normal(2, 1, v)).astype(np.float32)
        tok = ctx.spd_debug_nucleus(z, top_p, temperature, float(u))
        want, ok = accepted(z, temperature, top_p, float(u))
        assert tok in ok, (i, tok, want)
        exact += tok == want
    assert exact >= 30


def test_sampler_edge_cases(tiny_inputs):
    ctx, _ = make_tiny_pair(tiny_inputs)
    v = ctx.shape.vocab
    rng = np.random.default_rng(9)
    z = rng.normal(0, 1, v).astype(np.float32)
    # a vanishing p keeps the most probable token only: greedy
    assert ctx.spd_debug_nucleus(z, 1e-7, 1.0, 0.999) == int(np.argmax(z))
    # all logits equal: the nucleus is the first ceil(p V) ids and draw u takes id floor(u size); ties by id
    flat = np.full(v, -1.25, np.float32)
    for p, u in ((1.0, 0.0), (1.0, 0.5003), (1.0, 0.99999), (0.2503, 0.7001), (1e-7, 0.9)):
        size = int(np.ceil(p * v - 1e-9)) if p < 1 else v
        assert ctx.spd_debug_nucleus(flat, p, 1.0, u) == so.nucleus(flat, 1.0, p, u)[0] == int(u * max(size, 1))
    # two equal maxima far above the rest: ties go to the lower id first
    z2 = z.copy()
    z2[[123, 3001]] = 30.0
    assert ctx.spd_debug_nucleus(z2, 0.4, 1.0, 0.99) == 123
    assert ctx.spd_debug_nucleus(z2, 0.9, 1.0, 0.2) == 123
    assert ctx.spd_debug_nucleus(z2, 0.9, 1.0, 0.8) == 3001
    # negative zero and positive zero are one value; huge negative logits carry no mass
    z3 = np.full(v, -1e30, np.float32)
    z3[[7, 9]] = [-0.0, 0.0]
    assert ctx.spd_debug_nucleus(z3, 1.0, 1.0, 0.1) == 7 and ctx.spd_debug_nucleus(z3, 1.0, 1.0, 0.6) == 9
    # a cold temperature concentrates the mass on the maximum
    assert ctx.spd_debug_nucleus(z, 0.99, 1e-3, 0.7) == int(np.argmax(z))


def test_arguments_are_checked(tiny_inputs):
    ctx, _ = make_tiny_pair(tiny_inputs)
    _, _, _, prefix = tiny_inputs
    with pytest.raises(RuntimeError):
        ctx.spd_sample([0.5], 0.9, 1.0)               # before prefill
    ctx.spd_prefill(prefix)
    for bad in (([1.0], 0.9, 1.0), ([-0.1], 0.9, 1.0), ([0.5], 0.0, 1.0), ([0.5], 1.5, 1.0), ([0.5], 0.9, 0.0)):
        with pytest.raises(RuntimeError):
            ctx.spd_sample(*bad)
    ctx.spd_sample([0.5], 0.9, 1.0)
    ctx.spd_step()
    with pytest.raises(RuntimeError):
        ctx.spd_sample([0.5], 0.9, 1.0)               # drafts are under way: no splice any more


@pytest.mark.parametrize("kv", ["f32", "bf16"])
def test_spd_spliced_onto_a_sampled_prefix(tiny_inputs, kv):
    """Sample 10 tokens one call at a time, checking every draw and every pass against the oracle fed the same
    tokens; then the first timestep on prefix + sample and four SPD steps."""
    wl, _, _, prefix = tiny_inputs
    ctx, orc = make_tiny_pair(tiny_inputs, kv_dtype=kv)
    ctx.spd_prefill(prefix)
    top_p, temperature = 0.9, 0.25
    us = uniforms(10, 4)
    seq = list(prefix)
    exact = 0
    for u in us:
        z = ctx.spd_debug_read("LOGITS")
        new, ids, g = ctx.spd_sample([u], top_p, temperature)
        want, ok = accepted(z, temperature, top_p, float(u))
        assert int(new[0]) in ok
        exact += int(new[0]) == want
        seq.append(int(new[0]))
    assert exact >= 8
    stats = []
    compare_first_step(ctx, orc, seq, stats, device=(ids, g))     # includes the logits of the last sampled token's pass
    for _ in range(4):
        compare_step(ctx, orc, stats)
    assert max(s["eps_z"] for s in stats if "eps_z" in s) <= LOGIT_TOL


def test_one_launch_equals_single_draws(tiny_inputs):
    _, _, _, prefix = tiny_inputs
    a, _ = make_tiny_pair(tiny_inputs)
    b, _ = make_tiny_pair(tiny_inputs)
    us = uniforms(7, 8)
    a.spd_prefill(prefix)
    b.spd_prefill(prefix)
    one = []
    for u in us:
        new, ids_a, g_a = a.spd_sample([u], 0.92, 0.5)
        one.append(int(new[0]))
    new_b, ids_b, g_b = b.spd_sample(us, 0.92, 0.5)
    assert new_b.tolist() == one
    assert ids_a.tolist() == ids_b.tolist() and np.array_equal(g_a, g_b)
    assert np.array_equal(a.spd_debug_read("LOGITS"), b.spd_debug_read("LOGITS"))
    # and the drafts that follow are the same
    ta, _, _ = a.spd_generate(5, 6)
    tb, _, _ = b.spd_generate(5, 6)
    assert ta.tolist() == tb.tolist()


def test_n_sampled_prefixes_times_k_drafts(tiny_inputs):
    """NS_SPDk (Section 4.5): n nucleus-sampled continuations of one prefix, each extended by k superposed
    drafts, from n contexts over the same weights and tables.  Interleaving the contexts' calls changes nothing:
    each gives what it gives alone, and different random numbers give different continuations."""
    import paper_2405_18400_b200 as P

    wl, weights, tables, prefix = tiny_inputs
    packed = P.pack_weights(weights, "cuda:0")
    dtabs = P.build_ngram_tables(tables, "cuda:0")
    n, k, n_new, steps = 3, wl.k, 5, 4

    def make():
        return P.SpdContext(wl.shape, packed, dtabs, k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, wl.max_pos, "bf16")

    us = [uniforms(n_new, 100 + i) for i in range(n)]
    alone = []
    for i in range(n):
        c = make()
        c.spd_prefill(prefix)
        new, _, _ = c.spd_sample(us[i], 0.9, 0.3)
        toks, lp, g = c.spd_generate(steps, steps + 1)
        alone.append((new.tolist(), toks.tolist(), lp.tolist()))
        c.close()
    ctxs = [make() for _ in range(n)]
    for c in ctxs:
        c.spd_prefill(prefix)
    news, hist = [], []
    for i, c in enumerate(ctxs):
        new, ids, _ = c.spd_sample(us[i], 0.9, 0.3)
        news.append(new.tolist())
        hist.append([[int(t)] for t in ids])
    for _ in range(steps):                      # one step of every context in turn
        for i, c in enumerate(ctxs):
            ids, par, _ = c.spd_step()
            hist[i] = [hist[i][int(par[r])] + [int(ids[r])] for r in range(k)]
    for i, c in enumerate(ctxs):
        assert news[i] == alone[i][0] and hist[i] == alone[i][1]
        assert c.spd_debug_read("LOGP").tolist() == alone[i][2]
        c.close()
    assert len({tuple(a[0]) for a in alone}) > 1
    drafts = {tuple(row) for a in alone for row in a[1]}
    assert len(drafts) >= n * k - 1             # n k drafts, (nearly) all distinct
