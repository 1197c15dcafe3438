"""Prefixes of more than 32 tokens: all but the last 1..16 tokens go through the tensor-core path (tcgen05
products over tiles of 128 tokens, up to 512 tokens per job), the rest through the 16-token prefill kernel,
which ends with the first timestep (Eq. 1).  Both fill the same cache; the first timestep and the steps after
it are compared with the oracle as for short prefixes."""
import numpy as np
import pytest

import spd_inputs as si
from tests.gpu_common import compare_first_step, compare_step, make_pair, make_tiny_pair

pytestmark = pytest.mark.gpu


def _expected_launches(m, layers, job_tokens):
    tc = m - ((m - 1) % 16 + 1) if m > 32 else 0
    jobs = -(-tc // job_tokens) if tc else 0
    return jobs * 9 * layers + (m - tc + 15) // 16


@pytest.mark.parametrize("kv_dtype", ["bf16", "f32"])
@pytest.mark.parametrize("m", [33, 64, 65, 129, 145, 293, 700])
def test_long_prefix_tiny(tiny_inputs, m, kv_dtype):
    """Tiny shape: d_ffn = 688 leaves a ragged last 64-column stage and 2 d_ffn = 1376 a ragged last row tile;
    33 = the shortest prefix that takes the path (a job of 17 tokens: jobs of up to 128 tokens take the product made
    for few token rows, with token boxes of 16, 32, 64 or 128 rows), 64 and 65 = jobs of 48 and 64 tokens, 129 = 128
    tokens, 145 = 129 tokens (the shortest job on the 128-token tiles), 293 = one job of 288 tokens (a last tile of
    32), 700 = a job of 512 tokens and one of 176."""
    wl, _, _, _ = tiny_inputs
    prefix = si.make_prefix("zipf", m, wl.shape.vocab, 1.1, seed=500 + m)
    ctx, orc = make_tiny_pair(tiny_inputs, max_pos=1024, kv_dtype=kv_dtype)
    compare_first_step(ctx, orc, prefix)
    assert ctx.spd_launch_count() == _expected_launches(m, wl.shape.n_layers, 512)
    for _ in range(3):
        compare_step(ctx, orc)
    # and once more on the same context (the term buffers and the cache are reused)
    prefix2 = si.make_prefix("zipf", 257, wl.shape.vocab, 1.1, seed=900 + m)
    compare_first_step(ctx, orc, prefix2)
    compare_step(ctx, orc)
    ctx.close()


def test_long_prefix_head_dim_128():
    """head_dim 128 (the 7B shapes' attention layout), bf16 cache; max_pos 300 caps a job at 256 tokens."""
    shape = si.ModelShape("hd128", 2, 256, 2, 512, 1000)
    weights = si.make_weights(shape, seed=11)
    tables = si.make_ngram_tables(shape.vocab, 1.1, 50_000, (2, 3), 5000, seed=12)
    lam = [0.3, 0.2] + [0.0] * 6
    for max_pos, m in ((300, 290), (1024, 1000)):
        ctx, orc = make_pair(shape, weights, tables, 3, (2, 3), lam, 0.4, 0.2, 0.05, max_pos, "bf16")
        prefix = si.make_prefix("zipf", m, shape.vocab, 1.1, seed=77 + m)
        compare_first_step(ctx, orc, prefix)
        assert ctx.spd_launch_count() == _expected_launches(m, 2, 256 if max_pos == 300 else 512)
        for _ in range(3):
            compare_step(ctx, orc)
        ctx.close()


def test_reset_after_long_prefix(tiny_inputs):
    """A restart from a draft (Section 5.3) recomputes only the generated positions on top of a cache that the
    long-prefix path filled."""
    wl, _, _, _ = tiny_inputs
    prefix = si.make_prefix("zipf", 300, wl.shape.vocab, 1.1, seed=321)
    ctx, orc = make_tiny_pair(tiny_inputs, max_pos=512)
    compare_first_step(ctx, orc, prefix)
    for _ in range(4):
        compare_step(ctx, orc)
    compare_first_step(ctx, orc, None, reset_draft=1)
    compare_step(ctx, orc)
    ctx.close()


def test_expired_wait_in_the_products_is_reported_and_the_context_stays_usable(tiny_inputs):
    """A stage of operands that never arrives: the issuing thread's bounded wait runs out, the block records
    SPD_ETIMEOUT, frees its tensor memory and ends by itself; the same context then prefills a long prefix as a
    fresh one does.  A context without the long-prefix path refuses the hook."""
    import time
    import paper_2405_18400_b200 as P
    wl, _, _, _ = tiny_inputs
    prefix = si.make_prefix("zipf", 300, wl.shape.vocab, 1.1, seed=77)
    ctx, _ = make_tiny_pair(tiny_inputs, max_pos=512)
    ref, _ = make_tiny_pair(tiny_inputs, max_pos=512)
    ids0, g0 = ref.spd_prefill(prefix)
    t0 = time.perf_counter()
    status = ctx.spd_debug_expire_products()
    dt = time.perf_counter() - t0
    assert status == -7
    assert 1.0 < dt < 10.0
    with pytest.raises(P.SpdError) as e:            # no drafts to continue
        ctx.spd_step()
    assert e.value.status == -2
    ids, g = ctx.spd_prefill(prefix)
    assert ids.tolist() == ids0.tolist() and np.array_equal(g, g0)
    a, _, _ = ctx.spd_generate(4, 5)
    b, _, _ = ref.spd_generate(4, 5)
    assert a.tolist() == b.tolist()
    small, _ = make_tiny_pair(tiny_inputs, max_pos=64)
    assert small.spd_debug_expire_products() == -2
    ctx.close(); ref.close(); small.close()


def test_long_prefix_13b_width():
    """Two layers at the 13B shape's width (d_model 5120, 40 heads of 128, d_ffn 13824): 80 and 216 stages per
    row (10 and 27 accumulator segments, so the four accumulators are reused several times), 120 / 40 / 216 / 40
    row tiles, a job of 512 tokens and a partial one."""
    import torch
    import paper_2405_18400_b200 as P
    from oracle import spd_oracle as so

    shape = si.ModelShape("w13b", 2, 5120, 40, 13824, 2000)
    dev = torch.device("cuda:0")
    weights = si.make_weights(shape, seed=21, device=dev)
    host = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in weights.items()}
    tables = si.make_ngram_tables(shape.vocab, 1.1, 50_000, (2, 3), 5000, seed=22)
    lam = [0.3, 0.2] + [0.0] * 6
    packed = P.pack_weights(weights, dev, consume=True)
    del weights
    dtabs = P.build_ngram_tables(tables, dev)
    ctx = P.SpdContext(shape, packed, dtabs, 3, (2, 3), lam, 0.4, 0.2, 0.05, 640, "bf16")
    cfg = so.make_config(shape, 3, (2, 3), lam, 0.4, 0.2, 0.05, 640, "bf16")
    orc = so.Oracle(cfg, host, sorted(tables, key=lambda t: int(t["n"])))
    m = 600
    prefix = si.make_prefix("zipf", m, shape.vocab, 1.1, seed=23)
    stats = []
    compare_first_step(ctx, orc, prefix, stats)
    assert ctx.spd_launch_count() == _expected_launches(m, 2, 512)
    for _ in range(2):
        compare_step(ctx, orc, stats)
    assert max(s["eps_z"] for s in stats if "eps_z" in s) < 2e-3
    ctx.close()
    orc.close()


def test_both_prefill_paths_agree(tiny_inputs):
    """The same 100-token prefix through the 16-token kernel alone (a context of 128 positions has no long-prefix
    buffers) and through the long-prefix path (a context of 512 positions): same drafts, logits equal to float
    rounding, and the same continuation."""
    wl, _, _, _ = tiny_inputs
    prefix = si.make_prefix("zipf", 100, wl.shape.vocab, 1.1, seed=4242)
    a, _ = make_tiny_pair(tiny_inputs, max_pos=128, kv_dtype="f32")
    b, _ = make_tiny_pair(tiny_inputs, max_pos=512, kv_dtype="f32")
    ids_a, g_a = a.spd_prefill(prefix)
    ids_b, g_b = b.spd_prefill(prefix)
    assert a.spd_launch_count() == 7 and b.spd_launch_count() == 9 * wl.shape.n_layers + 1
    za, zb = a.spd_debug_read("LOGITS"), b.spd_debug_read("LOGITS")
    assert np.abs(za - zb).max() < 1e-4
    assert ids_a.tolist() == ids_b.tolist() and np.abs(g_a - g_b).max() < 1e-3
    ta, _, _ = a.spd_generate(5, 6)
    tb, _, _ = b.spd_generate(5, 6)
    assert ta.tolist() == tb.tolist()
    a.close(); b.close()


def test_long_context_decode_7b_width():
    """The long-prefix workload's regime at the 7B shape's width (d_model 4096, 32 heads of 128, d_ffn 11008; two
    layers keep the CPU oracle's dense pass over 2048 tokens to half a minute): a 2048-token prefix through four
    jobs of the long-prefix path and one launch of the 16-token kernel, then decode steps over more than 2048
    cached positions, where every head's positions are split over four blocks (bf16 cache, 16-byte loads, eight
    positions in flight per warp) and the partial results merged."""
    import torch
    import paper_2405_18400_b200 as P
    from oracle import spd_oracle as so

    shape = si.ModelShape("w7b", 2, 4096, 32, 11008, 2000)
    dev = torch.device("cuda:0")
    weights = si.make_weights(shape, seed=31, device=dev)
    host = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in weights.items()}
    tables = si.make_ngram_tables(shape.vocab, 1.1, 50_000, (2, 3), 5000, seed=32)
    lam = [0.3, 0.2] + [0.0] * 6
    packed = P.pack_weights(weights, dev, consume=True)
    del weights
    dtabs = P.build_ngram_tables(tables, dev)
    ctx = P.SpdContext(shape, packed, dtabs, 3, (2, 3), lam, 0.4, 0.2, 0.05, 2304, "bf16")
    cfg = so.make_config(shape, 3, (2, 3), lam, 0.4, 0.2, 0.05, 2304, "bf16")
    orc = so.Oracle(cfg, host, sorted(tables, key=lambda t: int(t["n"])))
    m = 2048
    prefix = si.make_prefix("zipf", m, shape.vocab, 1.1, seed=33)
    stats = []
    compare_first_step(ctx, orc, prefix, stats)
    assert ctx.spd_launch_count() == _expected_launches(m, 2, 512)
    for _ in range(3):
        ids, par, g = compare_step(ctx, orc, stats)
        assert abs(float(g.sum()) - 1.0) < 1e-5
    assert max(s["eps_z"] for s in stats if "eps_z" in s) < 2e-3
    print("7B width, 2048-token prefix: max logit error %.3g; cache values rounded the other way: %s" % (
        max(s["eps_z"] for s in stats if "eps_z" in s), [(s["path"], s["cache_flips"]) for s in stats if "path" in s]))
    ctx.close()
    orc.close()


def test_prefix_of_64_tokens_13b_width():
    """A 64-token prefix at the 13B shape's width (the fifth workload's prefix): a long-prefix job of 48 tokens on the
    product made for few token rows, then one launch of the 16-token kernel; five drafts, then decode steps."""
    import torch
    import paper_2405_18400_b200 as P
    from oracle import spd_oracle as so

    shape = si.ModelShape("w13b", 2, 5120, 40, 13824, 2000)
    dev = torch.device("cuda:0")
    weights = si.make_weights(shape, seed=41, device=dev)
    host = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in weights.items()}
    tables = si.make_ngram_tables(shape.vocab, 1.05, 50_000, (2, 3), 5000, seed=42)
    lam = [0.3, 0.2] + [0.0] * 6
    packed = P.pack_weights(weights, dev, consume=True)
    del weights
    dtabs = P.build_ngram_tables(tables, dev)
    ctx = P.SpdContext(shape, packed, dtabs, 5, (2, 3), lam, 0.4, 0.2, 0.05, 256, "bf16")
    cfg = so.make_config(shape, 5, (2, 3), lam, 0.4, 0.2, 0.05, 256, "bf16")
    orc = so.Oracle(cfg, host, sorted(tables, key=lambda t: int(t["n"])))
    prefix = si.make_prefix("zipf", 64, shape.vocab, 1.05, seed=43)
    stats = []
    compare_first_step(ctx, orc, prefix, stats)
    assert ctx.spd_launch_count() == 9 * shape.n_layers + 1
    for _ in range(3):
        compare_step(ctx, orc, stats)
    assert max(s["eps_z"] for s in stats if "eps_z" in s) < 2e-3
    ctx.close()
    orc.close()
