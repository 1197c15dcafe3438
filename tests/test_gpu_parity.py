"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element on seeded inputs."""
import numpy as np
import pytest
import torch

import spd_inputs as si
from oracle import spd_oracle as so
from tests.gpu_common import (GAMMA_TOL, LOGIT_TOL, compare_first_step, compare_step, make_pair, make_tiny_pair)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kv_dtype", ["bf16", "f32"])
def test_tiny_workload_stepwise(tiny_inputs, kv_dtype):
    wl, weights, tables, prefix = tiny_inputs
    ctx, orc = make_tiny_pair(tiny_inputs, kv_dtype=kv_dtype)
    ctx.spd_debug_trace(True)
    stats = []
    compare_first_step(ctx, orc, prefix, stats)
    tr, tr_o = ctx.spd_debug_read("TRACE").astype(np.float64), orc.trace()
    assert np.abs(tr - tr_o).max() < 1e-3
    for _ in range(wl.gen_tokens - 1):
        compare_step(ctx, orc, stats)
        assert np.abs(ctx.spd_debug_read("TRACE").astype(np.float64) - orc.trace()).max() < 1e-3
    errs = [s for s in stats if "eps_z" in s]
    assert max(s["eps_z"] for s in errs) < 2e-4           # far inside the 2e-2 bound when quantisation points agree
    if max(s["eps_z"] for s in errs) <= 2e-5:
        assert max(s["dgamma"] for s in errs) <= GAMMA_TOL
    toks, lp, g = ctx.spd_generate(1, wl.gen_tokens + 1)
    ids_o, par_o, g_o = orc.step()
    assert np.array_equal(toks, orc.drafts()[:, len(prefix):])
    ctx.close()


@pytest.mark.parametrize("k", [1, 2, 5, 16])
def test_draft_counts(tiny_inputs, k):
    wl, weights, tables, prefix = tiny_inputs
    ctx, orc = make_tiny_pair(tiny_inputs, k=k)
    compare_first_step(ctx, orc, prefix)
    for _ in range(4):
        ids, par, g = compare_step(ctx, orc)
        assert abs(float(g.sum()) - 1.0) < 1e-5 and np.all(np.diff(g) <= 0)
    ctx.close()


def test_one_launch_generate_equals_single_steps(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    a, orc = make_tiny_pair(tiny_inputs)
    b, _ = make_tiny_pair(tiny_inputs)
    a.spd_prefill(prefix)
    b.spd_prefill(prefix)
    hist = [[int(t)] for t in a.spd_debug_read("CAND_TOK")]
    for _ in range(6):
        ids, par, g = a.spd_step()
        hist = [hist[int(par[r])] + [int(ids[r])] for r in range(a.k)]
    toks, lp, g2 = b.spd_generate(6, 7)
    assert toks.tolist() == hist
    assert np.array_equal(g, g2) and np.array_equal(lp, a.spd_debug_read("LOGP"))       # bit-identical
    assert np.array_equal(a.spd_debug_read("LOGITS"), b.spd_debug_read("LOGITS"))
    pre = (len(prefix) + 15) // 16                  # prefill: 16 tokens per launch
    assert a.spd_launch_count() == pre + 6 and b.spd_launch_count() == pre + 1
    # and again from the start on the same context: prefill restarts it
    b.spd_prefill(prefix)
    toks2, lp2, g3 = b.spd_generate(6, 7)
    assert np.array_equal(toks, toks2) and np.array_equal(lp, lp2)
    a.close(); b.close()


def test_long_context_uses_split_attention(tiny_inputs):
    """A 200-token prefix makes the attention phase split each head's positions over several blocks."""
    wl, weights, tables, _ = tiny_inputs
    prefix = si.make_prefix("zipf", 200, wl.shape.vocab, 1.1, seed=7)
    ctx, orc = make_tiny_pair(tiny_inputs, max_pos=256)
    compare_first_step(ctx, orc, prefix)
    for _ in range(3):
        compare_step(ctx, orc)
    ctx.close()


@pytest.mark.parametrize("m", [1, 2, 16, 17, 18, 33, 49])
def test_prefill_chunk_boundaries(tiny_inputs, m):
    """The batched prefill takes 16 prefix tokens per launch, the last launch ending with the LM head and the
    first timestep: prefix lengths around those boundaries (one token, a full launch, one token over, several).  A
    context of 128 positions has no long-prefix buffers, so every token goes through this kernel."""
    wl, _, _, _ = tiny_inputs
    prefix = si.make_prefix("zipf", m, wl.shape.vocab, 1.1, seed=30 + m)
    ctx, orc = make_tiny_pair(tiny_inputs, max_pos=128)
    compare_first_step(ctx, orc, prefix)
    assert ctx.spd_launch_count() == (m + 15) // 16
    compare_step(ctx, orc)
    ctx.close()


def test_odd_shape_model():
    """head_dim 96, d_ffn not a multiple of the thread count, vocabulary not divisible by the grid."""
    shape = si.ModelShape("odd", 1, 192, 2, 200, 1000)
    weights = si.make_weights(shape, seed=4)
    tables = si.make_ngram_tables(shape.vocab, 1.1, 50_000, (2, 3), 5000, seed=8)
    lam = [0.3, 0.2] + [0.0] * 6
    ctx, orc = make_pair(shape, weights, tables, 4, (2, 3), lam, 0.4, 0.2, 0.05, 64, "f32")
    prefix = si.make_prefix("uniform", 9, shape.vocab, seed=9)
    compare_first_step(ctx, orc, prefix)
    for _ in range(5):
        compare_step(ctx, orc)
    ctx.close()


def test_head_dim_128_long_context():
    """head_dim 128 with a bf16 cache takes the attention fast path (half a warp per position, eight positions
    in flight per warp); a 300-token prefix spreads every head over several blocks and rounds, in the decode
    kernel and in the prefill kernel (position ranges merged by the last block to arrive)."""
    shape = si.ModelShape("hd128", 2, 256, 2, 512, 1000)
    weights = si.make_weights(shape, seed=11)
    tables = si.make_ngram_tables(shape.vocab, 1.1, 50_000, (2, 3), 5000, seed=12)
    lam = [0.3, 0.2] + [0.0] * 6
    ctx, orc = make_pair(shape, weights, tables, 3, (2, 3), lam, 0.4, 0.2, 0.05, 512, "bf16")
    for n in (1, 7, 260, 300):     # 260 = 16 launches of 16 tokens + one of 4: a split prefill attention with an empty token half
        prefix = si.make_prefix("zipf", n, shape.vocab, 1.1, seed=13 + n)
        compare_first_step(ctx, orc, prefix)
        for _ in range(4):
            compare_step(ctx, orc)
    ctx.close()


def _hit_case(tables, rng, k, vocab):
    big = tables[-1]
    n = int(big["n"])
    keys = big["keys"].numpy()
    rows = keys[rng.integers(0, keys.shape[0], size=k)]
    hist = np.concatenate([rng.integers(0, vocab, size=(k, 8 - (n - 1))), rows[:, : n - 1]], axis=1).astype(np.int32)
    cand = list(dict.fromkeys(int(rows[i % k, n - 1]) for i in range(max(1, k // 2))))
    while len(cand) < k:
        t = int(rng.integers(0, vocab))
        if t not in cand:
            cand.append(t)
    return hist, np.array(cand, np.int32)


@pytest.mark.parametrize("k", [2, 3, 5, 8, 16])
def test_scoring_stage_with_ngram_hits(tiny_inputs, k):
    """Random-weight models rarely hit the tables, so the hit path is driven directly: histories end
    in stored contexts and kept tokens include stored continuations (Eq. 5-7, Eq. 2, Eq. 4)."""
    wl, weights, tables, prefix = tiny_inputs
    ctx, orc = make_tiny_pair(tiny_inputs, k=k)
    rng = np.random.default_rng(100 + k)
    hits = 0
    for trial in range(12):
        hist, cand = _hit_case(tables, rng, k, wl.shape.vocab)
        if trial % 3 == 0:
            hist[k - 1] = rng.integers(0, wl.shape.vocab, size=8)
        hist_len = 8 if trial % 4 else 2                       # short histories skip the longer orders
        hist = np.ascontiguousarray(hist[:, 8 - hist_len:])
        logP = (-rng.random(k) * 3).astype(np.float32)
        cand_lp = np.sort((-rng.random(k) * 4).astype(np.float32))[::-1].copy()
        ctx.spd_debug_score(hist, logP, cand, cand_lp)
        want = so.score_stage(orc.cfg, orc.tables, hist, logP, cand, cand_lp)
        assert np.array_equal(ctx.spd_debug_read("CNT")[:, :3], want["cnt"])
        assert np.array_equal(ctx.spd_debug_read("TOT")[:, :3], want["tot"])
        hits += int((want["cnt"] > 0).sum())
        assert np.abs(ctx.spd_debug_read("PNG") - want["png"]).max() < 1e-6
        sc = ctx.spd_debug_read("SCORE").astype(np.float64)
        fin = np.isfinite(want["score"])
        assert np.array_equal(np.isfinite(sc), fin)
        assert np.abs(sc[fin] - want["score"][fin]).max() < 2e-5
        srt = np.sort(want["score"][fin])[::-1][: k + 1]
        if np.min(-np.diff(srt)) > 1e-4:
            assert ctx.spd_debug_read("SEL").tolist() == want["sel"].tolist()
            assert np.abs(ctx.spd_debug_read("LOGP") - want["logP"]).max() < 2e-5
    assert hits > 10
    ctx.close()


def test_every_stored_ngram_is_found_and_absent_ones_miss(tiny_inputs):
    wl, weights, tables, prefix = tiny_inputs
    k = 16
    ctx, orc = make_tiny_pair(tiny_inputs, k=k)
    rng = np.random.default_rng(77)
    for ti, t in enumerate(tables):
        n = int(t["n"])
        keys = t["keys"].numpy()
        cnts = t["counts"].numpy()
        for _ in range(6):
            idx = rng.integers(0, keys.shape[0], size=k)
            hist = np.ascontiguousarray(keys[idx, : n - 1]).astype(np.int32)
            cand = np.array(sorted(set(keys[idx, n - 1].tolist())), np.int32)
            while cand.size < k:
                c = int(rng.integers(0, wl.shape.vocab))
                if c not in cand:
                    cand = np.append(cand, np.int32(c))
            ctx.spd_debug_score(hist, np.zeros(k, np.float32), cand, np.zeros(k, np.float32))
            cnt = ctx.spd_debug_read("CNT").reshape(k, k, 8)
            want = so.score_stage(orc.cfg, orc.tables, hist, np.zeros(k), cand, np.zeros(k))
            assert np.array_equal(cnt[:, :, :3].reshape(k * k, 3), want["cnt"])
            for i in range(k):
                j = int(np.where(cand == keys[idx[i], n - 1])[0][0])
                assert cnt[i, j, ti] == cnts[idx[i]]
    ctx.close()


def test_counts_beyond_two_to_the_31(tiny_inputs):
    """Counts and context totals of a web-scale corpus pass 2^31: the device reads them as unsigned 32-bit numbers
    (a 3e9 total, a 4e9 count), and the n-gram probability is their ratio as in the oracle."""
    wl, weights, _, prefix = tiny_inputs
    big_tables = [{"n": 2, "keys": torch.tensor([[5, 7], [5, 9], [6, 7]], dtype=torch.int32),
                   "counts": torch.tensor([2_500_000_000, 500_000_000, 4_000_000_000], dtype=torch.int64)},
                  {"n": 3, "keys": torch.tensor([[4, 5, 7], [4, 5, 9]], dtype=torch.int32),
                   "counts": torch.tensor([2_147_483_648, 2_147_483_646], dtype=torch.int64)}]
    k = 3
    ctx, orc = make_tiny_pair(tiny_inputs, k=k, tables=big_tables + [{"n": 4, "keys": torch.zeros((0, 4), dtype=torch.int32),
                                                                      "counts": torch.zeros(0, dtype=torch.int64)}])
    hist = np.array([[1, 2, 3, 4, 5], [1, 2, 3, 4, 6], [1, 2, 3, 9, 5]], np.int32)
    cand = np.array([7, 9, 11], np.int32)
    logP = np.array([-0.1, -0.2, -0.3], np.float32)
    cand_lp = np.array([-0.5, -0.7, -0.9], np.float32)
    ctx.spd_debug_score(hist, logP, cand, cand_lp)
    want = so.score_stage(orc.cfg, orc.tables, hist, logP, cand, cand_lp)
    cnt, tot = ctx.spd_debug_read("CNT")[:, :3], ctx.spd_debug_read("TOT")[:, :3]
    assert np.array_equal(cnt, want["cnt"]) and np.array_equal(tot, want["tot"])
    assert tot[0, 0] == 3_000_000_000 and cnt[3, 0] == 4_000_000_000 and tot[0, 1] == 4_294_967_294
    assert np.abs(ctx.spd_debug_read("PNG") - want["png"]).max() < 1e-6
    sc = ctx.spd_debug_read("SCORE").astype(np.float64)
    fin = np.isfinite(want["score"])
    assert np.array_equal(np.isfinite(sc), fin) and np.abs(sc[fin] - want["score"][fin]).max() < 2e-5
    assert ctx.spd_debug_read("SEL").tolist() == want["sel"].tolist()
    ctx.close()


def test_self_generated_corpus_gives_hits_end_to_end(tiny_inputs):
    """Tables counted over text the model itself produces (greedy continuations of random prefixes)
    make the n-gram lookups hit during real decoding, so the interpolation path runs end to end."""
    wl, weights, tables, prefix = tiny_inputs
    empty = [{"n": n, "keys": np.zeros((0, n), np.int32), "counts": np.zeros(0, np.int64)} for n in wl.orders]
    cfg1 = so.make_config(wl.shape, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64, "bf16")
    stream = []
    for s in range(6):
        pf = prefix if s == 0 else si.make_prefix("uniform", 16, wl.shape.vocab, seed=50 + s)
        o = so.Oracle(cfg1, weights, empty)
        o.prefill(pf)
        for _ in range(10):
            o.step()
        for row in o.drafts():
            stream += row.tolist()
    st = torch.tensor(stream, dtype=torch.int64)
    own = [si.count_ngrams(st, n) for n in wl.orders]
    ctx, orc = make_tiny_pair(tiny_inputs, tables=own)
    compare_first_step(ctx, orc, prefix)
    hits = 0
    for _ in range(8):
        compare_step(ctx, orc)
        hits += int((ctx.spd_debug_read("CNT")[:, :3] > 0).sum())
    assert hits > 0
    ctx.close()


@pytest.mark.parametrize("kv_dtype", ["bf16", "f32"])
def test_resets_restart_from_a_chosen_draft(tiny_inputs, kv_dtype):
    """Section 5.3: every few steps one draft is chosen and generation restarts from it.  The device keeps the
    original prefix's cache and recomputes the generated positions from the draft's tokens; the oracle
    recomputes everything from prefix + draft."""
    wl, weights, tables, prefix = tiny_inputs
    ctx, orc = make_tiny_pair(tiny_inputs, kv_dtype=kv_dtype, max_pos=64)
    compare_first_step(ctx, orc, prefix)
    for draft in (1, 0, 2):
        for _ in range(3):
            compare_step(ctx, orc)
        before = orc.drafts()[draft].tolist()
        compare_first_step(ctx, orc, None, reset_draft=draft)
        assert orc.drafts()[:, :-1].tolist() == [before] * 3          # the chosen draft is now everyone's prefix
        toks, lp, g = ctx.spd_generate(1, 2)                          # history restarts after a reset
        orc.step()
        assert np.array_equal(toks, orc.drafts()[:, len(before):])
        compare_first_step(ctx, orc, before)                          # and a plain prefill on the longer prefix agrees too
    import paper_2405_18400_b200 as P
    with pytest.raises(P.SpdError) as e:
        ctx.spd_reset(3)
    assert e.value.status == -3
    ctx.close()


def test_call_order_and_range_errors(tiny_inputs):
    import paper_2405_18400_b200 as P
    wl, weights, tables, prefix = tiny_inputs
    ctx, _ = make_tiny_pair(tiny_inputs, max_pos=24)
    with pytest.raises(P.SpdError) as e:
        ctx.spd_step()
    assert e.value.status == -2
    with pytest.raises(P.SpdError) as e:
        ctx.spd_prefill([0, 5000])
    assert e.value.status == -3
    with pytest.raises(P.SpdError) as e:
        ctx.spd_prefill(list(range(24)))
    assert e.value.status == -3
    ctx.spd_prefill(prefix)                    # 16 positions used, 8 left
    with pytest.raises(P.SpdError) as e:
        ctx.spd_generate(9, 10)
    assert e.value.status == -3
    toks, lp, g = ctx.spd_generate(8, 9)
    assert toks.shape == (3, 9)
    with pytest.raises(P.SpdError) as e:
        ctx.spd_step()
    assert e.value.status == -3
    ctx.close()


@pytest.mark.parametrize("images", [False, True])
def test_ring_settings_do_not_change_results(tiny_inputs, images):
    wl, weights, tables, prefix = tiny_inputs
    ctx, _ = make_tiny_pair(tiny_inputs, images=images)
    ctx.spd_prefill(prefix)
    base, lp0, _ = ctx.spd_generate(5, 6)
    z0 = ctx.spd_debug_read("LOGITS")
    for sb, ns in [(2048, 2), (4096, 16), (65536, 3)]:
        ctx.spd_set_ring(sb, ns)
        ctx.spd_prefill(prefix)
        toks, lp, _ = ctx.spd_generate(5, 6)
        assert np.array_equal(toks, base)
        # with fragment-order images the stage size decides which warp adds which products of a row: the sums differ
        # in their last bits, and five timesteps carry that forward
        assert np.abs(ctx.spd_debug_read("LOGITS") - z0).max() < (1e-3 if images else 1e-4)
    import paper_2405_18400_b200 as P
    with pytest.raises(P.SpdError):
        ctx.spd_set_ring(1024, 4)              # a 688-column row (1376 bytes) does not fit
    ctx.close()


def test_fragment_order_image_layout():
    """spd_pack_image against its definition: vector 4 g + t of a block of 8 rows x 32 columns holds row g's column
    pairs 2t, 2t+8, 2t+16, 2t+24; blocks of a unit in column order, units in row order."""
    import torch
    import paper_2405_18400_b200 as P
    from paper_2405_18400_b200.binding import _image

    rows, cols = 24, 96
    w = torch.arange(rows * cols, dtype=torch.int16, device="cuda:0").view(torch.bfloat16).reshape(rows, cols)
    img = _image(w)
    torch.cuda.synchronize()
    got = img.view(torch.int16).cpu().numpy().reshape(-1)
    src = np.arange(rows * cols, dtype=np.int16).reshape(rows, cols)
    want = np.empty(rows * cols, np.int16)
    at = 0
    for unit in range(rows // 8):
        for blk in range(cols // 32):
            for lane in range(32):
                g, t = lane // 4, lane % 4
                for q in range(4):
                    c = blk * 32 + 2 * t + 8 * q
                    want[at: at + 2] = src[unit * 8 + g, c: c + 2]
                    at += 2
    assert np.array_equal(got, want)
    assert P.load_library().spd_pack_image(w.data_ptr(), 20, 96, img.data_ptr(), None) == -1    # rows must be a multiple of 8
    assert P.load_library().spd_pack_image(w.data_ptr(), 24, 80, img.data_ptr(), None) == -1    # columns a multiple of 32


def test_steps_without_images_match_oracle(tiny_inputs):
    """The float32 multiply loop (contexts whose weights come without fragment-order images) against the oracle."""
    ctx, orc = make_tiny_pair(tiny_inputs, images=False)
    wl, weights, tables, prefix = tiny_inputs
    compare_first_step(ctx, orc, prefix)
    for _ in range(4):
        compare_step(ctx, orc)
    ctx.close(); orc.close()


def test_malformed_table_is_reported_not_hung(tiny_inputs):
    """A table image without a single empty slot (never produced by spd_ngram_build) makes the probe of an absent
    key run to its bound: the step returns SPD_ETABLE, nothing hangs, and the context works again afterwards
    with a sound table."""
    import paper_2405_18400_b200 as P
    wl, weights, tables, prefix = tiny_inputs
    good = P.build_ngram_tables(tables, "cuda:0")
    slots = 1 << 15
    img = np.zeros((slots, 4), np.uint32)
    img[:, 0] = np.arange(slots, dtype=np.uint32) | 0xfff00000          # keys no lookup asks for (token ids >= 4096)
    img[:, 3] = 1
    bad = [dict(t) for t in good]
    bad[0] = {"n": 2, "ngram_slots": slots, "ctx_slots": slots,
              "ngram": torch.from_numpy(img.view(np.uint8).reshape(-1)).to("cuda:0"),
              "ctx": torch.from_numpy(img.view(np.uint8).reshape(-1)).to("cuda:0")}
    packed = P.pack_weights(weights, "cuda:0")
    ctx = P.SpdContext(wl.shape, packed, bad, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64)
    ctx.spd_prefill(prefix)                     # the first timestep does not touch the tables
    with pytest.raises(P.SpdError) as e:
        ctx.spd_step()
    assert e.value.status == -6
    with pytest.raises(P.SpdError) as e:        # the failed run invalidated the drafts
        ctx.spd_step()
    assert e.value.status == -2
    ctx.close()
    ok = P.SpdContext(wl.shape, packed, good, 3, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, 64)
    ok.spd_prefill(prefix)
    ids, par, g = ok.spd_step()
    assert abs(float(g.sum()) - 1) < 1e-5
    ok.close()


def test_expired_wait_is_reported_and_the_context_stays_usable(tiny_inputs):
    """One block withholds its arrival at a grid barrier of the prefill kernel: every other block's bounded wait
    runs out, the kernel ends by itself, the host reads SPD_ETIMEOUT, and the same context then decodes as a fresh
    one does."""
    import time
    wl, weights, tables, prefix = tiny_inputs
    ctx, _ = make_tiny_pair(tiny_inputs)
    ref, _ = make_tiny_pair(tiny_inputs)
    ids0, g0 = ref.spd_prefill(prefix)
    t0 = time.perf_counter()
    status = ctx.spd_debug_expire()
    dt = time.perf_counter() - t0
    assert status == -7
    assert 1.0 < dt < 10.0
    import paper_2405_18400_b200 as P
    with pytest.raises(P.SpdError) as e:            # no drafts to continue
        ctx.spd_step()
    assert e.value.status == -2
    ids, g = ctx.spd_prefill(prefix)
    assert ids.tolist() == ids0.tolist() and np.array_equal(g, g0)
    a, _, _ = ctx.spd_generate(4, 5)
    b, _, _ = ref.spd_generate(4, 5)
    assert a.tolist() == b.tolist()
    ctx.close(); ref.close()


@pytest.mark.parametrize("kv_dtype", ["f32", "bf16"])
def test_tiny_free_running(tiny_inputs, kv_dtype):
    """The whole tiny request (first timestep + 8 steps) with no forcing of the oracle: it never sees the device's
    cache or log-probabilities.  Every step is gated for both cache types: logits within 2e-2, kept tokens, counts,
    choices and parents exact (margin rule on near-ties), gamma within max(1e-4, accumulated 4 eps / tau).  Then the
    same request as one launch of all steps gives the same drafts."""
    from tests.gpu_common import free_run, show_run

    wl, weights, tables, prefix = tiny_inputs
    ctx, orc = make_tiny_pair(tiny_inputs, kv_dtype=kv_dtype)
    rec = free_run(ctx, orc, prefix, wl.gen_tokens)
    show_run("tiny free-running, %s cache" % kv_dtype, rec)
    assert len(rec) == wl.gen_tokens + 1
    assert all(r["logits_ok"] and r["ints_ok"] and r["gamma_ok"] for r in rec)
    toks = orc.drafts()[:, len(prefix):]
    ctx.spd_prefill(prefix)
    got, lp, g = ctx.spd_generate(wl.gen_tokens, wl.gen_tokens + 1)
    assert np.array_equal(got, toks) and np.abs(g - orc.gamma()).max() <= max(GAMMA_TOL, rec[-1]["acc"])
    ctx.close()


def test_stop_token_ends_the_run(tiny_inputs):
    """Algorithm 1 generates "until max generation length or stop token".  With the stop token set to the token the
    oracle's most probable draft emits at its fourth step, one launch asked for eight steps ends after that step on
    the device as in the oracle's loop: same length, same drafts, the context reports itself finished and refuses
    further steps until it is prefilled again; step-by-step calls stop at the same place."""
    import paper_2405_18400_b200 as P

    wl, weights, tables, prefix = tiny_inputs
    _, orc = make_tiny_pair(tiny_inputs, kv_dtype="f32")
    orc.prefill(prefix)
    tops = []
    for _ in range(6):
        ids, _, _ = orc.step()
        tops.append(int(ids[0]))
    eos = tops[3]
    want_steps = tops.index(eos) + 1
    orc.prefill(prefix)
    assert orc.generate(8, eos) == want_steps
    want = orc.drafts()[:, len(prefix):]
    packed = P.pack_weights(weights, "cuda:0")
    dtabs = P.build_ngram_tables(tables, "cuda:0")
    ctx = P.SpdContext(wl.shape, packed, dtabs, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, wl.max_pos, "f32",
                       eos_id=eos)
    ctx.spd_prefill(prefix)
    assert not ctx.spd_finished()
    toks, lp, g = ctx.spd_generate(8, 9)
    assert toks.shape == (wl.k, 1 + want_steps) and np.array_equal(toks, want)
    assert ctx.spd_finished() and abs(float(g.sum()) - 1) < 1e-5
    assert np.abs(g - orc.gamma()).max() < 1e-3
    with pytest.raises(P.SpdError) as e:
        ctx.spd_step()
    assert e.value.status == -2
    # the same by single steps; a fresh prefill clears the flag
    ctx.spd_prefill(prefix)
    assert not ctx.spd_finished()
    n = 0
    while not ctx.spd_finished():
        ids, par, g2 = ctx.spd_step()
        n += 1
        assert n <= 8
    assert n == want_steps and int(ids[0]) == eos and np.array_equal(g, g2)
    # a stop token that never comes changes nothing
    never = next(t for t in range(wl.shape.vocab) if t not in want and t not in tops)
    ctx2 = P.SpdContext(wl.shape, packed, dtabs, wl.k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, wl.max_pos, "f32",
                        eos_id=never)
    ctx2.spd_prefill(prefix)
    toks2, _, _ = ctx2.spd_generate(want_steps, 1 + want_steps)
    assert np.array_equal(toks2, want) and not ctx2.spd_finished()
    ctx.close(); ctx2.close()


def test_image_and_row_major_paths_agree_at_7b_width():
    """Two layers at the 7B shape's width (4096 / 11008 columns, head size 128): the decode steps of a context with
    fragment-order weight images (tensor-core multiply, 8-row units, two stages per unit) and of one without (float32
    loop for every matrix) give the same drafts and logits that differ by float rounding only."""
    import paper_2405_18400_b200 as P

    shape = si.ModelShape("w7b", 2, 4096, 32, 11008, 2000)
    dev = torch.device("cuda:0")
    weights = si.make_weights(shape, seed=61, device=dev)
    tables = si.make_ngram_tables(shape.vocab, 1.1, 100_000, (2, 3, 4, 5, 6), 5000, seed=62)
    lam = [0.01, 0.04, 0.15, 0.18, 0.12, 0.0, 0.0, 0.0]
    dtabs = P.build_ngram_tables(tables, dev)
    prefix = si.make_prefix("zipf", 15, shape.vocab, 1.1, seed=63)
    out = []
    for images in (True, False):
        packed = P.pack_weights(weights, dev, images=images)
        assert ("lm_head_img" in packed) == images
        # a float32 cache: with a bf16 cache the two paths' float differences flip cache roundings, which six
        # free-running steps carry forward (9e-4 on the logits)
        ctx = P.SpdContext(shape, packed, dtabs, 3, (2, 3, 4, 5, 6), lam, 0.54, 0.06, 0.01, 192, "f32")
        ctx.spd_prefill(prefix)
        toks, lp, g = ctx.spd_generate(6, 7)
        out.append((toks, lp, g, ctx.spd_debug_read("LOGITS")))
        ctx.close()
    assert np.array_equal(out[0][0], out[1][0])
    assert np.abs(out[0][3] - out[1][3]).max() < 1e-4
    assert np.abs(out[0][2] - out[1][2]).max() < 1e-4
