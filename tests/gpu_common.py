"""Helpers shared by the GPU parity tests: build the CUDA context and the oracle on the same seeded
inputs, and compare one timestep with the margin rule."""
import math

import numpy as np

import spd_inputs as si
from oracle import spd_oracle as so

LOGIT_TOL = 2e-2      # max-abs logit tolerance (bf16 weights, fp32 accumulation)
GAMMA_TOL = 1e-4


def make_pair(shape, weights, tables, k, orders, lam, alpha, tau, delta, max_pos, kv_dtype="bf16", device="cuda:0",
              images=True):
    """images=False: no fragment-order weight images, so the decode timesteps run the float32 multiply loop."""
    import paper_2405_18400_b200 as P

    packed = P.pack_weights(weights, device, images=images)
    dtabs = P.build_ngram_tables(tables, device)
    ctx = P.SpdContext(shape, packed, dtabs, k, orders, lam, alpha, tau, delta, max_pos, kv_dtype)
    cfg = so.make_config(shape, k, orders, lam, alpha, tau, delta, max_pos, kv_dtype)
    orc = so.Oracle(cfg, weights, sorted(tables, key=lambda t: int(t["n"])))
    return ctx, orc


def make_tiny_pair(tiny_inputs, k=None, kv_dtype="bf16", max_pos=None, tables=None, alpha=None, delta=None, images=True):
    wl, weights, tabs, prefix = tiny_inputs
    return make_pair(wl.shape, weights, tabs if tables is None else tables, wl.k if k is None else k, wl.orders,
                     wl.lambdas(), wl.alpha if alpha is None else alpha, wl.tau, wl.delta if delta is None else delta,
                     wl.max_pos if max_pos is None else max_pos, kv_dtype, images=images)


def top_gap(values, k):
    """Smallest gap between neighbours among the k+1 largest float32 values (inf if fewer exist)."""
    v = np.sort(np.asarray(values, dtype=np.float32)[np.isfinite(values)])[::-1][: k + 1].astype(np.float64)
    return float(np.min(-np.diff(v))) if v.size > 1 else math.inf


U32 = 2.0 ** -24      # unit roundoff of float32

# Bound on the device's float error in a cache value before it is rounded to bf16, in units of
# U32 * (layers + 1) * rms(cache).  A cache value of layer l is a float32 dot product over d terms (error of a
# few U32 relative to the rms of the values, the partial sums being added as a tree) of a residual stream
# that carries the errors of the l layers before it, each of the same kind; the sum grows at most linearly in
# l.  Decode steps accumulate in float32 with round-to-nearest, or, with fragment-order weight images, in chains of
# at most 16 tensor-core instructions whose sums are then added in float32 (measured: need <= ~3 of these units); the
# prefill kernels accumulate inside the tensor cores, which truncate every addition of a 96-instruction chain
# (measured: need <= ~40 units).  The constants leave a factor of about four over what was measured.
SLACK_UNITS = {"decode": 12.0, "prefill": 160.0}
# Share of the new cache values that may round the other way (measured: 0.1 % on decode steps, 1 % in prefill).
FLIP_RATE = {"decode": 0.004, "prefill": 0.03}


def _follow(ctx, orc, positions, path):
    """With a bf16 cache the oracle adopts the device's cache values wherever they are a valid rounding of its
    own exact values (rounding is a decision float error can tip; the rest of the pass is then comparable)."""
    if orc.cfg.kv_dtype != 1:
        return False
    kc, vc = ctx.spd_debug_read("KCACHE", positions), ctx.spd_debug_read("VCACHE", positions)
    rms = math.sqrt(0.5 * (float(np.mean(kc.astype(np.float64) ** 2)) + float(np.mean(vc.astype(np.float64) ** 2))))
    orc._slack_unit = U32 * (orc.cfg.n_layers + 1) * rms
    orc.follow_cache(kc, vc, slack=SLACK_UNITS[path] * orc._slack_unit)
    return True


def _followed(orc, new_positions, stats, path):
    flips, bad = orc.follow_cache(None)
    total = 2 * orc.cfg.n_layers * orc.cfg.d_model * new_positions
    assert bad == 0, "%d cache values are not a rounding of the oracle's" % bad
    assert flips <= FLIP_RATE[path] * total + 8, (flips, total)
    if stats is not None:
        stats.append({"cache_flips": flips, "cache_values": total, "path": path,
                      "slack_units_needed": orc.follow_need / orc._slack_unit})


def _sync_logp(ctx, orc, eps_z):
    """Both sides continue from the same draft log-probabilities (checked first): at tau = 0.06 a logit
    difference e moves gamma by about 4 e / tau, which would otherwise change the next step's input."""
    lp, lp_o = ctx.spd_debug_read("LOGP").astype(np.float64), orc.logP()
    assert np.abs(lp - lp_o).max() <= 4 * eps_z / orc.cfg.tau + 1e-4 * max(1.0, np.abs(lp_o).max())
    orc.set_logP(lp)


def compare_first_step(ctx, orc, prefix, stats=None, reset_draft=None, device=None):
    """First timestep on both sides.  With reset_draft, the restart from that draft (Section 5.3) instead: the
    device recomputes only the generated positions, the oracle everything.  With device = (ids, gamma), the
    device has already taken its first timestep on `prefix` (after sampling its tail, Section 4.5)."""
    if device is not None:
        ids, g = device
    elif reset_draft is None:
        ids, g = ctx.spd_prefill(prefix)
    else:
        prefix = orc.drafts()[reset_draft].tolist()
        ids, g = ctx.spd_reset(reset_draft)
    following = _follow(ctx, orc, len(prefix), "prefill")
    ids_o, g_o = orc.prefill(prefix)
    if following:
        _followed(orc, len(prefix), stats, "prefill")
    z, z_o = ctx.spd_debug_read("LOGITS").astype(np.float64), orc.logits()
    eps_z = float(np.abs(z - z_o).max())
    assert eps_z <= LOGIT_TOL, eps_z
    k = ctx.k
    assert top_gap(z_o, k) > 2 * eps_z, "fixture has a near-tie among the top logits"
    assert ids.tolist() == ids_o.tolist()
    assert np.abs(ctx.spd_debug_read("CAND_LP") - orc.cand_lp()).max() <= 2 * eps_z / orc.cfg.tau + 1e-4
    assert np.abs(g - g_o).max() <= max(GAMMA_TOL, 4 * eps_z / orc.cfg.tau)
    if stats is not None:
        stats.append({"eps_z": eps_z, "dgamma": float(np.abs(g - g_o).max())})
    _sync_logp(ctx, orc, eps_z)
    return ids, g


def compare_step(ctx, orc, stats=None, stepped=None, path="decode"):
    """One later timestep on both sides.  Exact ids / parents / counts when the oracle's margins exceed
    twice the measured float error; otherwise the device's choice must be one the oracle rates within
    that error of its own, and the oracle follows it.  `stepped` = (ids, parents, gamma) when the device has
    already taken the step (as one request of a batch); `path` names the kernels that wrote the new cache row."""
    k = ctx.k
    tau, alpha = orc.cfg.tau, orc.cfg.alpha
    hist_o = orc.drafts()
    logP_o = orc.logP()
    ids, par, g = ctx.spd_step() if stepped is None else stepped
    following = _follow(ctx, orc, orc.T() + 1, path)
    orc.step_forward()
    if following:
        _followed(orc, 1, stats, path)
    z, z_o = ctx.spd_debug_read("LOGITS").astype(np.float64), orc.logits()
    eps_z = float(np.abs(z - z_o).max())
    assert eps_z <= LOGIT_TOL, eps_z
    assert top_gap(z_o, k) > 2 * eps_z, "fixture has a near-tie among the top logits"
    cand = ctx.spd_debug_read("CAND_TOK")
    assert cand.tolist() == orc.cand_tok().tolist()
    cand_lp = ctx.spd_debug_read("CAND_LP").astype(np.float64)
    assert np.abs(cand_lp - orc.cand_lp()).max() <= 2 * eps_z / tau + 1e-4
    # the device scored the same drafts
    win = ctx.spd_debug_read("HIST_IN")
    w = min(8, hist_o.shape[1])
    assert np.array_equal(win[:, 8 - w:], hist_o[:, -w:])
    logP_in = ctx.spd_debug_read("LOGP_IN").astype(np.float64)
    sel_o, nl_o, ng_o = orc.step_score()
    nt = orc.tables.n
    assert np.array_equal(ctx.spd_debug_read("CNT")[:, :nt], orc.counts())      # integer lookups: always exact
    assert np.array_equal(ctx.spd_debug_read("TOT")[:, :nt], orc.totals())
    sc, sc_o = ctx.spd_debug_read("SCORE").astype(np.float64), orc.scores()
    assert np.array_equal(np.isfinite(sc), np.isfinite(sc_o))
    fin = np.isfinite(sc_o)
    eps_s = float(np.abs(sc[fin] - sc_o[fin]).max())
    assert eps_s <= np.abs(logP_in - logP_o).max() + (1 - alpha) / tau * 2 * eps_z + 1e-4
    sel = ctx.spd_debug_read("SEL")
    tie_free = top_gap(sc_o, k) > 2 * eps_s
    if tie_free:
        assert sel.tolist() == sel_o.tolist()
    else:
        kth = np.sort(sc_o[fin])[::-1][k - 1]
        assert all(sc_o[q] >= kth - 2 * eps_s for q in sel) and len(set(sel.tolist())) == k
    assert par.tolist() == (sel // k).tolist() and ids.tolist() == cand[sel % k].tolist()
    # stage check: the oracle's scoring stage on the device's own inputs reproduces choice and gamma
    st = so.score_stage(orc.cfg, orc.tables, hist_o[:, -w:], logP_in, cand, cand_lp)
    if top_gap(st["score"], k) > 1e-4:
        assert st["sel"].tolist() == sel.tolist()
        assert np.abs(st["gamma"] - g).max() <= GAMMA_TOL
        assert np.abs(st["logP"] - ctx.spd_debug_read("LOGP")).max() <= 1e-4 * max(1.0, np.abs(st["logP"]).max())
    orc.step_commit(sel, sc_o[sel])
    dg = float(np.abs(orc.gamma() - g).max())
    if stats is not None:
        stats.append({"eps_z": eps_z, "eps_s": eps_s, "dgamma": dg, "tie_free": tie_free})
    _sync_logp(ctx, orc, eps_z)
    return ids, par, g


def free_run(ctx, orc, prefix, n_steps, perturb_logP=None):
    """The whole request on both sides with NO forcing: the oracle never sees the device's cache or its
    log-probabilities.  The only following is the margin rule's: on a step whose oracle margins are below twice the
    measured float error the oracle takes the device's (checked) choice.  Nothing is asserted here: every timestep
    gives a record with the measured logit error `eps_z`, the bound `acc` on gamma's error that the logit errors so
    far imply (accumulated 4 eps / tau), and the verdicts `logits_ok` (within LOGIT_TOL), `ints_ok` (kept tokens,
    n-gram counts and totals exact; choices and parents exact on tie-free steps, else within the margin) and
    `gamma_ok` (within max(GAMMA_TOL, acc)).  The comparison stops where the drafts part.

    `ctx` may be a second oracle instead of the device context (same read-outs through `_OracleAsDevice`), which
    shows how two exact implementations drift apart from a float-sized difference alone."""
    k, tau = ctx.k, orc.cfg.tau
    rec = []
    ids, g = ctx.spd_prefill(prefix)
    if perturb_logP is not None:
        perturb_logP(ctx)
    ids_o, g_o = orc.prefill(prefix)
    z, z_o = ctx.spd_debug_read("LOGITS").astype(np.float64), orc.logits()
    eps_z = float(np.abs(z - z_o).max())
    acc = 4 * eps_z / tau
    same = ids.tolist() == ids_o.tolist()
    dg = float(np.abs(g - g_o).max())
    rec.append({"eps_z": eps_z, "acc": acc, "dgamma": dg, "same": same, "tie_free": top_gap(z_o, k) > 2 * eps_z,
                "logits_ok": eps_z <= LOGIT_TOL, "ints_ok": same, "gamma_ok": dg <= max(GAMMA_TOL, acc)})
    for _ in range(n_steps):
        if not same:
            break
        ids, par, g = ctx.spd_step()
        orc.step_forward()
        z, z_o = ctx.spd_debug_read("LOGITS").astype(np.float64), orc.logits()
        eps_z = float(np.abs(z - z_o).max())
        acc += 4 * eps_z / tau
        cand, cand_o = ctx.spd_debug_read("CAND_TOK"), orc.cand_tok()
        sel_o, _, _ = orc.step_score()
        sel = ctx.spd_debug_read("SEL")
        sc, sc_o = ctx.spd_debug_read("SCORE").astype(np.float64), orc.scores()
        fin = np.isfinite(sc_o)
        nt = orc.tables.n
        r = {"eps_z": eps_z, "acc": acc, "logits_ok": eps_z <= LOGIT_TOL, "gamma_ok": False,
             "near_tie_logits": top_gap(z_o, k) <= 2 * eps_z}
        same = (cand.tolist() == cand_o.tolist() and np.array_equal(np.isfinite(sc), fin)
                and np.array_equal(ctx.spd_debug_read("CNT")[:, :nt], orc.counts())
                and np.array_equal(ctx.spd_debug_read("TOT")[:, :nt], orc.totals()))
        if same:
            eps_s = float(np.abs(sc[fin] - sc_o[fin]).max())
            r["eps_s"] = eps_s
            r["tie_free"] = top_gap(sc_o, k) > 2 * eps_s
            if r["tie_free"]:
                same = sel.tolist() == sel_o.tolist()
            else:
                kth = np.sort(sc_o[fin])[::-1][k - 1]
                same = all(sc_o[q] >= kth - 2 * eps_s for q in sel) and len(set(sel.tolist())) == k
            same = same and par.tolist() == (sel // k).tolist() and ids.tolist() == cand[sel % k].tolist()
        if same:
            orc.step_commit(sel, sc_o[sel])      # the oracle's own scores: only the choice is the device's
            r["dgamma"] = float(np.abs(orc.gamma() - g).max())
            r["gamma_ok"] = r["dgamma"] <= max(GAMMA_TOL, acc)
        r["same"] = r["ints_ok"] = same
        rec.append(r)
    return rec


def show_run(title, rec):
    print(title)
    print("  logit error per step: " + " ".join("%.2g" % r["eps_z"] for r in rec))
    print("  gamma error per step: " + " ".join("%.2g" % r.get("dgamma", float("nan")) for r in rec))
    print("  gamma bound (acc. 4 eps / tau): " + " ".join("%.2g" % r["acc"] for r in rec))
    print("  drafts equal for %d timesteps" % sum(r["same"] for r in rec))


class OracleAsDevice:
    """A second oracle behind the read-outs free_run takes from the device context, free-running too."""

    def __init__(self, orc):
        self.o, self.k = orc, orc.cfg.k

    def spd_prefill(self, prefix):
        return self.o.prefill(prefix)

    def spd_step(self):
        return self.o.step()

    def spd_debug_read(self, what):
        o = self.o
        return {"LOGITS": o.logits, "CAND_TOK": o.cand_tok, "SEL": o.sel, "SCORE": o.scores, "CNT": o.counts,
                "TOT": o.totals}[what]().copy()
