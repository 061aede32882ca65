"""GPU parity of cascade_filter_logits (top-k / nucleus truncation of the target distribution) against the
checker: kept sets bit-exact for top-k; for top-p exact except tokens whose decision sits within 1e-5 of p."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

P_BAND = 1e-5       # a token whose "mass of the strictly larger logits" is this close to top_p may go either way


def mass_of_larger(row, keep_k):
    """Checker-side: per token, the probability (renormalised over keep_k) of the tokens with a larger logit."""
    p = O.softmax(np.where(keep_k, row, -np.inf))
    order = np.argsort(-row, kind="stable")
    sl, sp = row[order], p[order]
    before = np.cumsum(sp) - sp
    first = np.searchsorted(-sl, -sl, side="left")
    out = np.empty(len(row))
    out[order] = before[first]
    return out


def run_filter(V, logits, top_k, top_p, want_count=True):
    w = synth.workload("mini", B=1, V=V)
    ctx = G.make_ctx(w, 64)
    dev = torch.from_numpy(logits.astype(np.float32)).to(G.DEV)
    cnt = torch.full((logits.shape[0],), -1, dtype=torch.int32, device=G.DEV) if want_count else None
    cb.cascade_filter_logits(ctx, dev, top_k, top_p, cnt)
    torch.cuda.synchronize()
    ctx.check()
    n_launch = ctx.last_launch_count
    ctx.close()
    return dev.cpu().numpy(), None if cnt is None else cnt.cpu().numpy(), n_launch


def check(logits32, got, cnt, top_k, top_p):
    l = logits32.astype(np.float64)
    ref, kept = O.filter_logits(l, top_k, top_p)
    got_kept = ~np.isneginf(got) | np.isneginf(logits32)          # an input -inf stays "dropped" on both sides
    ref_kept = kept & ~np.isneginf(logits32) | np.isneginf(logits32)
    set_aside = 0
    for r in range(l.shape[0]):
        diff = np.nonzero(got_kept[r] != ref_kept[r])[0]
        if len(diff) == 0:
            continue
        assert top_p < 1.0, f"row {r}: top-k kept set differs at {diff[:8]}"
        V = l.shape[1]
        keep_k = np.ones(V, bool)
        if 0 < top_k < V:
            keep_k = l[r] >= np.sort(l[r])[V - top_k]
        larger = mass_of_larger(l[r], keep_k)
        assert np.all(np.abs(larger[diff] - top_p) < P_BAND), f"row {r}: nucleus differs outside the band"
        set_aside += len(diff)
    assert np.array_equal(got[got_kept & ~np.isneginf(logits32)], logits32[got_kept & ~np.isneginf(logits32)])   # kept logits untouched
    if cnt is not None:
        assert np.array_equal(cnt, (~np.isneginf(got)).sum(-1))
    return set_aside


def cluster_logits(rng, n, V, scale=8.0):
    """Rows shaped like the workloads' target logits: a few hundred near-identical codes share the mass."""
    centres = rng.normal(0, 1, (256,))
    base = centres[np.arange(V) % 256][None, :] * scale / 3 + rng.normal(0, 0.3, (n, V))
    return base.astype(np.float32)


@pytest.mark.parametrize("V,n", [(16384, 61), (65536, 9), (1024, 15), (2048 + 40, 5)])
def test_top_k_exact(V, n):
    rng = np.random.default_rng(V)
    logits = cluster_logits(rng, n, V)
    for k in (1, 2, 200, 2000, V - 1):
        if k >= V:
            continue
        got, cnt, n_launch = run_filter(V, logits, k, 1.0)
        assert check(logits, got, cnt, k, 1.0) == 0
        assert (cnt >= k).all() and n_launch == 1


@pytest.mark.parametrize("V,n", [(16384, 33), (4096, 8)])
def test_top_p_and_both(V, n):
    rng = np.random.default_rng(V + 1)
    logits = cluster_logits(rng, n, V)
    total_aside = 0
    for k, p in ((0, 0.9), (0, 0.5), (0, 0.01), (2000, 0.95), (50, 0.3)):
        got, cnt, _ = run_filter(V, logits, k, p)
        total_aside += check(logits, got, cnt, k, p)
    assert total_aside <= 4


def test_ties_and_degenerate_rows():
    V = 4096
    rng = np.random.default_rng(5)
    logits = (np.round(rng.normal(0, 2, (6, V)) * 2) / 2).astype(np.float32)      # many equal logits
    logits[1, :] = 0.25                                                           # a flat row: everything ties
    logits[2, ::3] = -np.inf                                                      # already truncated once
    for k, p in ((7, 1.0), (0, 0.4), (100, 0.8)):
        got, cnt, _ = run_filter(V, logits, k, p)
        check(logits, got, cnt, k, p)
        assert cnt[1] == V                                                        # ties stay together
    # applying the same truncation twice changes nothing
    once, c1, _ = run_filter(V, logits, 100, 1.0)
    twice, c2, _ = run_filter(V, once, 100, 1.0)
    assert np.array_equal(once, twice) and np.array_equal(c1, c2)


def test_long_rows_at_an_unaligned_address():
    """Rows longer than the register path holds, starting 4 bytes off a 16-byte boundary: the scalar loads."""
    V, n = 16384 + 1000, 3
    rng = np.random.default_rng(77)
    logits = cluster_logits(rng, n, V)
    w = synth.workload("mini", B=1, V=V)
    ctx = G.make_ctx(w, 64)
    buf = torch.zeros(n * V + 4, device=G.DEV)
    view = buf[1:1 + n * V].view(n, V)
    view.copy_(torch.from_numpy(logits))
    assert view.data_ptr() % 16 == 4
    cnt = torch.zeros(n, dtype=torch.int32, device=G.DEV)
    cb.cascade_filter_logits(ctx, view, 300, 0.9, cnt)
    torch.cuda.synchronize()
    ctx.check()
    check(logits, view.cpu().numpy(), cnt.cpu().numpy(), 300, 0.9)
    ctx.close()


def test_off_settings_and_errors():
    V = 1024
    logits = cluster_logits(np.random.default_rng(9), 4, V)
    for k in (0, V, V + 5):
        got, cnt, _ = run_filter(V, logits, k, 1.0)
        assert np.array_equal(got, logits) and (cnt == V).all()
    got, _, n_launch = run_filter(V, logits, 0, 1.0, want_count=False)
    assert np.array_equal(got, logits) and n_launch == 0                           # nothing to do: no launch
    w = synth.workload("mini", B=1, V=V)
    ctx = G.make_ctx(w, 16)
    d = torch.zeros((2, V), device=G.DEV)
    L = cb.lib()
    bad = [(None, 2, 5, 0.9), (d.data_ptr(), 0, 5, 0.9), (d.data_ptr(), 2, -1, 0.9), (d.data_ptr(), 2, 5, 0.0),
           (d.data_ptr(), 2, 5, 1.5), (d.data_ptr(), 2, 5, float("nan"))]
    for ptr, n, k, p in bad:
        assert L.cascade_filter_logits(ctx.handle, ptr, n, k, C.c_float(p), None, None) == cb.ERR_INVALID_ARG
    ctx.close()


def test_truncated_target_feeds_acceptance():
    """Head -> truncation -> acceptance on the device against the checker's rule on the checker-truncated
    logits of the same device logits (decisions bit-exact outside the near band)."""
    w = synth.workload("mini", B=2)
    parent = w.parent()
    T = len(parent)
    ctx = G.make_ctx(w, T)
    tree = cb.Tree(ctx, parent)
    rng = np.random.default_rng(21)
    E, hidden, gamma, tok, p, u = G.tail_inputs(w, rng, parent)
    dev = lambda a: torch.from_numpy(a).to(G.DEV)
    z = lambda *s, dt=torch.float32: torch.zeros(s, dtype=dt, device=G.DEV)
    logits, feat, fnorm, lse, cp, cg = z(w.B, T, w.V), z(w.B, T, w.h), z(w.B, T), z(w.B, T), z(w.B, T), z(w.B, T)
    cb.cascade_lm_head_cfg(ctx, tree, G.to_dev(hidden, w.dtype), dev(gamma), w.eps, G.to_dev(E, w.dtype), w.cfg_scale,
                           1.0, dev(tok), logits, feat, fnorm, lse, cp, cg)
    raw = logits.cpu().numpy().copy()
    top_k = max(8, w.V // 16)
    cb.cascade_filter_logits(ctx, logits, top_k, 1.0)
    scores = z(w.B, max(tree.num_pairs, 1))
    cb.cascade_similarity(ctx, tree, feat, w.h, fnorm, scores)
    accept = z(w.B, T, dt=torch.uint8)
    qR, tvd = z(w.B, T), z(w.B, T)
    near = z(w.B, dt=torch.int32)
    prm = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, cb.USE_I | cb.USE_C)
    cb.cascade_relaxed_accept(ctx, tree, scores, logits, None, None, None, dev(tok), dev(p), dev(u), prm, accept, qR,
                              tvd, near)
    nodes, plen, used = z(w.B, tree.depth + 1, dt=torch.int32), z(w.B, dt=torch.int32), z(w.B)
    cb.cascade_select_path(ctx, tree, accept, tvd, cb.SELECT_LONGEST, nodes, plen, used)
    torch.cuda.synchronize()
    ctx.check()
    filt, _ = O.filter_logits(raw.astype(np.float64), top_k, 1.0)
    assert np.array_equal(np.isneginf(filt), np.isneginf(logits.cpu().numpy()))
    f64 = feat.cpu().numpy().astype(np.float64)
    rows = [O.relaxed_accept(f64[b], filt[b], tok[b], parent, p[b], u[b], w.tau_pos, w.tau_seq, w.tvd_budget)
            for b in range(w.B)]
    stats = G.compare_decisions(parent, rows, accept.cpu().numpy(), nodes.cpu().numpy(), plen.cpu().numpy(),
                                cb.SELECT_LONGEST)
    dropped = sum(int(np.isneginf(filt[b][parent[j]][tok[b][j]])) for b in range(w.B) for j in range(1, T))
    print(f"truncation to top-{top_k}: {dropped} draft tokens outside the kept set, {stats}")
    tree.close()
    ctx.close()


@pytest.mark.parametrize("mode", [cb.SELECT_LONGEST, cb.SELECT_FIRST_ACCEPT])
def test_fused_step_with_truncation(mode):
    """cascade_verify_step with top_k / top_p set: the stored logits come back truncated as the checker
    truncates the untruncated ones, and accept bits and paths are the checker's rule on those."""
    from paper_2605_07230_b200.workload import PiecesWorkload
    w = synth.workload("mini", B=3, tree="topk60")
    wl = PiecesWorkload(w, n_sets=1, keep_logits=True, select_mode=mode)
    s = wl.run(0)
    torch.cuda.synchronize()
    wl.ctx.check()
    raw = s.out["logits"].cpu().numpy().copy()
    base_launches = wl.ctx.last_launch_count
    for top_k, top_p in ((w.V // 16, 0.0), (0, 0.9), (w.V // 8, 0.8)):
        s.step.top_k, s.step.top_p = top_k, top_p
        wl.run(0)
        torch.cuda.synchronize()
        wl.ctx.check()
        assert wl.ctx.last_launch_count == base_launches + 2          # truncation + row statistics
        got = s.out["logits"].cpu().numpy()
        filt, _ = O.filter_logits(raw.astype(np.float64), top_k, top_p if top_p > 0 else 1.0)
        differ = np.isneginf(filt) != np.isneginf(got)
        assert differ.sum() <= (2 if top_p > 0 else 0)                 # nucleus: tokens within the band of p
        if differ.any():
            continue
        feat = s.out["feat"].cpu().numpy().astype(np.float64)
        h = s.host
        rows = [O.relaxed_accept(feat[b], filt[b], h["tok"][b], wl.parent, h["draft_p"][b], h["uniforms"][b],
                                 w.tau_pos, w.tau_seq, w.tvd_budget) for b in range(w.B)]
        G.compare_decisions(wl.parent, rows, s.out["accept"].cpu().numpy(), s.out["path_nodes"].cpu().numpy(),
                            s.out["path_len"].cpu().numpy(), mode)
    # the truncation needs stored logits, and its parameters are validated
    import ctypes as C2
    s.step.top_k, s.step.top_p = 5, 0.0
    saved = s.step.logits
    s.step.logits = None
    assert cb.lib().cascade_verify_step(wl.ctx.handle, wl.tree.handle, C2.byref(s.step), None) == cb.ERR_INVALID_ARG
    s.step.logits = saved
    s.step.top_k, s.step.top_p = -1, 0.0
    assert cb.lib().cascade_verify_step(wl.ctx.handle, wl.tree.handle, C2.byref(s.step), None) == cb.ERR_INVALID_ARG
    s.step.top_k, s.step.top_p = 0, 1.5
    assert cb.lib().cascade_verify_step(wl.ctx.handle, wl.tree.handle, C2.byref(s.step), None) == cb.ERR_INVALID_ARG
    wl.close()
