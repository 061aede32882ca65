"""GPU parity of piece (b) in bf16: final norm + guidance mix + tcgen05 LM head + softmax statistics."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

LOGIT_TOL = 3e-2        # max-abs bound on logits against the fp64 checker


def run_head(w, parent, seed, want_logits=True, temperature=1.0):
    T = len(parent)
    ctx = G.make_ctx(w, T)
    tree = cb.Tree(ctx, parent)
    rng = np.random.default_rng(seed)
    E, hidden, gamma, tok, p, u = G.tail_inputs(w, rng, parent)
    dev = lambda a: torch.from_numpy(a).to(G.DEV)
    f = lambda *s: torch.full(s, float("nan"), device=G.DEV)
    logits = f(w.B, T, w.V) if want_logits else None
    feat, fnorm, lse, cp, cg = f(w.B, T, w.h), f(w.B, T), f(w.B, T), f(w.B, T), f(w.B, T)
    cb.cascade_lm_head_cfg(ctx, tree, G.to_dev(hidden, w.dtype), dev(gamma), w.eps, G.to_dev(E, w.dtype),
                           w.cfg_scale, temperature, dev(tok), logits, feat, fnorm, lse, cp, cg)
    torch.cuda.synchronize()
    ctx.check()
    ref = O.lm_head_cfg(hidden, gamma, w.eps, E, w.cfg_scale, temperature)
    out = dict(logits=None if logits is None else logits.cpu().numpy(), feat=feat.cpu().numpy(),
               fnorm=fnorm.cpu().numpy(), lse=lse.cpu().numpy(), cp=cp.cpu().numpy(), cg=cg.cpu().numpy())
    tree.close()
    ctx.close()
    return out, ref, tok


@pytest.mark.parametrize("name,over", [
    ("mini", {}),                                                  # M = 66 rows -> NB = 80
    ("mini", dict(B=1, tree="topk16", V=2048 + 8 * 5)),            # ragged last vocabulary tile
    ("mini", dict(B=1, tree="chain1", V=128)),                     # two rows, a single tile
    ("mini", dict(B=8, tree="topk60", h=256, V=4096)),             # M = 488 rows -> several row chunks
])
def test_head_against_checker(name, over):
    w = synth.workload(name, **over)
    parent = w.parent()
    got, ref, tok = run_head(w, parent, 11)
    err = np.abs(got["logits"] - ref["logits"]).max()
    assert err < LOGIT_TOL, err
    assert err < 2e-3                      # what the split operand actually delivers
    assert np.abs(got["feat"] - ref["feat"]).max() < 1e-4
    assert np.abs(got["fnorm"] / ref["feat_norm"] - 1).max() < 1e-5
    assert np.abs(got["lse"] - ref["lse"]).max() < 2e-3
    lp, lg = O.candidate_logits(ref["logits"], tok, parent)
    assert np.abs(got["cp"] - lp).max() < 2e-3 and np.abs(got["cg"] - lg).max() < 2e-3


def test_head_without_logits_store_and_with_temperature():
    w = synth.workload("mini")
    parent = w.parent()
    got, ref, tok = run_head(w, parent, 12, want_logits=False, temperature=1.7)
    assert got["logits"] is None
    assert np.abs(got["lse"] - ref["lse"]).max() < 2e-3
    lp, _ = O.candidate_logits(ref["logits"], tok, parent)
    assert np.abs(got["cp"] - lp).max() < 2e-3


def test_head_is_deterministic_run_to_run():
    w = synth.workload("mini")
    parent = w.parent()
    a, _, _ = run_head(w, parent, 13)
    b, _, _ = run_head(w, parent, 13)
    assert np.array_equal(a["logits"], b["logits"]) and np.array_equal(a["lse"], b["lse"])


def test_logit_space_similarity_and_acceptance():
    """Appendix B's variant: the cosines of Eq. 1 / Eq. 2 taken between rows of logits instead of hidden
    states -- cascade_similarity with feat = logits, feat_dim = V -- and the rule run on those scores."""
    w = synth.workload("mini", B=2)
    parent = w.parent()
    T = len(parent)
    ctx = G.make_ctx(w, T)
    tree = cb.Tree(ctx, parent)
    rng = np.random.default_rng(31)
    E, hidden, gamma, tok, p, u = G.tail_inputs(w, rng, parent)
    dev = lambda a: torch.from_numpy(a).to(G.DEV)
    z = lambda *s, dt=torch.float32: torch.zeros(s, dtype=dt, device=G.DEV)
    logits, feat, fnorm, lse, cp, cg = z(w.B, T, w.V), z(w.B, T, w.h), z(w.B, T), z(w.B, T), z(w.B, T), z(w.B, T)
    cb.cascade_lm_head_cfg(ctx, tree, G.to_dev(hidden, w.dtype), dev(gamma), w.eps, G.to_dev(E, w.dtype), w.cfg_scale,
                           1.0, dev(tok), logits, feat, fnorm, lse, cp, cg)
    scores = z(w.B, max(tree.num_pairs, 1))
    cb.cascade_similarity(ctx, tree, logits, w.V, None, scores)
    accept = z(w.B, T, dt=torch.uint8)
    qR, tvd = z(w.B, T), z(w.B, T)
    near = z(w.B, dt=torch.int32)
    prm = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, cb.USE_I | cb.USE_C)
    cb.cascade_relaxed_accept(ctx, tree, scores, None, lse, cp, cg, dev(tok), dev(p), dev(u), prm, accept, qR, tvd, near)
    nodes, plen, used = z(w.B, tree.depth + 1, dt=torch.int32), z(w.B, dt=torch.int32), z(w.B)
    cb.cascade_select_path(ctx, tree, accept, tvd, cb.SELECT_LONGEST, nodes, plen, used)
    torch.cuda.synchronize()
    ctx.check()
    lg = logits.cpu().numpy().astype(np.float64)
    pa, pb = tree.pairs()
    got = scores.cpu().numpy()
    for b in range(w.B):
        ref = np.array([O.cosine(lg[b][a], lg[b][c]) for a, c in zip(pa, pb)])
        assert np.abs(got[b] - ref).max() < 2e-5
    rows = [O.relaxed_accept(lg[b], lg[b], tok[b], parent, p[b], u[b], w.tau_pos, w.tau_seq, w.tvd_budget)
            for b in range(w.B)]
    G.compare_decisions(parent, rows, accept.cpu().numpy(), nodes.cpu().numpy(), plen.cpu().numpy(), cb.SELECT_LONGEST)
    tree.close()
    ctx.close()
