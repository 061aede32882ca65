"""cascade_tree_update: a different draft tree every step in one descriptor (no allocation).  A step through an
updated descriptor must give exactly what a freshly created descriptor of the same tree gives."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def run_pieces(ctx, tree, w, parent, seed):
    """attention + head + similarity + rule + path on seeded inputs of this tree; returns host arrays."""
    T = len(parent)
    rng = np.random.default_rng(seed)
    q, kp, vp, kt, vt, plen = G.attention_inputs(w, rng, T)
    E, hidden, gamma, tok, p, u = G.tail_inputs(w, rng, parent)
    dev = lambda a: torch.from_numpy(a).to(G.DEV)
    z = lambda *s, dt=torch.float32: torch.zeros(s, dtype=dt, device=G.DEV)
    out = torch.zeros((2 * w.B, T, w.n_heads, w.head_dim), dtype=torch.bfloat16, device=G.DEV)
    cb.cascade_tree_attn(ctx, tree, G.to_dev(q, "bf16"), G.to_dev(kp, "bf16"), G.to_dev(vp, "bf16"), w.prefix_len,
                         dev(plen), G.to_dev(kt, "bf16"), G.to_dev(vt, "bf16"), out, 1.0 / np.sqrt(w.head_dim))
    logits, feat, fnorm, lse, cp, cg = z(w.B, T, w.V), z(w.B, T, w.h), z(w.B, T), z(w.B, T), z(w.B, T), z(w.B, T)
    cb.cascade_lm_head_cfg(ctx, tree, G.to_dev(hidden, w.dtype), dev(gamma), w.eps, G.to_dev(E, w.dtype), w.cfg_scale,
                           1.0, dev(tok), logits, feat, fnorm, lse, cp, cg)
    scores = z(w.B, max(tree.num_pairs, 1))
    cb.cascade_similarity(ctx, tree, feat, w.h, fnorm, scores)
    accept = z(w.B, T, dt=torch.uint8)
    qR, tvd = z(w.B, T), z(w.B, T)
    near = z(w.B, dt=torch.int32)
    prm = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, cb.USE_I | cb.USE_C)
    cb.cascade_relaxed_accept(ctx, tree, scores, None, lse, cp, cg, dev(tok), dev(p), dev(u), prm, accept, qR, tvd, near)
    nodes, plen_o, used = z(w.B, tree.depth + 1, dt=torch.int32), z(w.B, dt=torch.int32), z(w.B)
    cb.cascade_select_path(ctx, tree, accept, tvd, cb.SELECT_LONGEST, nodes, plen_o, used)
    torch.cuda.synchronize()
    ctx.check()
    host = dict(q=q, kp=kp, vp=vp, kt=kt, vt=vt, plen=plen, tok=tok, p=p, u=u)
    return dict(attn=out.float().cpu().numpy(), logits=logits.cpu().numpy(), feat=feat.cpu().numpy(),
                scores=scores.cpu().numpy(), accept=accept.cpu().numpy(), nodes=nodes.cpu().numpy(),
                plen=plen_o.cpu().numpy()), host


def test_updated_descriptor_equals_a_fresh_one():
    w = synth.workload("mini", B=2, tree="topk60")
    trees = [synth.workload("mini", tree=t).parent() for t in ("topk60", "topk16", "nary3x3", "chain5", "topk32")]
    ctx = G.make_ctx(w, 64)
    tree = cb.Tree(ctx, trees[0])
    for i, parent in enumerate(trees):
        if i > 0:
            tree.update(parent)
        assert tree.T == len(parent) and tree.depth == int(O.tree_depth(parent).max())
        got, host = run_pieces(ctx, tree, w, parent, 100 + i)
        fresh = cb.Tree(ctx, parent)
        assert fresh.num_pairs == tree.num_pairs and fresh.pairs() == tree.pairs()
        want, _ = run_pieces(ctx, fresh, w, parent, 100 + i)
        fresh.close()
        for key in got:
            assert np.array_equal(got[key], want[key]), (i, key)
        # and against the checker: the mask the updated descriptor carries is this tree's
        ref = O.tree_attention(host["q"], host["kp"], host["vp"], host["plen"], host["kt"], host["vt"], parent,
                               1.0 / np.sqrt(w.head_dim))
        assert np.abs(got["attn"] - ref).max() < 2e-2
        f64 = got["feat"].astype(np.float64)
        rows = [O.relaxed_accept(f64[b], got["logits"][b], host["tok"][b], parent, host["p"][b], host["u"][b],
                                 w.tau_pos, w.tau_seq, w.tvd_budget) for b in range(w.B)]
        G.compare_decisions(parent, rows, got["accept"], got["nodes"], got["plen"], cb.SELECT_LONGEST)
    tree.close()
    ctx.close()


def test_bad_updates_leave_the_descriptor_alone():
    w = synth.workload("mini", B=1, tree="topk16")
    parent = w.parent()
    ctx = G.make_ctx(w, 32)
    tree = cb.Tree(ctx, parent)
    before = (tree.T, tree.depth, tree.num_pairs, tree.pairs())
    L = cb.lib()
    def upd(p):
        arr = (C.c_int32 * len(p))(*p)
        return L.cascade_tree_update(tree.handle, len(p), arr, None)
    assert upd([-1, 0, 0, 2, 1]) == cb.ERR_BAD_TREE                 # sibling groups not contiguous
    assert upd([0, 0, 1]) == cb.ERR_BAD_TREE                        # no root
    assert upd([-1] + [0] * 33) == cb.ERR_UNSUPPORTED_SHAPE         # too many rows / children for this context
    assert L.cascade_tree_update(tree.handle, 0, None, None) == cb.ERR_INVALID_ARG
    assert (L.cascade_tree_rows(tree.handle), L.cascade_tree_depth(tree.handle), L.cascade_tree_num_pairs(tree.handle)) == before[:3]
    assert tree.pairs() == before[3]
    got, _ = run_pieces(ctx, tree, w, parent, 7)                    # still usable, still the old tree
    fresh = cb.Tree(ctx, parent)
    want, _ = run_pieces(ctx, fresh, w, parent, 7)
    for key in got:
        assert np.array_equal(got[key], want[key])
    fresh.close()
    tree.close()
    ctx.close()
