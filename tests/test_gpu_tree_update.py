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


# ---- the descriptor built on the device from a device-resident parent[] -----------------------------------------


def _mask_words(parent):
    anc = O.ancestor_mask(parent)
    words = []
    for j in range(len(parent)):
        w4 = [0, 0, 0, 0]
        for i in np.nonzero(anc[j])[0]:
            w4[int(i) >> 6] |= 1 << (int(i) & 63)
        words.append(w4)
    return words


@pytest.mark.parametrize("tree", ["topk60", "nary2x7", "nary32x1", "nary15x2", "chain5", "chain0"])
def test_device_built_descriptor_is_bit_identical_to_the_host_built_one(tree):
    """255 rows in seven levels, one sibling group of 32, 1920 pairs, a chain, the root alone: every array of the
    descriptor equals what cascade_tree_create makes on the host, and the packed mask equals the checker's."""
    w = synth.workload("mini", B=1, tree=tree)
    parent = w.parent()
    T = len(parent)
    ctx = G.make_ctx(w, 256)
    host_tree = cb.Tree(ctx, parent)
    dev_tree = cb.Tree(ctx, synth.chain_tree(3))                       # some other tree first
    depth = int(O.tree_depth(parent).max())
    cap = max(host_tree.num_pairs, 1)                                  # a bound of 0 would mean "the context's maximum"
    dev_tree.update_device(T, depth, cap, torch.from_numpy(parent).to(G.DEV))
    torch.cuda.synchronize()
    ctx.check()
    assert (dev_tree.T, dev_tree.depth, dev_tree.num_pairs) == (T, depth, cap)
    want, got = host_tree.download(), dev_tree.download()
    names = ("parent", "depth", "child_begin", "child_count", "anc")
    for name, a, b in zip(names, want, got):
        if name == "child_begin":                                      # only meaningful where there are children
            a = [x if c else 0 for x, c in zip(a, want[3])]
            b = [x if c else 0 for x, c in zip(b, got[3])]
        assert a == b, name
    assert got[4] == _mask_words(parent)
    assert got[1] == O.tree_depth(parent).tolist()
    kids = O.children_of(parent)
    assert got[3] == [len(k) for k in kids]
    n = host_tree.num_pairs
    pa, pb = dev_tree.pairs()
    assert (pa[:n], pb[:n]) == host_tree.pairs() and all(x == -1 for x in pa[n:] + pb[n:])
    host_tree.close()
    dev_tree.close()
    ctx.close()


def test_a_different_device_built_tree_every_step_without_a_host_round_trip():
    """A decode-style loop: every step a new parent[] is written on the device, the descriptor is rebuilt there and
    the pieces run behind it on the same stream; results equal those through a host-built descriptor and the
    checker's.  The bounds (depth 7, 200 pairs) stay the same over the loop, as a drafter's limits would."""
    w = synth.workload("mini", B=2, tree="topk60")
    trees = [synth.workload("mini", tree=t).parent() for t in ("topk60", "topk16", "nary3x3", "chain5", "topk32")]
    ctx = G.make_ctx(w, 64)
    tree = cb.Tree(ctx, trees[0])
    DEPTH_CAP, PAIRS_CAP = 7, 200
    parent_dev = torch.zeros(64, dtype=torch.int32, device=G.DEV)
    for i, parent in enumerate(trees):
        parent_dev[: len(parent)].copy_(torch.from_numpy(parent), non_blocking=True)   # stands for the drafter's kernel
        tree.update_device(len(parent), DEPTH_CAP, PAIRS_CAP, parent_dev)
        assert (tree.T, tree.depth, tree.num_pairs) == (len(parent), min(DEPTH_CAP, len(parent) - 1), PAIRS_CAP)
        got, host = run_pieces(ctx, tree, w, parent, 200 + i)
        fresh = cb.Tree(ctx, parent)
        want, _ = run_pieces(ctx, fresh, w, parent, 200 + i)
        n = fresh.num_pairs
        d = fresh.depth
        fresh.close()
        for key in ("attn", "logits", "feat", "accept", "plen"):
            assert np.array_equal(got[key], want[key]), (i, key)
        assert np.array_equal(got["scores"][:, :n], want["scores"])      # rows are PAIRS_CAP long, the first n are used
        assert np.array_equal(got["nodes"][:, : d + 1], want["nodes"]) and np.all(got["nodes"][:, d + 1:] == -1)
        f64 = got["feat"].astype(np.float64)
        rows = [O.relaxed_accept(f64[b], got["logits"][b], host["tok"][b], parent, host["p"][b], host["u"][b],
                                 w.tau_pos, w.tau_seq, w.tvd_budget) for b in range(w.B)]
        st = G.compare_decisions(parent, rows, got["accept"], got["nodes"][:, : d + 1], got["plen"], cb.SELECT_LONGEST)
        assert st["nodes_compared"] > 0
    tree.close()
    ctx.close()


@pytest.mark.parametrize("bad,why", [
    ([-1, 0, 0, 2, 1], "sibling groups not contiguous"),
    ([0, 0, 1], "no root"),
    ([-1, 0, 1, 1, 0], "depth decreases with the index"),
    ([-1, 0, 5, 1], "parent after its child"),
    ([-1] + [0] * 33, "33 children"),
    ([-1, 0, 1, 2, 3], "deeper than the stated bound"),
    ([-1, 0, 0, 0, 0, 0, 0], "more pairs than the stated bound"),
])
def test_device_side_validation(bad, why):
    w = synth.workload("mini", B=1, tree="topk16")
    ctx = G.make_ctx(w, 64)
    tree = cb.Tree(ctx, w.parent())
    T = len(bad)
    depth_cap = 3 if why.startswith("deeper") else 8
    pairs_cap = 10 if why.startswith("more pairs") else 0
    tree.update_device(T, depth_cap, pairs_cap, torch.tensor(bad, dtype=torch.int32, device=G.DEV))
    with pytest.raises(cb.CascadeError) as e:
        ctx.check()
    assert e.value.status == cb.ERR_BAD_TREE, why
    # the neutral descriptor: every row a childless leaf below the root; a step behind it stays in bounds
    parent, depth, cbegin, ccount, anc = tree.download()
    assert parent == [-1] + [0] * (T - 1) and ccount == [0] * T and depth == [0] + [1] * (T - 1)
    assert all(a[0] & 1 for a in anc)
    wt = synth.workload("mini", B=1, tree=f"chain{T - 1}")
    run_pieces(ctx, tree, wt, np.asarray([-1] + [0] * (T - 1), np.int32), 3)     # runs, error word stays clear
    # and a good tree afterwards is taken as usual
    good = w.parent()
    tree.update_device(len(good), 8, 0, torch.from_numpy(good).to(G.DEV))
    torch.cuda.synchronize()
    ctx.check()
    assert tree.download()[0] == good.tolist()
    tree.close()
    ctx.close()
