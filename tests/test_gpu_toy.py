"""GPU parity, fp32 toy workload (hidden 256, 4 heads x 64, vocabulary 1024, 15-row binary tree):
every exported piece against the CPU checker, element by element."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def toy():
    w = synth.workload("toy")
    parent = w.parent()
    ctx = G.make_ctx(w, len(parent))
    tree = cb.Tree(ctx, parent)
    yield w, parent, ctx, tree
    tree.close()
    ctx.close()


def test_tree_descriptor(toy):
    w, parent, ctx, tree = toy
    assert tree.T == 15 and tree.depth == 3
    a, b = tree.pairs()
    cs, cc = O.similarity_scores(np.eye(15), parent)
    assert set(zip(a[:14], b[:14])) == set(cc)                       # edges first, edge of node j at j-1
    assert [(a[j - 1], b[j - 1]) for j in range(1, 15)] == [(parent[j], j) for j in range(1, 15)]
    assert set(zip(a[14:], b[14:])) == {k for k in cs if k[0] < k[1]}


def test_tree_attention_fp32(toy):
    w, parent, ctx, tree = toy
    rng = np.random.default_rng(w.seed)
    T = len(parent)
    q, kp, vp, kt, vt, plen = G.attention_inputs(w, rng, T, prefix_len=[w.prefix_len, w.prefix_len - 5])
    out = torch.empty((2, T, w.n_heads, w.head_dim), device=G.DEV)
    scale = 1 / np.sqrt(w.head_dim)
    cb.cascade_tree_attn(ctx, tree, G.to_dev(q, "f32"), G.to_dev(kp, "f32"), G.to_dev(vp, "f32"), w.prefix_len,
                         torch.from_numpy(plen).to(G.DEV), G.to_dev(kt, "f32"), G.to_dev(vt, "f32"), out, scale)
    ref = O.tree_attention(q, kp, vp, plen, kt, vt, parent, scale)
    assert np.abs(out.cpu().numpy() - ref).max() < 1e-5


def test_head_accept_path_fp32(toy):
    w, parent, ctx, tree = toy
    T = len(parent)
    fired = 0
    for seed in range(6):
        rng = np.random.default_rng(1000 + seed)
        E, hidden, gamma, tok, p, u = G.tail_inputs(w, rng, parent)
        dev = lambda a: torch.from_numpy(a).to(G.DEV)
        logits = torch.empty((w.B, T, w.V), device=G.DEV)
        feat = torch.empty((w.B, T, w.h), device=G.DEV)
        fnorm = torch.empty((w.B, T), device=G.DEV)
        lse = torch.empty((w.B, T), device=G.DEV)
        cp = torch.empty((w.B, T), device=G.DEV)
        cg = torch.empty((w.B, T), device=G.DEV)
        d_tok = dev(tok)
        cb.cascade_lm_head_cfg(ctx, tree, dev(hidden), dev(gamma), w.eps, dev(E), w.cfg_scale, 1.0, d_tok, logits,
                               feat, fnorm, lse, cp, cg)
        ref = O.lm_head_cfg(hidden, gamma, w.eps, E, w.cfg_scale, 1.0)
        assert np.abs(logits.cpu().numpy() - ref["logits"]).max() < 2e-4
        assert np.abs(feat.cpu().numpy() - ref["feat"]).max() < 1e-5
        assert np.abs(fnorm.cpu().numpy() - ref["feat_norm"]).max() < 1e-4
        assert np.abs(lse.cpu().numpy() - ref["lse"]).max() < 1e-4
        lp, lg = O.candidate_logits(ref["logits"], tok, parent)
        assert np.abs(cp.cpu().numpy() - lp).max() < 2e-4 and np.abs(cg.cpu().numpy() - lg).max() < 2e-4

        scores = torch.empty((w.B, tree.num_pairs), device=G.DEV)
        cb.cascade_similarity(ctx, tree, feat, w.h, fnorm, scores)
        pa, pb = tree.pairs()
        feat_h = feat.cpu().numpy().astype(np.float64)
        want = np.array([[O.cosine(feat_h[b, i], feat_h[b, j]) for i, j in zip(pa, pb)] for b in range(w.B)])
        assert np.abs(scores.cpu().numpy() - want).max() < 1e-5
        scores2 = torch.empty_like(scores)
        cb.cascade_similarity(ctx, tree, feat, w.h, None, scores2)       # norms computed in the kernel
        assert np.abs(scores2.cpu().numpy() - want).max() < 1e-5

        for flags in (cb.USE_I | cb.USE_C, cb.USE_I, cb.USE_C, 0, cb.USE_I | cb.USE_C | cb.CONV_DIST_SELF):
            prm = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, flags)
            accept = torch.zeros((w.B, T), dtype=torch.uint8, device=G.DEV)
            qR = torch.empty((w.B, T), device=G.DEV)
            tvd = torch.empty((w.B, T), device=G.DEV)
            near = torch.zeros(w.B, dtype=torch.int32, device=G.DEV)
            # once from the head's fused statistics, once from the logits themselves
            for use_logits in (False, True):
                cb.cascade_relaxed_accept(ctx, tree, scores, logits if use_logits else None,
                                          None if use_logits else lse, None if use_logits else cp,
                                          None if use_logits else cg, d_tok, dev(p), dev(u), prm, accept, qR, tvd,
                                          near)
                logits_h = logits.cpu().numpy()
                rows = [O.relaxed_accept(feat_h[b], logits_h[b], tok[b], parent, p[b], u[b], w.tau_pos, w.tau_seq,
                                         w.tvd_budget, flags) for b in range(w.B)]
                for mode in (cb.SELECT_LONGEST, cb.SELECT_FIRST_ACCEPT):
                    nodes = torch.zeros((w.B, tree.depth + 1), dtype=torch.int32, device=G.DEV)
                    plen = torch.zeros(w.B, dtype=torch.int32, device=G.DEV)
                    used = torch.zeros(w.B, device=G.DEV)
                    cb.cascade_select_path(ctx, tree, accept, tvd, mode, nodes, plen, used)
                    st = G.compare_decisions(parent, rows, accept.cpu().numpy(), nodes.cpu().numpy(),
                                             plen.cpu().numpy(), mode)
                    for b, r in enumerate(rows):
                        if not np.any(r["near"]):
                            assert np.abs(qR.cpu().numpy()[b] - r["q_relaxed"]).max() < 1e-5
                            assert np.abs(tvd.cpu().numpy()[b] - r["tvd_out"]).max() < 1e-5
                            _, _, tu = O.select_path(r["accept"], parent, r["tvd_out"], mode)
                            assert abs(float(used[b]) - tu) < 1e-5
                            assert int(near[b]) == 0
                fired += sum(int((r["q_relaxed"] > r["q_plain"]).sum()) for r in rows)
    assert fired > 20        # the relaxation really took part


def test_bad_arguments_are_refused_on_the_host(toy):
    w, parent, ctx, tree = toy
    import ctypes as C
    L = cb.lib()
    h = C.c_void_p()
    assert L.cascade_tree_create(ctx.handle, 3, (C.c_int32 * 3)(-1, 0, 2), C.byref(h)) == cb.ERR_BAD_TREE
    assert L.cascade_tree_create(ctx.handle, 3, (C.c_int32 * 3)(0, 0, 1), C.byref(h)) == cb.ERR_BAD_TREE
    assert L.cascade_tree_create(ctx.handle, 4, (C.c_int32 * 4)(-1, 0, 1, 0), C.byref(h)) == cb.ERR_BAD_TREE
    assert L.cascade_tree_create(ctx.handle, 99, (C.c_int32 * 99)(*([-1] + list(range(98)))),
                                 C.byref(h)) == cb.ERR_UNSUPPORTED_SHAPE
    assert L.cascade_tree_attn(ctx.handle, tree.handle, None, None, None, 0, None, None, None, None, 1.0,
                               None) == cb.ERR_INVALID_ARG
    bad = cb.Shape(cb.F32, 1, 15, 64, 250, 4, 4, 64, 1024, 0)
    assert L.cascade_create(C.byref(h), C.byref(bad)) == cb.ERR_UNSUPPORTED_SHAPE
    bad = cb.Shape(cb.F32, 1, 999, 64, 256, 4, 4, 64, 1024, 0)
    assert L.cascade_create(C.byref(h), C.byref(bad)) == cb.ERR_UNSUPPORTED_SHAPE
    ctx.check()
