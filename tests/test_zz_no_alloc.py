"""The allocation-free entry point against the regular ones.

cascade_accept_static serves callers that are not allowed to allocate device memory (no context, no
tree object: its scratch is a static device array inside the library).  It must give exactly what
cascade_similarity + cascade_relaxed_accept + cascade_select_path give on the same inputs, and it
must do so on every call although all calls share one scratch array that keeps its old contents.
Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _inputs(w, parent, seed):
    rng = np.random.default_rng(seed)
    T = len(parent)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(G.DEV)
    tok, p = synth.cluster_drafter(rng, parent, w.B, w.V, w.n_clusters)
    E = synth.clustered_codebook(rng, w.V, w.h, w.n_clusters, w.sigma)
    feat = (E[tok] + 0.003 * rng.standard_normal((w.B, T, w.h), dtype=np.float32)).astype(np.float32)
    row_lse = rng.normal(3.0, 0.2, (w.B, T)).astype(np.float32)
    cand_p = (row_lse[:, [max(int(x), 0) for x in parent]] + np.log(p) + rng.normal(0, 0.7, (w.B, T))).astype(np.float32)
    cand_g = (cand_p - 1.0).astype(np.float32)
    return dict(feat=dev(feat), row_lse=dev(row_lse), cand_p=dev(cand_p), cand_g=dev(cand_g), tok=dev(tok),
                draft_p=dev(p), u=dev(synth.uniforms(rng, w.B, T)))


def _regular(w, parent, x, params, mode):
    T = len(parent)
    ctx = G.make_ctx(w, T)
    tree = cb.Tree(ctx, parent)
    scores = torch.zeros((w.B, max(tree.num_pairs, 1)), device=G.DEV)
    out = _outputs(w.B, T, tree.depth)
    cb.cascade_similarity(ctx, tree, x["feat"], w.h, None, scores)
    cb.cascade_relaxed_accept(ctx, tree, scores, None, x["row_lse"], x["cand_p"], x["cand_g"], x["tok"], x["draft_p"],
                              x["u"], params, out["accept"], out["q_relaxed"], out["tvd_out"], out["near"])
    cb.cascade_select_path(ctx, tree, out["accept"], out["tvd_out"], mode, out["nodes"], out["plen"], out["tvd_used"])
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy().copy() for k, v in out.items()}
    depth = tree.depth
    tree.close()
    ctx.close()
    return res, depth


def _outputs(B, T, depth):
    return dict(accept=torch.full((B, T), 7, dtype=torch.uint8, device=G.DEV),
                q_relaxed=torch.full((B, T), float("nan"), device=G.DEV),
                tvd_out=torch.full((B, T), float("nan"), device=G.DEV),
                near=torch.full((B,), -1, dtype=torch.int32, device=G.DEV),
                nodes=torch.full((B, depth + 1), -7, dtype=torch.int32, device=G.DEV),
                plen=torch.full((B,), -1, dtype=torch.int32, device=G.DEV),
                tvd_used=torch.full((B,), float("nan"), device=G.DEV))


@pytest.mark.parametrize("mode", [cb.SELECT_LONGEST, cb.SELECT_FIRST_ACCEPT])
def test_static_scratch_entry_matches_regular_entries_twice_in_a_row(mode):
    params = cb.Params(0.85, 0.5, 0.5, cb.USE_I | cb.USE_C)
    # two different trees and batch sizes back to back: the second call finds the first call's
    # descriptor, scores and counters in the shared array
    cases = [(synth.workload("mini", B=3, tree="topk60"), 5), (synth.workload("mini", B=2, tree="topk16"), 6)]
    for w, seed in cases:
        parent = w.parent()
        T = len(parent)
        x = _inputs(w, parent, seed)
        want, depth = _regular(w, parent, x, params, mode)
        got = _outputs(w.B, T, depth)
        cb.cascade_accept_static(w.B, parent, x["feat"], w.h, None, x["row_lse"], x["cand_p"], x["cand_g"], x["tok"],
                                 x["draft_p"], x["u"], params, mode, got["accept"], got["q_relaxed"], got["tvd_out"],
                                 got["near"], got["nodes"], got["plen"], got["tvd_used"])
        torch.cuda.synchronize()
        assert want["accept"].sum() > w.B            # something beyond the roots was accepted
        for k in ("accept", "nodes", "plen", "near"):   # integer results: bit-exact
            assert np.array_equal(got[k].cpu().numpy(), want[k]), k
        for k in ("q_relaxed", "tvd_out", "tvd_used"):  # same kernel, same order of operations
            assert np.allclose(got[k].cpu().numpy(), want[k], rtol=0, atol=1e-6), k


def test_static_scratch_entry_rejects_sizes_beyond_its_array():
    import ctypes as C
    L = cb.lib()
    params = cb.Params(0.85, 0.5, 0.5, cb.USE_I | cb.USE_C)
    parent = (C.c_int32 * 2)(-1, 0)
    one = torch.zeros(16, device=G.DEV)
    p = one.data_ptr()
    too_many_prompts = L.cascade_accept_static(33, 2, parent, p, 4, None, p, p, p, p, p, p, C.byref(params), 0, p, None,
                                               None, None, p, p, None, None)
    assert too_many_prompts == cb.ERR_UNSUPPORTED_SHAPE
    big = (C.c_int32 * 300)(*([-1] + list(range(299))))
    too_many_rows = L.cascade_accept_static(1, 300, big, p, 4, None, p, p, p, p, p, p, C.byref(params), 0, p, None,
                                            None, None, p, p, None, None)
    assert too_many_rows == cb.ERR_UNSUPPORTED_SHAPE


def test_static_scratch_entry_against_the_checker():
    """The same entry against the fp64 checker directly: logits are made on the host, the row statistics and
    candidate logits the entry takes are derived from them with the checker's own helpers, and the decisions must
    equal the checker's rule on those logits and features (near-threshold nodes set aside as everywhere)."""
    from oracle import cascade_oracle as O
    w = synth.workload("mini", B=3, tree="topk32", V=512)
    parent = w.parent()
    T = len(parent)
    rng = np.random.default_rng(77)
    tok, p = synth.cluster_drafter(rng, parent, w.B, w.V, w.n_clusters)
    E = synth.clustered_codebook(rng, w.V, w.h, w.n_clusters, w.sigma)
    feat = (E[tok] + 0.003 * rng.standard_normal((w.B, T, w.h), dtype=np.float32)).astype(np.float32)
    # target logits that favour each row's own cluster, so that drafted tokens carry real mass
    logits = (rng.normal(0, 1, (w.B, T, w.V)) + 4.0 * ((np.arange(w.V)[None, None, :] % w.n_clusters) ==
                                                        (tok[:, :, None] % w.n_clusters))).astype(np.float32)
    u = synth.uniforms(rng, w.B, T)
    lse = O.log_sum_exp(logits).astype(np.float32)
    cp, cg = (x.astype(np.float32) for x in O.candidate_logits(logits, tok, parent))
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(G.DEV)
    params = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, cb.USE_I | cb.USE_C)
    depth = int(O.tree_depth(parent).max())
    got = _outputs(w.B, T, depth)
    cb.cascade_accept_static(w.B, parent, dev(feat), w.h, None, dev(lse), dev(cp), dev(cg), dev(tok), dev(p), dev(u), params,
                             cb.SELECT_LONGEST, got["accept"], got["q_relaxed"], got["tvd_out"], got["near"], got["nodes"],
                             got["plen"], got["tvd_used"])
    torch.cuda.synchronize()
    rows = [O.relaxed_accept(feat[b].astype(np.float64), logits[b], tok[b], parent, p[b], u[b], w.tau_pos, w.tau_seq,
                             w.tvd_budget) for b in range(w.B)]
    st = G.compare_decisions(parent, rows, got["accept"].cpu().numpy(), got["nodes"].cpu().numpy(),
                             got["plen"].cpu().numpy(), cb.SELECT_LONGEST)
    assert st["nodes_compared"] > 0.8 * st["nodes"]
    qR = got["q_relaxed"].cpu().numpy()
    for b in range(w.B):
        if not rows[b]["near"].any():
            assert np.abs(qR[b] - rows[b]["q_relaxed"]).max() < 1e-4
    assert sum(int(r["accept"].sum()) for r in rows) > w.B     # drafts were accepted
