"""GPU parity of a short speculative decode loop (verification step through several layers, bonus token,
cache append) against the checker.  The checker follows the device's decisions from step to step
(its own caches, its own arithmetic), so that a near-tie in one step cannot derail the comparison of
the next."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from paper_2605_07230_b200.workload import DecodeLoop
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,over,n_layers,steps,graph_after", [
    ("mini", dict(B=2, tree="topk32", prefix_len=40), 2, 3, None),
    ("mini", dict(B=1, tree="topk60", prefix_len=130), 3, 2, None),
    ("mini", dict(B=2, tree="topk32", prefix_len=40), 2, 4, 1),     # steps after the first replay a recorded CUDA graph
    # the decode loop's own widths (hidden 4096, 32 heads x 128, SwiGLU 11008, vocabulary 16384, 64-row prompt cache,
    # 61-row trees): two of its layers, two steps, the second replayed from a recorded graph
    pytest.param("janus", dict(prefix_len=64), 2, 2, 1, id="full-width-2-layers"),
])
def test_decode_loop(name, over, n_layers, steps, graph_after):
    w = synth.workload(name, **over)
    loop = DecodeLoop(w, n_layers, max_steps=steps, seed=11)
    B, parent = w.B, loop.parent
    h = loop.host
    k_cache = [np.array(x, np.float64) for x in h["k_prefix"]]
    v_cache = [np.array(x, np.float64) for x in h["v_prefix"]]
    plen = h["prefix_len"].astype(np.int64).copy()
    total_accepted = 0
    for it in range(steps):
        if graph_after is not None and it == graph_after:
            loop.capture()
        drafted = loop.draft()
        tok, p, u, ub = drafted
        ref = O.verify_step(h["embed"], h["layers"], h["gamma_final"], h["w_head"], tok, parent, k_cache, v_cache, plen,
                            p, u, w.n_heads, w.head_dim, w.eps, w.rope_base, w.cfg_scale, 1.0, w.tau_pos, w.tau_seq,
                            w.tvd_budget)
        res = loop.step(drafted)
        torch.cuda.synchronize()
        o = loop.set.out
        logits = o["logits"].cpu().numpy()
        # 3e-2 per step through one layer.  At full width the second layer rounds its queries, keys and values to
        # bf16 from inputs that already differ from the checker's in the last bits, so isolated elements land on the
        # neighbouring bf16 value (a 0.4 % step) in one computation and not in the other: the two part by up to one
        # layer's tolerance per layer.  (tests/test_gpu_fullsize.py holds every layer to 3e-2 on identical inputs.)
        tol = 3e-2 * (n_layers if name != "mini" else 1)
        assert np.abs(logits - ref["head"]["logits"]).max() < tol
        feat = o["feat"].cpu().numpy().astype(np.float64)
        rows = [O.relaxed_accept(feat[b], logits[b], tok[b], parent, p[b], u[b], w.tau_pos, w.tau_seq, w.tvd_budget)
                for b in range(B)]
        G.compare_decisions(parent, rows, o["accept"].cpu().numpy(), res["path_nodes"], res["path_len"], cb.SELECT_LONGEST)
        kids = O.children_of(parent)
        paths = []
        for b in range(B):
            path = [int(x) for x in res["path_nodes"][b][: res["path_len"][b] + 1]]
            paths.append(path)
            end = path[-1]
            want, mass = O.bonus_token(logits[b, end], [tok[b, c] for c in kids[end]], ub[b])
            if want != res["bonus"][b]:
                # only a draw that lands on a boundary of the cumulative distribution may differ, by one place
                g = O.softmax(logits[b, end].astype(np.float64))
                for c in kids[end]:
                    g[tok[b, c]] = 0
                c = np.cumsum(g)
                assert abs(c[min(want, res["bonus"][b])] - ub[b] * g.sum()) < 1e-5
            assert abs(float(loop.mass[b]) - mass) < 1e-4
            total_accepted += len(path) - 1
        # cache append: exactly the rotated tree rows of the path, at the old prefix lengths, in every layer
        k_out = o["k_tree_out"].float().cpu().numpy()
        v_out = o["v_tree_out"].float().cpu().numpy()
        new_len = loop.set.dev["prefix_len"].cpu().numpy()
        for li in range(n_layers):
            kc = loop.set.dev["layers"][li]["k_prefix"].float().cpu().numpy()
            vc = loop.set.dev["layers"][li]["v_prefix"].float().cpu().numpy()
            for b in range(B):
                for r in (b, B + b):
                    n = len(paths[b])
                    assert np.array_equal(kc[r, plen[r]:plen[r] + n], k_out[li, r, paths[b]])
                    assert np.array_equal(vc[r, plen[r]:plen[r] + n], v_out[li, r, paths[b]])
                    assert new_len[r] == plen[r] + n
            # the checker's caches take its own rows for the same path
            q_ref, k_ref, v_ref = ref["attn_io"][li]
            O.append_path_kv(k_cache[li], v_cache[li], plen, k_ref, v_ref, paths, B)
        plen = np.array([plen[r] + len(paths[r % B]) for r in range(2 * B)])
        assert np.array_equal(plen, loop.prefix_len_host)
    assert total_accepted > 0
    assert all(len(e) >= steps for e in loop.emitted)
    loop.close()


def test_append_beyond_the_cache_is_refused_not_written():
    w = synth.workload("mini", B=1, tree="topk16", prefix_len=40)
    loop = DecodeLoop(w, 1, max_steps=1, seed=3)
    loop.step()
    with pytest.raises(cb.CascadeError) as e:   # the second step has no room left
        loop.step()
        loop.step()
    assert e.value.status == cb.ERR_OVERFLOW
    loop.close()


def test_residual_draw_of_algorithm_1():
    """cascade_bonus_token with the drafter's full row at the path's end node: [q - p]+ normalised after a
    rejection, q after a fully accepted path, q where nothing of q lies above p.  Paths are set by hand so that
    all three cases occur; many uniforms per case."""
    from paper_2605_07230_b200.workload import PiecesWorkload
    w = synth.workload("mini", B=4, tree="topk32", V=4096)
    wl = PiecesWorkload(w, n_sets=1, keep_logits=True)
    s = wl.run(0)
    torch.cuda.synchronize()
    logits = s.out["logits"].cpu().numpy()
    parent = wl.parent
    kids = O.children_of(parent)
    depth = O.tree_depth(parent)
    leaf = next(j for j in range(len(parent)) if not kids[j] and depth[j] == wl.tree.depth)
    inner = next(j for j in range(1, len(parent)) if kids[j])
    ends = [0, inner, leaf, inner]                       # prompt 3: the drafter's row equals the target's
    nodes = np.full((w.B, wl.tree.depth + 1), -1, np.int32)
    plen = np.zeros(w.B, np.int32)
    for b, end in enumerate(ends):
        path = []
        i = end
        while i >= 0:
            path.append(i)
            i = parent[i]
        path.reverse()
        nodes[b, : len(path)] = path
        plen[b] = len(path) - 1
    rng = np.random.default_rng(23)
    draft = np.zeros((w.B, w.V), np.float32)
    for b, end in enumerate(ends):
        q = O.softmax(logits[b, end].astype(np.float64))
        if b == 3:
            draft[b] = q
            draft[b] = np.maximum(draft[b], q.astype(np.float32) * (1 + 1e-6))   # p >= q everywhere, in fp32 too
        else:
            soft = O.softmax(logits[b, end].astype(np.float64) / 1.5 + rng.normal(0, 0.5, w.V))
            draft[b] = soft
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(G.DEV)
    d_nodes, d_plen, d_draft = dev(nodes), dev(plen), dev(draft)
    token = torch.zeros(w.B, dtype=torch.int32, device=G.DEV)
    mass = torch.zeros(w.B, device=G.DEV)
    differ = 0
    for it in range(40):
        u = rng.random(w.B, dtype=np.float32)
        cb.cascade_bonus_token(wl.ctx, wl.tree, s.out["logits"], s.dev["tok"], d_nodes, d_plen, dev(u), token, mass,
                               draft_row=d_draft)
        torch.cuda.synchronize()
        got, got_mass = token.cpu().numpy(), mass.cpu().numpy()
        for b, end in enumerate(ends):
            want, total = O.residual_token(logits[b, end], draft[b], bool(kids[end]), u[b])
            assert abs(got_mass[b] - total) < 1e-4, (b, got_mass[b], total)
            if got[b] != want:
                # only a draw within 1e-5 of a step of the cumulative distribution may fall to the neighbour
                qv = O.softmax(logits[b, end].astype(np.float64))
                wgt = np.maximum(qv - draft[b], 0) if (kids[end] and np.maximum(qv - draft[b], 0).sum() > 0) else qv
                c = np.cumsum(wgt) / wgt.sum()
                assert abs(c[min(got[b], want)] - u[b]) < 1e-5, (b, got[b], want)
                differ += 1
    assert differ <= 4
    # without the drafter's row the entry keeps its other rule (children's tokens removed)
    u = rng.random(w.B, dtype=np.float32)
    cb.cascade_bonus_token(wl.ctx, wl.tree, s.out["logits"], s.dev["tok"], d_nodes, d_plen, dev(u), token, mass)
    torch.cuda.synchronize()
    tok = s.host["tok"]
    for b, end in enumerate(ends):
        want, total = O.bonus_token(logits[b, end], [tok[b, c] for c in kids[end]], u[b])
        assert abs(float(mass[b]) - total) < 1e-4
    wl.ctx.check()
    wl.close()
