"""GPU parity of the fused verification step (pieces (a)-(d) in one enqueue), device and host entry."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from paper_2605_07230_b200.workload import PiecesWorkload
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def check_step(wl: PiecesWorkload, s, mode, flags):
    w, parent, T = wl.w, wl.parent, wl.T
    h = s.host
    torch.cuda.synchronize()
    wl.ctx.check()
    scale = 1.0 / np.sqrt(w.head_dim)
    # (a) numerics
    ref_att = O.tree_attention(h["q"], h["k_prefix"], h["v_prefix"], h["prefix_len"], h["k_tree"], h["v_tree"],
                               parent, scale)
    att_err = np.abs(s.out["attn_out"].float().cpu().numpy() - ref_att).max()
    assert att_err < (2e-2 if w.dtype == "bf16" else 1e-5), att_err
    # (b) numerics
    ref_head = O.lm_head_cfg(h["hidden"], h["gamma_final"], w.eps, h["w_head"], w.cfg_scale, 1.0)
    logits = s.out["logits"].cpu().numpy()
    assert np.abs(logits - ref_head["logits"]).max() < 3e-2
    assert np.abs(s.out["row_lse"].cpu().numpy() - ref_head["lse"]).max() < 3e-3
    # (c)+(d): the checker's rule applied to the device's own features / logits must give the same bits
    feat = s.out["feat"].cpu().numpy().astype(np.float64)
    rows = [O.relaxed_accept(feat[b], logits[b], h["tok"][b], parent, h["draft_p"][b], h["uniforms"][b], w.tau_pos,
                             w.tau_seq, w.tvd_budget, flags) for b in range(w.B)]
    st = G.compare_decisions(parent, rows, s.out["accept"].cpu().numpy(), s.out["path_nodes"].cpu().numpy(),
                             s.out["path_len"].cpu().numpy(), mode)
    # end to end (checker from the raw inputs): reported, and expected to agree except at near ties
    full = [O.relaxed_accept(ref_head["feat"][b], ref_head["logits"][b], h["tok"][b], parent, h["draft_p"][b],
                             h["uniforms"][b], w.tau_pos, w.tau_seq, w.tvd_budget, flags) for b in range(w.B)]
    # fraction of nodes on which the two accept masks agree (a score inside the near band, or a logit
    # that differs in its last bits, may flip a node: reported, with a loose floor)
    got = s.out["accept"].cpu().numpy()
    agree = np.mean([np.mean(full[b]["accept"] == got[b]) for b in range(w.B)])
    return st, agree, rows


@pytest.mark.parametrize("name,over", [
    ("toy", {}),
    ("mini", {}),
    ("mini", dict(B=4, tree="topk60", tau_pos=0.95, tau_seq=0.925, cfg_scale=3.0)),
    ("mini", dict(B=3, tree="topk128", prefix_len=130)),
])
@pytest.mark.parametrize("mode", [cb.SELECT_LONGEST, cb.SELECT_FIRST_ACCEPT])
def test_fused_step(name, over, mode):
    w = synth.workload(name, **over)
    flags = cb.USE_I | cb.USE_C
    wl = PiecesWorkload(w, n_sets=2, keep_logits=True, select_mode=mode, flags=flags)
    compared = relaxed = 0
    agree = []
    for i in range(2):
        s = wl.run(i)
        st, a, rows = check_step(wl, s, mode, flags)
        compared += st["paths_compared"]
        relaxed += sum(int((r["q_relaxed"] > r["q_plain"]).sum()) for r in rows)
        agree.append(a)
    assert compared >= 1
    assert relaxed > 0                      # the relaxation took part in these decisions
    assert np.mean(agree) >= 0.9
    assert wl.ctx.last_launch_count >= 4
    wl.close()


def test_host_entry_matches_device_entry():
    w = synth.workload("mini", B=2)
    wl = PiecesWorkload(w, n_sets=1, keep_logits=True)
    s = wl.run(0)
    torch.cuda.synchronize()
    want = {k: s.out[k].cpu().numpy().copy() for k in ("accept", "path_nodes", "path_len")}
    pin = lambda a: torch.from_numpy(a).pin_memory()
    tok, p, u = pin(s.host["tok"]), pin(s.host["draft_p"]), pin(s.host["uniforms"])
    accept = torch.zeros((w.B, wl.T), dtype=torch.uint8).pin_memory()
    nodes = torch.zeros((w.B, wl.tree.depth + 1), dtype=torch.int32).pin_memory()
    plen = torch.zeros(w.B, dtype=torch.int32).pin_memory()
    for _ in range(2):
        cb.cascade_verify_step_host(wl.ctx, wl.tree, s.step, tok, p, u, accept, nodes, plen)
        assert np.array_equal(accept.numpy(), want["accept"])
        assert np.array_equal(nodes.numpy(), want["path_nodes"])
        assert np.array_equal(plen.numpy(), want["path_len"])
    wl.close()


def test_host_entry_replays_a_recorded_graph_with_new_inputs():
    """On a stream of its own the host entry records the repeated call as a CUDA graph (from the second
    identical call on); every call must still give what the device entry gives for that call's inputs,
    also when the caller alternates between two step structures."""
    w = synth.workload("mini", B=2)
    wl = PiecesWorkload(w, n_sets=2, keep_logits=True)
    rng = np.random.default_rng(3)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    accept = torch.zeros((w.B, wl.T), dtype=torch.uint8).pin_memory()
    nodes = torch.zeros((w.B, wl.tree.depth + 1), dtype=torch.int32).pin_memory()
    plen = torch.zeros(w.B, dtype=torch.int32).pin_memory()
    side = torch.cuda.Stream()
    lengths = set()
    for it in range(8):
        st = wl.sets[it % 2]
        u = rng.random((w.B, wl.T), dtype=np.float32)            # new uniforms every call: different decisions
        tok, p = st.host["tok"], st.host["draft_p"]
        st.dev["uniforms"].copy_(torch.from_numpy(u))
        wl.run(it % 2)                                             # device entry on the same inputs
        torch.cuda.synchronize()
        want = {k: st.out[k].cpu().numpy().copy() for k in ("accept", "path_nodes", "path_len")}
        with torch.cuda.stream(side):
            cb.cascade_verify_step_host(wl.ctx, wl.tree, st.step, pin(tok), pin(p), pin(u), accept, nodes, plen)
        assert wl.ctx.last_launch_count == 4
        assert np.array_equal(accept.numpy(), want["accept"]), it
        assert np.array_equal(nodes.numpy(), want["path_nodes"]) and np.array_equal(plen.numpy(), want["path_len"])
        lengths.add(tuple(plen.numpy().tolist()))
    assert len(lengths) > 1                                        # the replays really saw different inputs
    wl.ctx.check()
    wl.close()


def test_step_refuses_bad_arguments():
    w = synth.workload("mini", B=1)
    wl = PiecesWorkload(w, n_sets=1)
    import copy
    import ctypes as C
    L = cb.lib()
    st = wl.sets[0].step
    saved = st.tok
    st.tok = None
    assert L.cascade_verify_step(wl.ctx.handle, wl.tree.handle, C.byref(st), None) == cb.ERR_INVALID_ARG
    st.tok = saved
    st.params.tvd_budget = -1.0
    assert L.cascade_verify_step(wl.ctx.handle, wl.tree.handle, C.byref(st), None) == cb.ERR_INVALID_ARG
    st.params.tvd_budget = 0.5
    st.select_mode = 7
    assert L.cascade_verify_step(wl.ctx.handle, wl.tree.handle, C.byref(st), None) == cb.ERR_INVALID_ARG
    wl.close()


@pytest.mark.parametrize("tree", [
    "chain0",        # the root alone: nothing drafted, the path is the root
    "nary32x1",      # one sibling group of the maximum width (496 sibling pairs)
    "nary2x7",       # 255 rows, seven levels: the row limit of a tree is 256
    "nary15x2",      # 241 rows, 1680 sibling pairs + 240 edges
])
def test_degenerate_and_maximal_trees(tree):
    w = synth.workload("mini", B=2, tree=tree, prefix_len=70)
    for mode in (cb.SELECT_LONGEST, cb.SELECT_FIRST_ACCEPT):
        wl = PiecesWorkload(w, n_sets=1, keep_logits=True, select_mode=mode, flags=cb.USE_I | cb.USE_C)
        s = wl.run(0)
        st, agree, rows = check_step(wl, s, mode, cb.USE_I | cb.USE_C)
        assert st["prompts"] == w.B
        if tree == "chain0":
            assert s.out["path_len"].cpu().tolist() == [0, 0] and s.out["accept"].cpu().numpy().all()
        wl.close()
