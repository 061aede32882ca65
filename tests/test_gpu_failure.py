"""Failure detection on the device and stale-state hazards of the host-buffer entry point.

No test here faults, traps or hangs a GPU: the only device-side failure is a bounded wait on a barrier that
nothing arrives on, which gives up after one millisecond and returns through the kernel's normal teardown."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from paper_2605_07230_b200.workload import PiecesWorkload
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _step_matches_checker(wl):
    w = wl.w
    s = wl.run(0)
    torch.cuda.synchronize()
    wl.ctx.check()
    h = s.host
    ref = O.lm_head_cfg(h["hidden"], h["gamma_final"], w.eps, h["w_head"], w.cfg_scale, 1.0)
    logits = s.out["logits"].cpu().numpy()
    assert np.abs(logits - ref["logits"]).max() < 3e-2
    att = O.tree_attention(h["q"], h["k_prefix"], h["v_prefix"], h["prefix_len"], h["k_tree"], h["v_tree"], wl.parent,
                           1.0 / np.sqrt(w.head_dim))
    assert np.abs(s.out["attn_out"].float().cpu().numpy() - att).max() < 2e-2
    feat = s.out["feat"].cpu().numpy().astype(np.float64)
    rows = [O.relaxed_accept(feat[b], logits[b], h["tok"][b], wl.parent, h["draft_p"][b], h["uniforms"][b], w.tau_pos,
                             w.tau_seq, w.tvd_budget) for b in range(w.B)]
    G.compare_decisions(wl.parent, rows, s.out["accept"].cpu().numpy(), s.out["path_nodes"].cpu().numpy(),
                        s.out["path_len"].cpu().numpy(), cb.SELECT_LONGEST)


def test_a_wait_that_cannot_end_times_out_and_the_context_stays_usable():
    w = synth.workload("mini", B=2)
    wl = PiecesWorkload(w, n_sets=1, keep_logits=True)
    _step_matches_checker(wl)
    wl.ctx.set_wait_limit(1_000_000)                   # 1 ms
    waited = torch.zeros(1, dtype=torch.int32, device=G.DEV)
    wl.ctx.wait_probe(waited)
    with pytest.raises(cb.CascadeError) as e:
        wl.ctx.check()
    assert e.value.status == cb.ERR_TIMEOUT
    ns = int(waited.item())
    assert 1_000_000 <= ns < 100_000_000, ns           # it waited out the limit, not the default two seconds
    wl.ctx.check()                                      # the error word was cleared by the failed check
    wl.ctx.set_wait_limit(2_000_000_000)
    _step_matches_checker(wl)                           # same context, same scratch, tensor memory free again
    with pytest.raises(cb.CascadeError):
        wl.ctx.set_wait_limit(10)                       # below a microsecond: refused
    wl.close()


def test_host_entry_does_not_replay_a_graph_recorded_for_a_destroyed_tree():
    """A tree destroyed and another created right after often gets the same host address; the step recorded for
    the first one (its row count, grid sizes, device arrays) must not be replayed for the second."""
    w = synth.workload("mini", B=2, tree="topk60")
    wl = PiecesWorkload(w, n_sets=1, keep_logits=True)
    s = wl.sets[0]
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    side = torch.cuda.Stream()

    def host_call(tree, T, tok, p, u):
        accept = torch.zeros((w.B, T), dtype=torch.uint8).pin_memory()
        nodes = torch.zeros((w.B, tree.depth + 1), dtype=torch.int32).pin_memory()
        plen = torch.zeros(w.B, dtype=torch.int32).pin_memory()
        with torch.cuda.stream(side):
            cb.cascade_verify_step_host(wl.ctx, tree, s.step, pin(tok), pin(p), pin(u), accept, nodes, plen)
        return accept.numpy().copy(), nodes.numpy().copy(), plen.numpy().copy()

    for _ in range(3):                                  # the second call records, the third replays
        host_call(wl.tree, wl.T, s.host["tok"], s.host["draft_p"], s.host["uniforms"])
    wl.tree.close()
    # a smaller tree in a new descriptor; the step's big inputs are reused with the first T2 rows' worth of data
    w2 = synth.workload("mini", B=2, tree="topk16")
    parent2 = w2.parent()
    T2 = len(parent2)
    tree2 = cb.Tree(wl.ctx, parent2)
    rng = np.random.default_rng(9)
    host2 = synth.tail_inputs(w2, rng, parent2)
    att2 = synth.attention_inputs(w2, rng, T2)
    d = s.dev
    el = torch.bfloat16
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(G.DEV)
    bufs = dict(hidden=G.to_dev(host2["hidden"], "bf16"), q=G.to_dev(att2["q"], "bf16"),
                k_tree=G.to_dev(att2["k_tree"], "bf16"), v_tree=G.to_dev(att2["v_tree"], "bf16"),
                tok=dev(host2["tok"]), draft_p=dev(host2["draft_p"]), uniforms=dev(host2["uniforms"]))
    out2 = dict(attn_out=torch.zeros((2 * w.B, T2, w.n_heads, w.head_dim), dtype=el, device=G.DEV),
                accept=torch.zeros((w.B, T2), dtype=torch.uint8, device=G.DEV),
                path_nodes=torch.zeros((w.B, tree2.depth + 1), dtype=torch.int32, device=G.DEV),
                path_len=torch.zeros(w.B, dtype=torch.int32, device=G.DEV))
    step2 = cb.make_step(layers=None, gamma_final=d["gamma_final"], w_head=d["w_head"], prefix_cap=w.prefix_len,
                         prefix_len=d["prefix_len"], eps=w.eps, rope_base=w.rope_base,
                         softmax_scale=float(1.0 / np.sqrt(w.head_dim)), cfg_scale=w.cfg_scale, temperature=1.0,
                         tok=bufs["tok"], draft_p=bufs["draft_p"], uniforms=bufs["uniforms"], hidden_in=bufs["hidden"],
                         q=bufs["q"], k_tree=bufs["k_tree"], v_tree=bufs["v_tree"], k_prefix=d["k_prefix"],
                         v_prefix=d["v_prefix"], attn_out=out2["attn_out"], params=wl.params,
                         select_mode=cb.SELECT_LONGEST, accept=out2["accept"], path_nodes=out2["path_nodes"],
                         path_len=out2["path_len"])
    cb.cascade_verify_step(wl.ctx, tree2, step2)
    torch.cuda.synchronize()
    want = {k: out2[k].cpu().numpy().copy() for k in ("accept", "path_nodes", "path_len")}
    s.step = step2                                      # host_call passes s.step
    for _ in range(3):
        a, n, l = host_call(tree2, T2, host2["tok"], host2["draft_p"], host2["uniforms"])
        assert np.array_equal(a, want["accept"]) and np.array_equal(n, want["path_nodes"]) and np.array_equal(l, want["path_len"])
    wl.ctx.check()
    tree2.close()
    wl.ctx.close()


def test_allocation_free_entry_refuses_a_stream_that_is_recording():
    """Its copies read host memory of the call itself, so they must not end up in a recorded graph.  Nothing is
    enqueued: the capture below ends empty."""
    import ctypes as C
    L = cb.lib()
    params = cb.Params(0.85, 0.5, 0.5, cb.USE_I | cb.USE_C)
    parent = (C.c_int32 * 2)(-1, 0)
    buf = torch.zeros(64, device=G.DEV)
    p = buf.data_ptr()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        g.capture_begin()
        rc = L.cascade_accept_static(1, 2, parent, p, 4, None, p, p, p, p, p, p, C.byref(params), 0, p, None, None,
                                     None, p, p, None, side.cuda_stream)
        g.capture_end()
    assert rc == cb.ERR_INVALID_ARG
