"""GPU parity of the verification step run through decoder layers (embedding, layers with tree attention,
final norm, LM head, relaxed acceptance, path) against the fp64 checker on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from paper_2605_07230_b200.workload import LayerWorkload
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def oracle_step(wl, host):
    w = wl.w
    return O.verify_step(host["embed"], host["layers"], host["gamma_final"], host["w_head"], host["tok"], wl.parent,
                         host["k_prefix"], host["v_prefix"], host["prefix_len"], host["draft_p"], host["uniforms"],
                         w.n_heads, w.head_dim, w.eps, w.rope_base, w.cfg_scale, 1.0, w.tau_pos, w.tau_seq,
                         w.tvd_budget, kv_bf16=w.dtype == "bf16")


@pytest.mark.parametrize("name,over,n_layers", [
    ("toy", {}, 1),                                   # config 1: fp32, 15 rows, one layer
    ("mini", {}, 1),                                  # bf16, 33 rows x 2 prompts
    ("mini", dict(B=1, tree="topk60", prefix_len=130), 2),   # two layers, 61 rows
])
def test_step_through_layers(name, over, n_layers):
    w = synth.workload(name, **over)
    host = None
    if name == "toy":
        # config 1: plain N(0, 0.02) weights and draft tokens sampled from the target's softmax at T = 1.5
        parent = w.parent()
        host = synth.layer_step_inputs(w, np.random.default_rng(w.seed), parent, n_layers)
        host["tok"], host["draft_p"] = G.target_sampled_drafts(w, host, parent, np.random.default_rng(7))
    wl = LayerWorkload(w, n_layers=n_layers, keep_logits=True, host=host)
    s = wl.run(0)
    torch.cuda.synchronize()
    wl.ctx.check()
    ref = oracle_step(wl, s.host)
    bf16 = w.dtype == "bf16"
    # rotated keys / values of the tree rows (what a caller appends to the cache)
    for li in range(n_layers):
        q, k, v = ref["attn_io"][li]
        assert np.abs(s.out["k_tree_out"][li].float().cpu().numpy() - k).max() < (4e-2 if bf16 else 1e-5)
        assert np.abs(s.out["v_tree_out"][li].float().cpu().numpy() - v).max() < (4e-2 if bf16 else 1e-5)
    hid_err = np.abs(s.out["hidden_out"].cpu().numpy() - ref["hidden"]).max()
    assert hid_err < (2e-2 if bf16 else 1e-4), hid_err
    logits = s.out["logits"].cpu().numpy()
    logit_err = np.abs(logits - ref["head"]["logits"]).max()
    assert logit_err < (3e-2 if bf16 else 1e-3), logit_err
    # decisions: the checker's rule on the device's own features and logits
    feat = s.out["feat"].cpu().numpy().astype(np.float64)
    rows = [O.relaxed_accept(feat[b], logits[b], s.host["tok"][b], wl.parent, s.host["draft_p"][b],
                             s.host["uniforms"][b], w.tau_pos, w.tau_seq, w.tvd_budget) for b in range(w.B)]
    G.compare_decisions(wl.parent, rows, s.out["accept"].cpu().numpy(), s.out["path_nodes"].cpu().numpy(),
                        s.out["path_len"].cpu().numpy(), cb.SELECT_LONGEST)
    accepted = int(s.out["accept"].cpu().numpy().sum()) - w.B
    assert accepted > 0                      # the workload is not degenerate: some drafts are accepted
    print(f"{name} x{n_layers}: hidden max-abs {hid_err:.2e}, logits max-abs {logit_err:.2e}, "
          f"{wl.ctx.last_launch_count} kernels, {accepted} drafts accepted, path lengths {s.out['path_len'].cpu().tolist()}")
    wl.close()


def test_step_without_hidden_output_matches():
    """Without hidden_out the last MLP output is added inside the final norm (one kernel fewer): same
    arithmetic in the same order, so logits, features and decisions are bit-identical."""
    w = synth.workload("mini", B=2)
    a = LayerWorkload(w, n_layers=2, keep_logits=True)
    b = LayerWorkload(w, n_layers=2, keep_logits=True, want_hidden=False)
    sa, sb = a.run(0), b.run(0)
    torch.cuda.synchronize()
    a.ctx.check()
    b.ctx.check()
    assert b.ctx.last_launch_count == a.ctx.last_launch_count - 1
    for key in ("logits", "feat", "accept", "path_nodes", "path_len", "row_lse"):
        assert torch.equal(sa.out[key], sb.out[key]), key
    a.close()
    b.close()


def test_layers_need_stacked_projection_weights():
    w = synth.workload("mini", B=1)
    wl = LayerWorkload(w, n_layers=1)
    st = wl.sets[0].step
    import ctypes as C
    saved = st.layers[0].wk
    st.layers[0].wk = st.layers[0].wv          # no longer right behind wq in memory
    assert cb.lib().cascade_verify_step(wl.ctx.handle, wl.tree.handle, C.byref(st), None) == cb.ERR_UNSUPPORTED_SHAPE
    st.layers[0].wk = saved
    wl.close()
