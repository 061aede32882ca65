"""GPU parity at the full sizes of the batched sweep (8 prompts x CFG pair, 7B-shaped widths): the checker
computes sampled attention rows and sampled logits rows one by one, and the acceptance rule for every
prompt from the device's own features and logits."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from paper_2605_07230_b200.workload import PiecesWorkload
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

CELLS = [  # draft nodes, prefix length, cluster tightness
    (16, 256, 0.05),
    (32, 1024, 0.1),
    (64, 2048, 0.3),
    (128, 2880, 0.1),
]


@pytest.mark.parametrize("nodes,prefix,sigma", CELLS)
def test_sweep_cell(nodes, prefix, sigma):
    w = synth.workload("sweep", tree=f"topk{nodes}", prefix_len=prefix, sigma=sigma)
    wl = PiecesWorkload(w, n_sets=1, keep_logits=True)
    s = wl.run(0)
    torch.cuda.synchronize()
    wl.ctx.check()
    h, parent, T, B = s.host, wl.parent, wl.T, w.B
    rng = np.random.default_rng(nodes)
    # (a) attention: a few (CFG row, head) pairs, all tree rows
    att = s.out["attn_out"].float().cpu().numpy()
    scale = 1.0 / np.sqrt(w.head_dim)
    for _ in range(4):
        r, hd = int(rng.integers(0, 2 * B)), int(rng.integers(0, w.n_heads))
        sl = (slice(r, r + 1), slice(None), slice(hd, hd + 1))
        ref = O.tree_attention(h["q"][sl], h["k_prefix"][sl], h["v_prefix"][sl], h["prefix_len"][r:r + 1], h["k_tree"][sl],
                               h["v_tree"][sl], parent, scale)
        assert np.abs(att[r, :, hd] - ref[0, :, 0]).max() < 2e-2
    # (b) logits: a few (prompt, tree row) pairs, all vocabulary entries
    logits = s.out["logits"].cpu().numpy()
    lse = s.out["row_lse"].cpu().numpy()
    for _ in range(6):
        b, j = int(rng.integers(0, B)), int(rng.integers(0, T))
        hid = h["hidden"][[b, B + b], j][:, None, :]
        ref = O.lm_head_cfg(hid, h["gamma_final"], w.eps, h["w_head"], w.cfg_scale, 1.0)
        assert np.abs(logits[b, j] - ref["logits"][0, 0]).max() < 3e-2
        assert abs(lse[b, j] - ref["lse"][0, 0]) < 3e-3
    # (c), (d): the rule for every prompt, bit-exact away from the near band
    feat = s.out["feat"].cpu().numpy().astype(np.float64)
    rows = [O.relaxed_accept(feat[b], logits[b], h["tok"][b], parent, h["draft_p"][b], h["uniforms"][b], w.tau_pos,
                             w.tau_seq, w.tvd_budget) for b in range(B)]
    st = G.compare_decisions(parent, rows, s.out["accept"].cpu().numpy(), s.out["path_nodes"].cpu().numpy(),
                             s.out["path_len"].cpu().numpy(), cb.SELECT_LONGEST)
    assert st["paths_compared"] >= 1
    relaxed = sum(int((r["q_relaxed"] > r["q_plain"]).sum()) for r in rows)
    print(f"cell T={T} P={prefix} sigma={sigma}: relaxation raised {relaxed} nodes, "
          f"paths {s.out['path_len'].cpu().tolist()}, set aside {st['prompts_set_aside']} prompts")
    wl.close()
