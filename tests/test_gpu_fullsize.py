"""GPU parity at the sizes the benchmark runs: the Janus-Pro-7B- and Lumina-mGPT-7B-768-shaped verification
steps through one full-width decoder layer (hidden 4096, 32 heads x 128, SwiGLU 11008, vocabulary 16384 / 65536,
prefix 384 / 2480, 61 tree rows), the LM head alone at vocabulary 65536 with 61 and 122 rows, and the tree
attention alone at 32 heads over a 2480-key prefix -- every output element against the fp64 checker on the same
seeded inputs.  These are the launch configurations bench.py times: the projections' sliced and balanced modes with
dozens of units per CTA, the head's contiguous mode with several whole tiles per CTA and both hand-off roles in
one CTA, the attention with 32 heads x 2 splits."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from paper_2605_07230_b200.workload import LayerWorkload
from tests import gpu_util as G
from tests.test_gpu_attention import ATTN_TOL, run_attention
from tests.test_gpu_head import LOGIT_TOL, run_head

pytestmark = pytest.mark.gpu

HIDDEN_TOL = 2e-2


@pytest.mark.parametrize("name", ["janus", "lumina", "llamagen"])
def test_full_width_step_through_one_layer(name):
    w = synth.workload(name)
    wl = LayerWorkload(w, n_layers=1, keep_logits=True)
    s = wl.run(0)
    torch.cuda.synchronize()
    wl.ctx.check()
    h = s.host
    ref = O.verify_step(h["embed"], h["layers"], h["gamma_final"], h["w_head"], h["tok"], wl.parent, h["k_prefix"],
                        h["v_prefix"], h["prefix_len"], h["draft_p"], h["uniforms"], w.n_heads, w.head_dim, w.eps,
                        w.rope_base, w.cfg_scale, 1.0, w.tau_pos, w.tau_seq, w.tvd_budget, kv_bf16=True)
    q, k, v = ref["attn_io"][0]
    k_err = np.abs(s.out["k_tree_out"][0].float().cpu().numpy() - k).max()
    v_err = np.abs(s.out["v_tree_out"][0].float().cpu().numpy() - v).max()
    assert k_err < 4e-2 and v_err < 4e-2, (k_err, v_err)       # one bf16 step at |k| up to ~8
    hid_err = np.abs(s.out["hidden_out"].cpu().numpy() - ref["hidden"]).max()
    assert hid_err < HIDDEN_TOL, hid_err
    logits = s.out["logits"].cpu().numpy()
    logit_err = np.abs(logits - ref["head"]["logits"]).max()
    assert logit_err < LOGIT_TOL, logit_err
    # a row's log-sum-exp moves by at most the largest error of its logits; against the device's own stored logits
    # it must be tight
    lse = s.out["row_lse"].cpu().numpy()
    assert np.abs(lse - ref["head"]["lse"]).max() < LOGIT_TOL
    assert np.abs(lse - O.log_sum_exp(logits)).max() < 2e-3
    assert np.abs(s.out["feat"].cpu().numpy() - ref["head"]["feat"]).max() < 2e-2
    # decisions: the checker's rule on the device's own features and logits, bit-exact outside the near band
    feat = s.out["feat"].cpu().numpy().astype(np.float64)
    rows = [O.relaxed_accept(feat[b], logits[b], h["tok"][b], wl.parent, h["draft_p"][b], h["uniforms"][b], w.tau_pos,
                             w.tau_seq, w.tvd_budget) for b in range(w.B)]
    st = G.compare_decisions(wl.parent, rows, s.out["accept"].cpu().numpy(), s.out["path_nodes"].cpu().numpy(),
                             s.out["path_len"].cpu().numpy(), cb.SELECT_LONGEST)
    # the checker end to end (its own hidden states and logits): reported, with a loose floor
    agree = float(np.mean([np.mean(s.out["accept"][b].cpu().numpy() == ref["accept"][b]["accept"]) for b in range(w.B)]))
    assert agree >= 0.9, agree
    print(f"{name} full width: k/v {k_err:.1e}/{v_err:.1e}, hidden {hid_err:.2e}, logits {logit_err:.2e}, "
          f"{wl.ctx.last_launch_count} kernels, nodes compared {st['nodes_compared']}/{st['nodes']}, set aside "
          f"{st['nodes_set_aside']}, device near count {s.out['near_count'].cpu().tolist()}, end-to-end node agreement "
          f"{agree:.3f}, path lengths {s.out['path_len'].cpu().tolist()}")
    wl.close()


def test_two_full_width_layers_each_against_the_checker_on_the_same_input():
    """The decode loop's widths (hidden 4096, 32 heads x 128, SwiGLU 11008, vocabulary 16384, a 64-row prompt cache,
    61 tree rows), two layers.  Layer 1 is compared with the checker from the token embeddings; layer 2 and the head
    are compared with the checker run on the DEVICE's layer-1 output, so that both sides round the same values to
    bf16 where the workload stores bf16 (rotated queries, keys, values).  End to end -- the checker on its own
    layer-1 output -- the two computations part by isolated bf16 steps in layer 2's operands; that figure is
    reported and held to twice the single-layer tolerance."""
    w = synth.workload("janus", prefix_len=64)
    parent = w.parent()
    host = synth.layer_step_inputs(w, np.random.default_rng(w.seed), parent, 2)
    first = dict(host, layers=host["layers"][:1], k_prefix=host["k_prefix"][:1], v_prefix=host["v_prefix"][:1])
    wl1 = LayerWorkload(w, n_layers=1, host=first)
    s1 = wl1.run(0)
    torch.cuda.synchronize()
    wl1.ctx.check()
    x1_dev = s1.out["hidden_out"].cpu().numpy().astype(np.float64)
    wl1.close()
    wl2 = LayerWorkload(w, n_layers=2, keep_logits=True, host=host)
    s2 = wl2.run(0)
    torch.cuda.synchronize()
    wl2.ctx.check()
    x2_dev = s2.out["hidden_out"].cpu().numpy()
    logits = s2.out["logits"].cpu().numpy()
    # layer 1 from the embeddings
    x0 = np.asarray(host["embed"], np.float64)[np.concatenate([host["tok"], host["tok"]], 0)]
    x1_ref, *_ = O.decoder_layer(x0, host["layers"][0], host["k_prefix"][0], host["v_prefix"][0], host["prefix_len"], parent,
                                 w.n_heads, w.head_dim, w.eps, w.rope_base, True)
    e1 = np.abs(x1_dev - x1_ref).max()
    assert e1 < HIDDEN_TOL, e1
    # layer 2 + head from the device's layer-1 output
    x2_ref, q, k, v = O.decoder_layer(x1_dev, host["layers"][1], host["k_prefix"][1], host["v_prefix"][1], host["prefix_len"],
                                      parent, w.n_heads, w.head_dim, w.eps, w.rope_base, True)
    e2 = np.abs(x2_dev - x2_ref).max()
    assert e2 < HIDDEN_TOL, e2
    assert np.abs(s2.out["k_tree_out"][1].float().cpu().numpy() - k).max() < 4e-2
    head = O.lm_head_cfg(x2_ref, host["gamma_final"], w.eps, host["w_head"], w.cfg_scale, 1.0)
    e_logits = np.abs(logits - head["logits"]).max()
    assert e_logits < LOGIT_TOL, e_logits
    # end to end, for the record
    x2_own, *_ = O.decoder_layer(x1_ref, host["layers"][1], host["k_prefix"][1], host["v_prefix"][1], host["prefix_len"], parent,
                                 w.n_heads, w.head_dim, w.eps, w.rope_base, True)
    own = O.lm_head_cfg(x2_own, host["gamma_final"], w.eps, host["w_head"], w.cfg_scale, 1.0)
    e_end = np.abs(logits - own["logits"]).max()
    assert e_end < 2 * LOGIT_TOL, e_end
    print(f"two full-width layers: hidden after layer 1 {e1:.2e}, after layer 2 (same input) {e2:.2e}, logits (same input) "
          f"{e_logits:.2e}, logits end to end {e_end:.2e}")
    wl2.close()


@pytest.mark.parametrize("nodes,prefix,sigma", [(16, 256, 0.3), (64, 1024, 0.1)])
def test_sweep_cell_through_one_layer(nodes, prefix, sigma):
    """Two cells of the batched sweep (8 prompts x CFG pair, 7B-shaped widths) as the benchmark runs them: through
    one full-width decoder layer, every output element.  The 64-node cell has 1040 projection rows (nine row chunks),
    the wide form of the attention (65 rows in one 128-row block) and the head's whole-item mode (520 rows)."""
    w = synth.workload("sweep", tree=f"topk{nodes}", prefix_len=prefix, sigma=sigma)
    wl = LayerWorkload(w, n_layers=1, keep_logits=True)
    s = wl.run(0)
    torch.cuda.synchronize()
    wl.ctx.check()
    h = s.host
    ref = O.verify_step(h["embed"], h["layers"], h["gamma_final"], h["w_head"], h["tok"], wl.parent, h["k_prefix"],
                        h["v_prefix"], h["prefix_len"], h["draft_p"], h["uniforms"], w.n_heads, w.head_dim, w.eps,
                        w.rope_base, w.cfg_scale, 1.0, w.tau_pos, w.tau_seq, w.tvd_budget, kv_bf16=True)
    hid_err = np.abs(s.out["hidden_out"].cpu().numpy() - ref["hidden"]).max()
    assert hid_err < HIDDEN_TOL, hid_err
    logits = s.out["logits"].cpu().numpy()
    logit_err = np.abs(logits - ref["head"]["logits"]).max()
    assert logit_err < LOGIT_TOL, logit_err
    feat = s.out["feat"].cpu().numpy().astype(np.float64)
    rows = [O.relaxed_accept(feat[b], logits[b], h["tok"][b], wl.parent, h["draft_p"][b], h["uniforms"][b], w.tau_pos,
                             w.tau_seq, w.tvd_budget) for b in range(w.B)]
    st = G.compare_decisions(wl.parent, rows, s.out["accept"].cpu().numpy(), s.out["path_nodes"].cpu().numpy(),
                             s.out["path_len"].cpu().numpy(), cb.SELECT_LONGEST)
    print(f"sweep cell {nodes} nodes, prefix {prefix}, sigma {sigma}, through one layer: hidden {hid_err:.2e}, logits "
          f"{logit_err:.2e}, nodes compared {st['nodes_compared']}/{st['nodes']}, paths {s.out['path_len'].cpu().tolist()}")
    wl.close()


@pytest.mark.parametrize("B", [1, 2])
def test_head_at_vocabulary_65536(B):
    """61 and 122 activation rows against a [65536, 4096] head: 512 vocabulary tiles x 32 K blocks over 148 CTAs, so
    every CTA holds whole tiles, finishes a tile another CTA began and hands its last one on."""
    w = synth.workload("lumina", B=B)
    parent = w.parent()
    got, ref, tok = run_head(w, parent, 41)
    err = np.abs(got["logits"] - ref["logits"]).max()
    assert err < LOGIT_TOL, err
    assert np.abs(got["feat"] - ref["feat"]).max() < 1e-4
    assert np.abs(got["lse"] - ref["lse"]).max() < 2e-3
    lp, lg = O.candidate_logits(ref["logits"], tok, parent)
    assert np.abs(got["cp"] - lp).max() < 2e-3 and np.abs(got["cg"] - lg).max() < 2e-3
    print(f"head V=65536, {B * len(parent)} rows: logits max-abs {err:.2e}")


@pytest.mark.parametrize("name", ["janus", "lumina"])
def test_attention_at_32_heads(name):
    w = synth.workload(name)
    got, ref, _ = run_attention(w, w.parent(), 43)
    assert np.isfinite(got).all()
    err = np.abs(got - ref).max()
    assert err < ATTN_TOL, err
    print(f"attention {name}: 32 heads, prefix {w.prefix_len}, max-abs {err:.2e}")
