"""Pins for the CPU checker's tree attention: textbook special cases and invariants."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import synth


def _rand(rng, R, T, P, Hq, Hkv, D):
    q = rng.standard_normal((R, T, Hq, D))
    kp = rng.standard_normal((R, P, Hkv, D))
    vp = rng.standard_normal((R, P, Hkv, D))
    kt = rng.standard_normal((R, T, Hkv, D))
    vt = rng.standard_normal((R, T, Hkv, D))
    return q, kp, vp, kt, vt


def test_chain_tree_is_causal_attention_library():
    """A chain tree is plain causal attention over prefix+tree tokens (torch SDPA as the library)."""
    rng = np.random.default_rng(0)
    R, T, P, H, D = 2, 7, 11, 3, 16
    q, kp, vp, kt, vt = _rand(rng, R, T, P, H, H, D)
    out = O.tree_attention(q, kp, vp, [P, P], kt, vt, synth.chain_tree(T - 1), 1 / np.sqrt(D))
    for r in range(R):
        k_all = torch.from_numpy(np.concatenate([kp[r], kt[r]], 0)).permute(1, 0, 2)  # [H,P+T,D]
        v_all = torch.from_numpy(np.concatenate([vp[r], vt[r]], 0)).permute(1, 0, 2)
        # pad the queries with dummies for the prefix positions so is_causal lines up
        q_all = torch.cat([torch.zeros(H, P, D, dtype=torch.float64), torch.from_numpy(q[r]).permute(1, 0, 2)], 1)
        ref = torch.nn.functional.scaled_dot_product_attention(q_all, k_all, v_all, is_causal=True)
        ref = ref[:, P:].permute(1, 0, 2).numpy()
        assert np.allclose(out[r], ref, atol=1e-12)


def test_single_row_is_decode_attention():
    rng = np.random.default_rng(1)
    R, T, P, H, D = 1, 1, 9, 2, 8
    q, kp, vp, kt, vt = _rand(rng, R, T, P, H, H, D)
    out = O.tree_attention(q, kp, vp, [P], kt, vt, np.array([-1]), 0.3)
    for hd in range(H):
        keys = np.concatenate([kp[0, :, hd], kt[0, :, hd]])
        vals = np.concatenate([vp[0, :, hd], vt[0, :, hd]])
        s = 0.3 * keys @ q[0, 0, hd]
        w = torch.softmax(torch.from_numpy(s), 0).numpy()
        assert np.allclose(out[0, 0, hd], w @ vals, atol=1e-13)


def test_two_key_closed_form():
    """One prefix key + the root itself: weights are a logistic function of the score difference."""
    D = 4
    q = np.array([1.0, 0, 0, 0]).reshape(1, 1, 1, D)
    kp = np.array([2.0, 0, 0, 0]).reshape(1, 1, 1, D)
    kt = np.array([-1.0, 5, 5, 5]).reshape(1, 1, 1, D)
    vp = np.array([1.0, 0, 0, 0]).reshape(1, 1, 1, D)
    vt = np.array([0.0, 1, 0, 0]).reshape(1, 1, 1, D)
    out = O.tree_attention(q, kp, vp, [1], kt, vt, np.array([-1]), 1.0)
    w_prefix = 1 / (1 + np.exp(-3.0))  # scores 2 and -1
    assert np.allclose(out[0, 0, 0], [w_prefix, 1 - w_prefix, 0, 0], atol=1e-15)


def test_equal_values_give_that_value_and_prefix_len_is_respected():
    rng = np.random.default_rng(2)
    R, T, P, H, D = 2, 15, 10, 2, 8
    q, kp, vp, kt, vt = _rand(rng, R, T, P, H, H, D)
    parent = synth.complete_tree(2, 3)
    vp[:] = 0.25
    vt[:] = 0.25
    out = O.tree_attention(q, kp, vp, [P, P - 3], kt, vt, parent, 0.5)
    assert np.allclose(out, 0.25, atol=1e-14)
    # entries of the cache beyond prefix_len must not matter
    vp2 = rng.standard_normal(vp.shape)
    kp2 = kp.copy()
    a = O.tree_attention(q, kp, vp2, [P, P - 3], kt, vt, parent, 0.5)
    kp2[1, P - 3:] += 100.0
    vp3 = vp2.copy()
    vp3[1, P - 3:] -= 7.0
    b = O.tree_attention(q, kp2, vp3, [P, P - 3], kt, vt, parent, 0.5)
    assert np.array_equal(a, b)


def test_row_ignores_non_ancestors():
    rng = np.random.default_rng(3)
    R, T, P, H, D = 1, 15, 5, 2, 8
    parent = synth.complete_tree(2, 3)
    q, kp, vp, kt, vt = _rand(rng, R, T, P, H, H, D)
    base = O.tree_attention(q, kp, vp, [P], kt, vt, parent, 0.4)
    anc = O.ancestor_mask(parent)
    for j in [3, 9, 14]:
        kt2, vt2 = kt.copy(), vt.copy()
        others = ~anc[j]
        kt2[0, others] += rng.standard_normal((int(others.sum()), H, D)) * 5
        vt2[0, others] += 3.0
        pert = O.tree_attention(q, kp, vp, [P], kt2, vt2, parent, 0.4)
        assert np.array_equal(base[0, j], pert[0, j])
        # ... and does depend on every ancestor
        for i in np.nonzero(anc[j])[0]:
            vt3 = vt.copy()
            vt3[0, i] += 1.0
            assert not np.allclose(base[0, j], O.tree_attention(q, kp, vp, [P], kt, vt3, parent, 0.4)[0, j])


def test_ancestor_mask_of_toy_tree():
    anc = O.ancestor_mask(synth.complete_tree(2, 3))
    assert anc.sum(1).tolist() == [1, 2, 2, 3, 3, 3, 3] + [4] * 8
    assert anc[14].nonzero()[0].tolist() == [0, 2, 6, 14]
    assert anc[7].nonzero()[0].tolist() == [0, 1, 3, 7]


def test_grouped_query_heads_share_kv():
    rng = np.random.default_rng(4)
    R, T, P, Hq, Hkv, D = 1, 4, 6, 4, 2, 8
    q, kp, vp, kt, vt = _rand(rng, R, T, P, Hq, Hkv, D)
    parent = synth.chain_tree(T - 1)
    out = O.tree_attention(q, kp, vp, [P], kt, vt, parent, 0.35)
    rep = lambda x: np.repeat(x, Hq // Hkv, axis=2)
    ref = O.tree_attention(q, rep(kp), rep(vp), [P], rep(kt), rep(vt), parent, 0.35)
    assert np.allclose(out, ref, atol=1e-14)
