"""Pins for the CPU checker's final norm + LM head + guidance mixing + vocabulary softmax."""
import numpy as np
import scipy.special
import torch

from oracle import cascade_oracle as O


def _case(seed=0, B=2, T=5, h=32, V=97):
    rng = np.random.default_rng(seed)
    hidden = rng.standard_normal((2 * B, T, h)) * 3
    gamma = rng.uniform(0.5, 1.5, h)
    W = rng.standard_normal((V, h)) * 0.1
    return hidden, gamma, W


def _library_logits(x, gamma, eps, W):
    xt = torch.from_numpy(x)
    n = torch.nn.functional.rms_norm(xt, (x.shape[-1],), torch.from_numpy(gamma), eps)
    return torch.nn.functional.linear(n, torch.from_numpy(W)).numpy(), n.numpy()


def test_scale_one_is_cond_and_zero_is_uncond():
    hidden, gamma, W = _case()
    B = hidden.shape[0] // 2
    l_c, n_c = _library_logits(hidden[:B], gamma, 1e-6, W)
    l_u, _ = _library_logits(hidden[B:], gamma, 1e-6, W)
    out1 = O.lm_head_cfg(hidden, gamma, 1e-6, W, 1.0)
    out0 = O.lm_head_cfg(hidden, gamma, 1e-6, W, 0.0)
    assert np.allclose(out1["logits"], l_c, atol=1e-12)
    assert np.allclose(out0["logits"], l_u, atol=1e-12)
    assert np.allclose(out1["feat"], n_c, atol=1e-13)
    assert np.allclose(out1["feat_norm"], np.linalg.norm(n_c, axis=-1), atol=1e-12)


def test_guidance_extrapolates_and_temperature_divides():
    hidden, gamma, W = _case(1)
    B = hidden.shape[0] // 2
    l_c, _ = _library_logits(hidden[:B], gamma, 1e-5, W)
    l_u, _ = _library_logits(hidden[B:], gamma, 1e-5, W)
    out = O.lm_head_cfg(hidden, gamma, 1e-5, W, 5.0, temperature=2.0)
    assert np.allclose(out["logits"], (5 * l_c - 4 * l_u) / 2.0, atol=1e-11)


def test_mixing_commutes_with_the_head():
    """W (n_u + s (n_c - n_u)) equals the two-product form: the fact the GPU path relies on."""
    hidden, gamma, W = _case(2)
    B = hidden.shape[0] // 2
    n = O.rmsnorm(hidden, gamma, 1e-6)
    mixed = (n[B:] + 3.0 * (n[:B] - n[B:])) @ W.T
    assert np.allclose(O.lm_head_cfg(hidden, gamma, 1e-6, W, 3.0)["logits"], mixed, atol=1e-11)


def test_rmsnorm_closed_form():
    x = np.array([[3.0, -4.0, 0.0, 0.0]])
    out = O.rmsnorm(x, np.array([1.0, 2.0, 1.0, 1.0]), 0.0)
    # mean square = 25/4, rms = 2.5
    assert np.allclose(out, [[1.2, -3.2, 0.0, 0.0]])


def test_lse_and_softmax_against_library():
    rng = np.random.default_rng(3)
    l = rng.standard_normal((3, 4, 50)) * 10 + 300  # large offset: must not overflow
    assert np.allclose(O.log_sum_exp(l), scipy.special.logsumexp(l, axis=-1), rtol=0, atol=1e-10)
    sm = O.softmax(l)
    assert np.allclose(sm.sum(-1), 1.0, atol=1e-12)
    assert np.allclose(sm, scipy.special.softmax(l, axis=-1), atol=1e-13)
    out = O.lm_head_cfg(*_case(4)[:2], 1e-6, _case(4)[2], 2.0)
    assert np.allclose(out["lse"], scipy.special.logsumexp(out["logits"], axis=-1), atol=1e-11)


def test_candidate_logits_pick_parent_and_grandparent_rows():
    logits = np.arange(2 * 4 * 10, dtype=np.float64).reshape(2, 4, 10)
    parent = np.array([-1, 0, 0, 1])
    tok = np.array([[9, 1, 2, 3], [0, 4, 5, 6]])
    lp, lg = O.candidate_logits(logits, tok, parent)
    assert lp[0].tolist() == [0, 1, 2, 13] and lg[0].tolist() == [0, 0, 0, 3]
    assert lp[1].tolist() == [0, 44, 45, 56] and lg[1].tolist() == [0, 0, 0, 46]
