"""GPU parity of the drafter loss kernel (Section 4.3, Eq. 4) against the fp64 checker."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _inputs(rng, K, V, h, conv_frac=0.5):
    """Target logits shaped like the workloads' (mass on a few hundred near-identical codes), a drafter that is a
    noisy copy, and hidden states that drift slowly over some stretches (convergent) and jump elsewhere."""
    centres = rng.normal(0, 1, 256)
    tl = (centres[np.arange(V) % 256][None, :] * (8.0 / 3.0) + rng.normal(0, 0.3, (K, V))).astype(np.float32)
    dl = (tl / 1.5 + rng.normal(0, 0.5, (K, V))).astype(np.float32)
    feat = np.zeros((K, h), np.float32)
    cur = rng.standard_normal(h)
    for k in range(K):
        cur = cur + 0.2 * rng.standard_normal(h) if rng.random() < conv_frac else rng.standard_normal(h)
        feat[k] = cur
    return tl, dl, feat


@pytest.mark.parametrize("K,V,h", [(64, 16384, 4096), (7, 1000, 64), (1, 8, 4), (33, 65536, 1280)])
def test_drafter_loss_against_checker(K, V, h):
    rng = np.random.default_rng(K + V)
    tl, dl, feat = _inputs(rng, K, V, h)
    dev = lambda a: torch.from_numpy(a).to(G.DEV)
    loss = torch.full((K,), float("nan"), device=G.DEV)
    w = torch.full((K,), float("nan"), device=G.DEV)
    total = torch.full((1,), float("nan"), device=G.DEV)
    cb.cascade_drafter_loss(dev(tl), dev(dl), dev(feat), 0.5, 2.0, loss, w, total)
    torch.cuda.synchronize()
    per, weights, tot = O.drafter_loss(tl, dl, feat, 0.5, 2.0)
    # weights are exact unless a cosine sits within 1e-5 of the threshold
    cos = np.array([O.cosine(feat[k], feat[k + 1]) for k in range(K - 1)] + [0.0])
    firm = np.abs(cos - 0.5) > 1e-5
    assert np.array_equal(w.cpu().numpy()[firm], weights[firm].astype(np.float32))
    if K > 4:
        assert 0 < (weights == 2.0).sum() < K             # both kinds of positions occur
    got = loss.cpu().numpy()
    assert np.abs(got[firm] - per[firm]).max() < 2e-4 * max(1.0, np.abs(per).max())
    if firm.all():
        assert abs(float(total) - tot) < 2e-4 * K * max(1.0, np.abs(per).max())
    # run twice: the total is added in a fixed order
    total2 = torch.zeros(1, device=G.DEV)
    cb.cascade_drafter_loss(dev(tl), dev(dl), dev(feat), 0.5, 2.0, loss, w, total2)
    torch.cuda.synchronize()
    assert float(total2) == float(total)


def test_drafter_loss_rejects_bad_arguments_and_handles_zero_probability_tokens():
    L = cb.lib()
    x = torch.zeros(16, device=G.DEV)
    p = x.data_ptr()
    assert L.cascade_drafter_loss(None, p, p, 1, 4, 4, 0.5, 2.0, p, None, None, None) == cb.ERR_INVALID_ARG
    assert L.cascade_drafter_loss(p, p, p, 0, 4, 4, 0.5, 2.0, p, None, None, None) == cb.ERR_INVALID_ARG
    assert L.cascade_drafter_loss(p, p, p, 1, 4, 4, 0.5, 0.0, p, None, None, None) == cb.ERR_INVALID_ARG
    # a target row truncated by top-k (-inf logits): those tokens carry no weight even where the drafter is -inf too
    tl = np.array([[0.0, 1.0, -np.inf, -np.inf]], np.float32)
    dl = np.array([[0.5, 0.2, -np.inf, 3.0]], np.float32)
    feat = np.ones((1, 4), np.float32)
    loss = torch.zeros(1, device=G.DEV)
    cb.cascade_drafter_loss(torch.from_numpy(tl).to(G.DEV), torch.from_numpy(dl).to(G.DEV), torch.from_numpy(feat).to(G.DEV),
                            0.5, 2.0, loss)
    torch.cuda.synchronize()
    q = np.exp([0.0, 1.0]) / np.exp([0.0, 1.0]).sum()
    logp = np.array([0.5, 0.2]) - np.log(np.exp(0.5) + np.exp(0.2) + np.exp(3.0))
    assert abs(float(loss) + (q * logp).sum()) < 1e-5
