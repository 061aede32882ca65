"""Pins for the checker's drafter loss (Section 4.3, Eq. 4)."""
import numpy as np
import torch
from scipy.special import rel_entr
from scipy.stats import entropy

from oracle import cascade_oracle as O


def _case(seed, K=9, V=37, h=12):
    rng = np.random.default_rng(seed)
    return rng.normal(0, 2, (K, V)), rng.normal(0, 2, (K, V)), rng.standard_normal((K, h))


def test_unweighted_loss_is_the_library_soft_cross_entropy():
    tl, dl, feat = _case(1)
    per, w, total = O.drafter_loss(tl, dl, feat, tau_seq=2.0, c=7.0)          # no cosine reaches 2: every weight 1
    assert np.array_equal(w, np.ones(len(tl)))
    want = torch.nn.functional.cross_entropy(torch.from_numpy(dl), torch.softmax(torch.from_numpy(tl), -1),
                                             reduction="none").numpy()         # class-probability targets
    assert np.allclose(per, want, atol=1e-12) and abs(total - want.sum()) < 1e-10
    # soft cross-entropy = KL(q || p) + H(q)
    q, p = O.softmax(tl), O.softmax(dl)
    assert np.allclose(per, rel_entr(q, p).sum(-1) + entropy(q, axis=-1), atol=1e-12)
    # a drafter that equals the target leaves the target's entropy
    per_same, _, _ = O.drafter_loss(tl, tl, feat, 2.0, 7.0)
    assert np.allclose(per_same, entropy(q, axis=-1), atol=1e-12)


def test_weights_follow_the_convergence_of_consecutive_positions():
    tl, dl, _ = _case(2, K=6, h=4)
    e = np.eye(4)
    # positions 0,1 identical (cos 1), 1->2 orthogonal (0), 2->3 at 45 degrees (0.7071), 3->4 opposite (-1), 4->5 identical
    feat = np.stack([e[0], e[0], e[1], (e[1] + e[2]), -(e[1] + e[2]), -3.0 * (e[1] + e[2])])
    per1, w1, t1 = O.drafter_loss(tl, dl, feat, 2.0, 2.0)
    per, w, total = O.drafter_loss(tl, dl, feat, 0.7, 2.0)
    assert w.tolist() == [2.0, 1.0, 2.0, 1.0, 2.0, 1.0]                      # the last position has no successor
    assert np.allclose(per, w * per1) and abs(total - (w * per1).sum()) < 1e-12
    assert O.drafter_loss(tl, dl, feat, 0.7072, 2.0)[1].tolist() == [2.0, 1.0, 1.0, 1.0, 2.0, 1.0]   # >= tau, as in Eq. 2
    assert O.drafter_loss(tl, dl, feat, 0.7, 1.0)[2] == t1                   # c = 1 switches the re-weighting off
    # the weight depends on directions only
    assert O.drafter_loss(tl, dl, 5.0 * feat, 0.7, 2.0)[1].tolist() == w.tolist()
