"""Pins of the checker's top-k / top-p truncation of the target distribution (Appendix D.1 settings)."""
import numpy as np
import torch

from oracle import cascade_oracle as O


def rows(seed, n=5, V=97, ties=False):
    rng = np.random.default_rng(seed)
    l = rng.normal(0.0, 2.0, (n, V))
    if ties:
        l = np.round(l * 2) / 2        # many equal logits
    return l


def test_no_truncation_is_identity():
    l = rows(0)
    for k, p in ((0, 1.0), (97, 1.0), (1000, 1.0)):
        f, kept = O.filter_logits(l, k, p)
        assert kept.all() and np.array_equal(f, l)


def test_top_k_matches_the_library_routine():
    l = rows(1, n=8, V=257)
    for k in (1, 2, 17, 100, 256):
        f, kept = O.filter_logits(l, k, 1.0)
        thr = torch.topk(torch.from_numpy(l), k, dim=-1).values[:, -1].numpy()   # library step: k-th largest
        assert np.array_equal(kept, l >= thr[:, None])
        assert (kept.sum(-1) == k).all()                                          # no ties in continuous draws
        assert np.array_equal(f[kept], l[kept]) and np.isneginf(f[~kept]).all()


def test_top_k_one_is_the_argmax_with_probability_one():
    l = rows(2)
    f, kept = O.filter_logits(l, 1, 1.0)
    assert np.array_equal(kept.argmax(-1), l.argmax(-1)) and (kept.sum(-1) == 1).all()
    assert np.allclose(O.softmax(f).max(-1), 1.0)


def test_ties_stay_together():
    l = rows(3, ties=True)
    f, kept = O.filter_logits(l, 5, 1.0)
    for r in range(l.shape[0]):
        kth = np.sort(l[r])[-5]
        assert kept[r].sum() == (l[r] >= kth).sum() >= 5
    f, kept = O.filter_logits(l, 0, 0.3)
    for r in range(l.shape[0]):
        for v in np.unique(l[r]):
            assert len(set(kept[r][l[r] == v])) == 1     # equal logits share their fate


def brute_force_nucleus(row, top_p):
    """Add tokens from the most likely down, a whole group of equal logits at a time, until the mass that
    was already in reaches top_p."""
    p = np.exp(row - row.max())
    p /= p.sum()
    keep = np.zeros(len(row), bool)
    mass = 0.0
    for v in sorted(set(row), reverse=True):
        if mass >= top_p:
            break
        grp = row == v
        keep |= grp
        mass += p[grp].sum()
    return keep


def test_top_p_matches_brute_force():
    for ties in (False, True):
        l = rows(4, n=6, V=61, ties=ties)
        for p in (0.05, 0.3, 0.5, 0.9, 0.999):
            _, kept = O.filter_logits(l, 0, p)
            for r in range(l.shape[0]):
                assert np.array_equal(kept[r], brute_force_nucleus(l[r], p)), (ties, p, r)


def test_top_p_is_minimal_and_sufficient():
    l = rows(5, n=6, V=128)
    for p in (0.2, 0.6, 0.95):
        _, kept = O.filter_logits(l, 0, p)
        probs = O.softmax(l)
        for r in range(l.shape[0]):
            mass = probs[r][kept[r]].sum()
            assert mass >= p - 1e-12
            smallest = np.where(kept[r], l[r], np.inf).argmin()
            assert mass - probs[r][smallest] < p            # dropping the least likely kept token falls short
            assert l[r][kept[r]].min() >= l[r][~kept[r]].max() if (~kept[r]).any() else True   # upward closed


def test_top_p_applies_to_the_top_k_renormalised_distribution():
    l = rows(6, n=4, V=64)
    k, p = 8, 0.7
    _, kept = O.filter_logits(l, k, p)
    for r in range(l.shape[0]):
        idx = np.argsort(-l[r])[:k]
        q = np.exp(l[r][idx] - l[r][idx].max())
        q /= q.sum()
        n_keep = int(np.searchsorted(np.cumsum(q), p, side="left")) + 1   # first prefix whose mass reaches p
        assert set(np.nonzero(kept[r])[0]) == set(idx[:n_keep])


def test_monotone_in_k_and_p():
    l = rows(7, n=3, V=200)
    prev = None
    for k in (1, 5, 50, 199):
        _, kept = O.filter_logits(l, k, 1.0)
        if prev is not None:
            assert (kept | ~prev).all()
        prev = kept
    prev = None
    for p in (0.1, 0.5, 0.9):
        _, kept = O.filter_logits(l, 0, p)
        if prev is not None:
            assert (kept | ~prev).all()
        prev = kept


def test_filtered_rows_feed_the_acceptance_rule():
    """A dropped token has target mass zero: with the relaxation off its draft is rejected, a kept token's
    mass is its renormalised probability."""
    rng = np.random.default_rng(8)
    V, h = 50, 16
    parent = np.array([-1, 0, 0])
    feat = rng.normal(size=(3, h))
    logits = rng.normal(0, 2, (3, V))
    f, kept = O.filter_logits(logits, 5, 1.0)
    top = int(np.argmax(logits[0])); low = int(np.argmin(logits[0]))
    tok = np.array([0, top, low])
    r = O.relaxed_accept(feat, f, tok, parent, np.array([1.0, 0.5, 0.5]), np.array([0.0, 0.0, 0.0]), 2.0, 2.0, 0.5)
    assert np.isclose(r["q_plain"][1], O.softmax(f[0])[top]) and r["q_plain"][2] == 0.0
    assert r["accept"][1] == 1 and r["accept"][2] == 0


def test_hand_computed_row():
    """softmax([2, 1, 0, -1]) = [0.6439, 0.2369, 0.0871, 0.0321] (e^2 : e : 1 : 1/e over their sum 11.4752)."""
    l = np.array([[2.0, 1.0, 0.0, -1.0]])
    z = np.exp(2) + np.exp(1) + 1 + np.exp(-1)
    p = np.array([np.exp(2), np.exp(1), 1.0, np.exp(-1)]) / z
    assert np.allclose(p, [0.6439, 0.2369, 0.0871, 0.0321], atol=5e-5)
    cases = {
        (2, 1.0): [1, 1, 0, 0],       # the two largest
        (0, 0.6): [1, 0, 0, 0],       # 0.6439 alone reaches 0.6
        (0, 0.7): [1, 1, 0, 0],       # 0.6439 < 0.7 <= 0.8808
        (0, 0.9): [1, 1, 1, 0],       # 0.8808 < 0.9 <= 0.9679
        (3, 0.7): [1, 1, 0, 0],       # renormalised over three: 0.6652, 0.2447, 0.0900 -> 0.6652 < 0.7 <= 0.9100
        (2, 0.72): [1, 0, 0, 0],      # renormalised over two: 0.7311 reaches 0.72 alone
    }
    for (k, top_p), want in cases.items():
        f, kept = O.filter_logits(l, k, top_p)
        assert kept[0].astype(int).tolist() == want, (k, top_p)
        assert np.isneginf(f[0][~kept[0]]).all()
