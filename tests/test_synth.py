"""Host-side checks of the seeded input generators."""
import numpy as np
import pytest

from paper_2605_07230_b200 import synth


def test_bf16_round_trip_and_ties():
    x = np.array([1.0, 1.0 + 2**-8, 1.0 + 2**-7, 1.0 + 3 * 2**-8, -2.5, 0.0, 3.14159], np.float32)
    r = synth.round_to_bf16(x)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: goes to the even mantissa (1.0)
    assert r[1] == 1.0 and r[2] == 1.0 + 2**-7
    # 1 + 3*2^-8 is a tie between 1+2^-7 (odd) and 1+2^-6 (even)
    assert r[3] == 1.0 + 2**-6
    assert np.all(np.abs(r - x) <= np.abs(x) * 2**-8)
    assert np.array_equal(synth.round_to_bf16(r), r)


def test_bf16_matches_torch():
    torch = pytest.importorskip("torch")
    x = np.random.default_rng(0).standard_normal(4096).astype(np.float32)
    ours = synth.round_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours, ref)


def test_toy_tree_is_complete_binary():
    p = synth.complete_tree(2, 3)
    assert len(p) == 15 and synth.level_widths(p) == [2, 4, 8]


@pytest.mark.parametrize("n", [16, 32, 60, 64, 128])
def test_static_tree_is_bfs_and_reaches_depth_6(n):
    p = synth.static_topk_tree(n)
    assert len(p) == n + 1 and p[0] == -1
    d = synth.tree_depth(p)
    assert d.max() == 6
    assert np.all(np.diff(d) >= 0)            # BFS order
    assert np.all(np.diff(p[1:]) >= 0)        # siblings contiguous, groups in parent order
    assert np.all(p[1:] < np.arange(1, n + 1))
    kids = np.bincount(p[1:], minlength=n + 1)
    branching = (4, 3, 2, 2, 1, 1)
    for j in range(n + 1):
        if d[j] < 6:
            assert kids[j] <= branching[d[j]]


def test_static_tree_60_level_widths():
    assert synth.level_widths(synth.static_topk_tree(60)) == [4, 8, 9, 13, 13, 13]


def test_cluster_drafter_is_seeded_and_distinct():
    p = synth.static_topk_tree(32)
    a = synth.cluster_drafter(np.random.default_rng(5), p, 2, 2048, 64)
    b = synth.cluster_drafter(np.random.default_rng(5), p, 2, 2048, 64)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    tok, prob = a
    assert prob.min() > 0 and prob.max() <= 1
    for bi in range(2):
        for j in range(len(p)):
            kids = np.nonzero(p == j)[0]
            assert len(set(tok[bi, kids].tolist())) == len(kids)   # drawn without replacement
            assert np.all(np.diff(prob[bi, kids]) <= 0)            # best first
