"""GPU parity of piece (a) in bf16: split-KV tree attention on tcgen05 against the dense masked softmax."""
import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

ATTN_TOL = 2e-2     # max-abs bound on attention outputs against the fp64 checker


def run_attention(w, parent, seed, prefix_len=None, hkv=None, tail_garbage=False, scale=None):
    T = len(parent)
    rng = np.random.default_rng(seed)
    R, H, D, P = 2 * w.B, w.n_heads, w.head_dim, w.prefix_len
    hkv = hkv or H
    ctx = cb.Context(cb.BF16, w.B, T, P, w.h, H, hkv, D, w.V, 0)
    tree = cb.Tree(ctx, parent)
    q = G.quantize(rng.standard_normal((R, T, H, D), dtype=np.float32), "bf16")
    kp, vp = (G.quantize(rng.standard_normal((R, P, hkv, D), dtype=np.float32), "bf16") for _ in range(2))
    kt, vt = (G.quantize(rng.standard_normal((R, T, hkv, D), dtype=np.float32), "bf16") for _ in range(2))
    plen = np.full(R, P, np.int32) if prefix_len is None else np.asarray(prefix_len, np.int32)
    if tail_garbage:                       # cache rows past prefix_len hold large finite junk
        for r in range(R):
            kp[r, plen[r]:] = 32768.0
            vp[r, plen[r]:] = -8192.0
    out = torch.full((R, T, H, D), float("nan"), dtype=torch.bfloat16, device=G.DEV)
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    cb.cascade_tree_attn(ctx, tree, G.to_dev(q, "bf16"), G.to_dev(kp, "bf16"), G.to_dev(vp, "bf16"), P,
                         torch.from_numpy(plen).to(G.DEV), G.to_dev(kt, "bf16"), G.to_dev(vt, "bf16"), out, scale)
    torch.cuda.synchronize()
    ctx.check()
    launches = ctx.last_launch_count
    ref = O.tree_attention(q, kp, vp, plen, kt, vt, parent, scale)
    got = out.float().cpu().numpy()
    tree.close()
    ctx.close()
    return got, ref, launches


CASES = [
    # name, overrides, prefix_len per CFG row (None = full)
    ("mini", dict(), None),                                            # P=200: two prefix tiles, ragged
    ("mini", dict(), [200, 137, 128, 1]),                              # different lengths per row
    ("mini", dict(B=1, prefix_len=0), None),                           # no prefix at all
    ("mini", dict(B=1, tree="chain1", prefix_len=64), None),           # two rows
    ("mini", dict(B=1, tree="topk64", prefix_len=1000), None),         # 65 rows: two row blocks, many splits
    ("mini", dict(B=1, tree="topk128", prefix_len=300), None),         # 129 rows: three row blocks, two tree tiles
    ("mini", dict(B=8, tree="topk16", n_heads=8, prefix_len=256), None),  # enough CTAs for a single split
    ("mini", dict(B=1, tree="topk60", prefix_len=384), None),          # 61 rows, whole prefix tiles only: rows 61-63 of the block are padding
    ("mini", dict(B=1, tree="topk63", prefix_len=640), None),          # exactly one full 64-row block
    ("mini", dict(B=1, tree="topk60", prefix_len=2480), None),         # 19 whole prefix tiles and a ragged one, two splits
]


@pytest.mark.parametrize("name,over,plen", CASES)
def test_tree_attention_against_checker(name, over, plen):
    w = synth.workload(name, **over)
    parent = w.parent()
    got, ref, _ = run_attention(w, parent, 21, prefix_len=plen, tail_garbage=plen is not None)
    assert np.isfinite(got).all()
    err = np.abs(got - ref).max()
    assert err < ATTN_TOL, err


@pytest.mark.parametrize("scale", [1e-6, 0.5])
def test_flat_and_peaked_weights(scale):
    """A tiny scale weighs every visible key alike (the output is close to the plain mean of the visible value rows);
    a scale of 0.5 on unit-variance scores of 128 terms makes the weights one-hot-like and the running maximum
    jump between tiles.  Both go through the unmasked whole-tile shortcut on the prefix."""
    w = synth.workload("mini", B=1, prefix_len=384)
    parent = w.parent()
    got, ref, _ = run_attention(w, parent, 24, scale=scale)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() < ATTN_TOL


def test_grouped_query_heads():
    w = synth.workload("mini", B=1, n_heads=8)
    got, ref, _ = run_attention(w, w.parent(), 22, hkv=2)
    assert np.abs(got - ref).max() < ATTN_TOL


def test_attention_is_deterministic_and_rows_ignore_non_ancestors():
    w = synth.workload("mini", B=1)
    parent = w.parent()
    a, _, _ = run_attention(w, parent, 23)
    b, _, _ = run_attention(w, parent, 23)
    assert np.array_equal(a, b)
