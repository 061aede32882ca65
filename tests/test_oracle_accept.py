"""Pins for the CPU checker's relaxed acceptance (Eq. 1-3, Algorithm 2) and path selection."""
import itertools
import json
import os

import numpy as np
import pytest
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))


def make_case(seed, T=15, V=40, h=12, n_protos=3, noise=0.35, tree=None):
    """Random prompt whose features cluster around a few prototypes, so both sets fire often."""
    rng = np.random.default_rng(seed)
    parent = synth.random_tree(rng, T) if tree is None else tree
    T = len(parent)
    protos = rng.standard_normal((n_protos, h))
    feat = protos[rng.integers(0, n_protos, T)] + noise * rng.standard_normal((T, h))
    logits = rng.standard_normal((T, V)) * 2.0
    tok = np.zeros(T, np.int64)
    for j in range(T):
        kids = np.nonzero(parent == j)[0]
        # a few duplicated ids across levels on purpose; siblings distinct
        tok[kids] = rng.choice(V // 4, size=len(kids), replace=False)
    draft_p = rng.uniform(0.02, 0.6, T)
    u = rng.random(T)
    return parent, feat, logits, tok, draft_p, u


# --------------------------------------------------------------------------------------------
# an independently written sequential walk of Algorithm 2 (torch for softmax / cosine)
# --------------------------------------------------------------------------------------------

def algorithm2_walk(parent, feat, logits, tok, draft_p, u, tau_pos, tau_seq, eps_tvd):
    feat_t = torch.from_numpy(np.asarray(feat, np.float64))
    cos = lambda a, b: float(torch.nn.functional.cosine_similarity(feat_t[a], feat_t[b], dim=0, eps=0.0))
    alpha, curr_tvd, node = 0, 0.0, 0
    visited = {}
    while True:
        level = [c for c in range(len(parent)) if parent[c] == node]     # active sequences
        if not level:
            break
        gtp = torch.softmax(torch.from_numpy(np.asarray(logits[node], np.float64)), 0).numpy()
        taken = None
        for x in level:
            q_x = gtp[tok[x]]
            others = [b for b in level if b != x and cos(x, b) >= tau_pos]
            nxt = [c for c in range(len(parent)) if parent[c] == x and cos(x, c) >= tau_seq]
            ids_i = set(int(tok[b]) for b in others) - {int(tok[x])}
            ids_c = set(int(tok[c]) for c in nxt) - {int(tok[x])} - ids_i
            if others:
                m = sum(gtp[i] for i in sorted(ids_i))
                if curr_tvd + m <= eps_tvd:
                    q_x += m
                    curr_tvd += m
            if nxt:
                m = sum(gtp[i] for i in sorted(ids_c))
                if curr_tvd + m <= eps_tvd:
                    q_x += m
                    curr_tvd += m
            visited[x] = (q_x, curr_tvd)
            if u[x] < min(1.0, q_x / draft_p[x]):
                taken = x
                alpha += 1
                break
        if taken is None:
            break
        node = taken
    return alpha, node, curr_tvd, visited


@pytest.mark.parametrize("seed", range(40))
def test_tree_threaded_budget_equals_sequential_walk(seed):
    budget = 0.5 if seed % 2 else 0.1
    parent, feat, logits, tok, p, u = make_case(seed)
    tau_pos, tau_seq = 0.8, 0.6
    res = O.relaxed_accept(feat, logits, tok, parent, p, u, tau_pos, tau_seq, budget)
    path, alpha, tvd_used = O.select_path(res["accept"], parent, res["tvd_out"], O.SELECT_FIRST_ACCEPT)
    w_alpha, w_end, w_tvd, visited = algorithm2_walk(parent, feat, logits, tok, p, u, tau_pos, tau_seq, budget)
    assert alpha == w_alpha and path[-1] == w_end
    assert abs(tvd_used - w_tvd) < 1e-12
    # every node the walk visited got the walk's relaxed probability and budget state
    for x, (q_x, t_x) in visited.items():
        assert abs(res["q_relaxed"][x] - q_x) < 1e-12
        assert abs(res["tvd_out"][x] - t_x) < 1e-12


def test_sets_actually_fire_in_these_cases():
    fired_i = fired_c = skipped = 0
    for seed in range(40):
        parent, feat, logits, tok, p, u = make_case(seed)
        res = O.relaxed_accept(feat, logits, tok, parent, p, u, 0.8, 0.6, 0.5)
        fired_i += int((res["size_i"] > 0).sum())
        fired_c += int((res["size_c"] > 0).sum())
        tight = O.relaxed_accept(feat, logits, tok, parent, p, u, 0.8, 0.6, 0.1)
        skipped += int(((tight["size_i"] + tight["size_c"] > 0) & (tight["q_relaxed"] == tight["q_plain"])).sum())
    assert fired_i > 50 and fired_c > 50 and skipped > 10   # budget refusals are exercised too


# --------------------------------------------------------------------------------------------
# relaxation off -> Algorithm 1's test at every node
# --------------------------------------------------------------------------------------------

@pytest.mark.parametrize("how", ["thresholds", "flags", "budget"])
def test_relaxation_off_is_standard_acceptance(how):
    for seed in range(10):
        parent, feat, logits, tok, p, u = make_case(100 + seed)
        if how == "thresholds":
            res = O.relaxed_accept(feat, logits, tok, parent, p, u, 1.5, 1.5, 0.5)
        elif how == "flags":
            res = O.relaxed_accept(feat, logits, tok, parent, p, u, 0.0, 0.0, 0.5, flags=0)
        else:
            # a zero budget admits only zero mass: thresholds at -1 put every pair in the sets
            res = O.relaxed_accept(feat, logits, tok, parent, p, u, -1.0, -1.0, 0.0)
        for j in range(1, len(parent)):
            q = torch.softmax(torch.from_numpy(logits[parent[j]]), 0)[tok[j]].item()
            assert abs(res["q_relaxed"][j] - q) < 1e-15 + (how == "budget") * 1e-12
            assert res["accept"][j] == (u[j] < min(1.0, q / p[j]))
        if how != "budget":
            assert np.all(res["tvd_out"] == 0)


def test_chain_with_relaxation_off_is_algorithm1_prefix_rule():
    rng = np.random.default_rng(7)
    K, V = 8, 30
    parent = synth.chain_tree(K)
    for trial in range(20):
        logits = rng.standard_normal((K + 1, V))
        tok = rng.integers(0, V, K + 1)
        p = rng.uniform(0.01, 0.3, K + 1)
        u = rng.random(K + 1)
        feat = rng.standard_normal((K + 1, 5))
        res = O.relaxed_accept(feat, logits, tok, parent, p, u, 2.0, 2.0, 0.5)
        _, alpha, _ = O.select_path(res["accept"], parent, res["tvd_out"])
        # Algorithm 1: accept draft tokens in order until the first failure
        n = 0
        for t in range(1, K + 1):
            q = np.exp(logits[t - 1, tok[t]]) / np.exp(logits[t - 1]).sum()
            if u[t] < min(1.0, q / p[t]):
                n += 1
            else:
                break
        assert alpha == n


# --------------------------------------------------------------------------------------------
# invariants and closed forms
# --------------------------------------------------------------------------------------------

def test_bounds_and_budget_invariants():
    for seed in range(30):
        parent, feat, logits, tok, p, u = make_case(200 + seed)
        for budget in [0.05, 0.5, 10.0]:
            r = O.relaxed_accept(feat, logits, tok, parent, p, u, 0.7, 0.5, budget)
            assert np.all(r["q_relaxed"] >= r["q_plain"])
            assert np.all(r["q_relaxed"] <= 1 + 1e-12)          # distinct tokens under one distribution
            assert np.all(r["tvd_out"] <= budget + 1e-15)
            kids = O.children_of(parent)
            for j in range(len(parent)):
                t = r["tvd_out"][j]
                for c in kids[j]:                                 # non-decreasing along the threading
                    assert r["tvd_out"][c] >= t
                    t = r["tvd_out"][c]
            # the charge equals the mass added
            for j in range(len(parent)):
                start = r["tvd_out"][j]
                for c in kids[j]:
                    assert abs((r["tvd_out"][c] - start) - (r["q_relaxed"][c] - r["q_plain"][c])) < 1e-12
                    start = r["tvd_out"][c]


def test_identical_sibling_features_pool_all_sibling_mass():
    parent = np.array([-1, 0, 0, 0, 0])
    feat = np.tile(np.array([[0.3, -1.0, 2.0]]), (5, 1))
    feat[0] = [1, 0, 0]
    g = np.array([0.05, 0.1, 0.15, 0.2, 0.5])
    tok = np.array([4, 0, 1, 2, 3])
    r = O.relaxed_accept(feat, np.log(g)[None].repeat(5, 0), tok, parent, np.full(5, 0.5), np.full(5, 0.4),
                         0.999, 2.0, 10.0)
    assert np.allclose(r["q_relaxed"][1:], 0.5)                  # .05+.1+.15+.2
    assert r["size_i"][1:].tolist() == [3, 3, 3, 3]
    assert np.allclose(r["tvd_out"][1:], np.cumsum(0.5 - g[:4]))


def test_duplicate_tokens_are_counted_once_and_own_token_never():
    parent = np.array([-1, 0, 0, 1, 1, 1])
    feat = np.ones((6, 4))
    g0 = np.array([0.4, 0.3, 0.2, 0.1])
    tok = np.array([0, 1, 2, 1, 2, 2])     # children of node 1 repeat tok_1, tok_2 and each other
    logits = np.log(g0)[None].repeat(6, 0)
    r = O.relaxed_accept(feat, logits, tok, parent, np.full(6, 0.5), np.full(6, 0.9), 0.9, 0.9, 10.0)
    # node 1: q=.3; I={2}->{2}: .2; C={3,4,5} tokens {1,2,2} minus own {1} minus I's {2} -> nothing
    assert abs(r["q_relaxed"][1] - 0.5) < 1e-12 and r["size_c"][1] == 3


def test_drafter_equal_to_target_accepts_everything():
    for seed in range(5):
        parent, feat, logits, tok, _, u = make_case(300 + seed)
        q = np.array([0.0] + [O.softmax(logits[parent[j]])[tok[j]] for j in range(1, len(parent))])
        q[0] = 1.0
        r = O.relaxed_accept(feat, logits, tok, parent, q, u, 0.8, 0.6, 0.5)
        assert r["accept"].all()
        path, alpha, _ = O.select_path(r["accept"], parent, r["tvd_out"])
        assert alpha == synth.tree_depth(parent).max()


def test_zero_drafter_probability_rejects():
    parent, feat, logits, tok, p, u = make_case(5)
    p[3] = 0.0
    assert O.relaxed_accept(feat, logits, tok, parent, p, u, 0.8, 0.6, 0.5)["accept"][3] == 0


@pytest.mark.parametrize("seed", range(15))
def test_accept_set_grows_as_thresholds_drop_when_budget_is_unbounded(seed):
    parent, feat, logits, tok, p, u = make_case(400 + seed)
    taus = [1.1, 0.95, 0.8, 0.6, 0.3, -1.0]
    for ts in taus:
        prev = None
        for tp in taus:
            a = O.relaxed_accept(feat, logits, tok, parent, p, u, tp, ts, np.inf)["accept"].astype(bool)
            if prev is not None:
                assert np.all(a | ~prev)          # 1 stays 1
            prev = a
    for tp in taus:
        prev = None
        for ts in taus:
            a = O.relaxed_accept(feat, logits, tok, parent, p, u, tp, ts, np.inf)["accept"].astype(bool)
            if prev is not None:
                assert np.all(a | ~prev)
            prev = a


def test_finite_budget_is_not_monotone_counter_example():
    """All-or-nothing charging: a looser threshold can grow a set past the budget and lose the mass."""
    parent = np.array([-1, 0, 0, 0])
    feat = np.array([[1, 0], [1, 0], [1, 0.2], [1, 1.0]])        # cos(1,2)=.98, cos(1,3)=.707
    g = np.array([0.1, 0.3, 0.35, 0.25])
    tok = np.array([3, 0, 1, 2])
    args = (feat, np.log(g)[None].repeat(4, 0), tok, parent, np.full(4, 0.9), np.array([0, 0.4, 0.99, 0.99]))
    tight = O.relaxed_accept(*args, 0.9, 2.0, 0.5)                # I_1={2}: +.3 -> .4/.9=.44 > .4 accept
    loose = O.relaxed_accept(*args, 0.7, 2.0, 0.5)                # I_1={2,3}: +.65 > .5 refused -> .1/.9 reject
    assert tight["accept"][1] == 1 and loose["accept"][1] == 0


# --------------------------------------------------------------------------------------------
# path selection
# --------------------------------------------------------------------------------------------

def _all_root_paths(parent):
    T = len(parent)
    for end in range(T):
        path = [end]
        while parent[path[-1]] >= 0:
            path.append(parent[path[-1]])
        yield path[::-1]


@pytest.mark.parametrize("T", [1, 2, 6, 15])
def test_longest_path_by_brute_force(T):
    rng = np.random.default_rng(T)
    for trial in range(200):
        parent = synth.random_tree(rng, T) if T > 1 else np.array([-1])
        if T == 15 and trial % 2:
            parent = synth.complete_tree(2, 3)
        accept = (rng.random(len(parent)) < 0.6).astype(np.uint8)
        accept[0] = 1
        best = max((p for p in _all_root_paths(parent) if all(accept[i] for i in p)),
                   key=lambda p: (len(p), -p[-1]))
        path, alpha, _ = O.select_path(accept, parent)
        assert path == best and alpha == len(best) - 1
        fpath, falpha, _ = O.select_path(accept, parent, mode=O.SELECT_FIRST_ACCEPT)
        assert falpha <= alpha
        assert all(accept[i] for i in fpath) and fpath[0] == 0
        for a, b in zip(fpath, fpath[1:]):
            assert parent[b] == a
            earlier = [c for c in range(len(parent)) if parent[c] == a and c < b]
            assert not any(accept[c] for c in earlier)            # it took the FIRST accepted child
        depth = synth.tree_depth(parent)
        valid = [all(accept[i] for i in p) for p in _all_root_paths(parent)]
        per_level = np.bincount(depth[np.array(valid)], minlength=depth.max() + 1)
        if per_level.max() <= 1:
            assert fpath == path


def test_exhaustive_accept_patterns_on_small_tree():
    parent = np.array([-1, 0, 0, 1, 1, 2, 3])
    for bits in itertools.product([0, 1], repeat=6):
        accept = np.array((1,) + bits, np.uint8)
        best = max((p for p in _all_root_paths(parent) if all(accept[i] for i in p)),
                   key=lambda p: (len(p), -p[-1]))
        assert O.select_path(accept, parent)[0] == best


# --------------------------------------------------------------------------------------------
# hand-worked example
# --------------------------------------------------------------------------------------------

def test_hand_worked_tree():
    with open(os.path.join(HERE, "golden", "hand_tree.json")) as f:
        g = json.load(f)
    e = g["expect"]
    args = (np.array(g["feat"], float), np.log(np.array(g["gtp"])), np.array(g["tok"]), np.array(g["parent"]),
            np.array(g["draft_p"]), np.array(g["u"]), g["tau_pos"], g["tau_seq"], g["tvd_budget"])
    r = O.relaxed_accept(*args)
    assert np.allclose(r["q_plain"], e["q_plain"], atol=1e-12)
    assert np.allclose(r["q_relaxed"], e["q_relaxed"], atol=1e-12)
    assert np.allclose(r["tvd_out"], e["tvd_out"], atol=1e-12)
    assert r["accept"].tolist() == e["accept"]
    assert r["size_i"].tolist() == e["size_i"] and r["size_c"].tolist() == e["size_c"]
    assert r["near"].tolist() == [0] * 6
    for mode in (O.SELECT_LONGEST, O.SELECT_FIRST_ACCEPT):
        path, alpha, tvd_used = O.select_path(r["accept"], np.array(g["parent"]), r["tvd_out"], mode)
        assert path == e["path"] and alpha == e["alpha"] and abs(tvd_used - e["tvd_used"]) < 1e-12
    off = O.relaxed_accept(*args[:6], 2.0, 2.0, g["tvd_budget"])
    assert off["accept"].tolist() == e["accept_without_relaxation"]
    sd = O.relaxed_accept(*args, flags=O.USE_I | O.USE_C | O.CONV_DIST_SELF)
    assert abs(sd["q_relaxed"][2] - e["self_dist"]["q_relaxed_2"]) < 1e-12
    assert abs(sd["tvd_out"][2] - e["self_dist"]["tvd_out_2"]) < 1e-12
    only_i = O.relaxed_accept(*args, flags=O.USE_I)
    assert np.allclose(only_i["q_relaxed"], [0, 0.7, 0.2, 0.7, 0.3, 0.25], atol=1e-12)
    only_c = O.relaxed_accept(*args, flags=O.USE_C)
    # without I, node 1's C-set {3} contributes tok 1 under row 0 (.2); node 2's {5} contributes .1
    assert np.allclose(only_c["q_relaxed"], [0, 0.7, 0.3, 0.4, 0.3, 0.25], atol=1e-12)


def test_cosine_properties():
    rng = np.random.default_rng(0)
    a, b = rng.standard_normal(9), rng.standard_normal(9)
    assert abs(O.cosine(a, a) - 1) < 1e-15
    assert O.cosine(a, b) == O.cosine(b, a)
    assert abs(O.cosine(3.5 * a, 0.01 * b) - O.cosine(a, b)) < 1e-15
    assert abs(O.cosine(a, -a) + 1) < 1e-15 and abs(O.cosine(a, b)) <= 1
    assert abs(O.cosine([1, 0], [1, 1]) - 2 ** -0.5) < 1e-15
    assert abs(O.cosine([3, 4], [4, -3])) < 1e-15
    cs, cc = O.similarity_scores(np.array([[1.0, 0], [1, 0], [0, 2], [1, 1]]), np.array([-1, 0, 0, 1]))
    assert set(cs) == {(1, 2), (2, 1)} and set(cc) == {(0, 1), (0, 2), (1, 3)}
    assert cs[(1, 2)] == 0 and abs(cc[(1, 3)] - 2 ** -0.5) < 1e-15


# ---- bonus token (Algorithm 1's final draw) and cache append ---------------------------------------


def test_bonus_token_is_the_inverse_cdf_sample_of_the_renormalised_target():
    rng = np.random.default_rng(3)
    logits = rng.normal(0, 2, 50)
    g = np.exp(logits - logits.max())
    g /= g.sum()
    # nothing rejected: plain inverse CDF, checked against a brute-force scan
    for u in [0.0, 0.1, 0.5, 0.999999]:
        tok, total = O.bonus_token(logits, [], u)
        acc, want = 0.0, None
        for v in range(50):
            acc += g[v]
            if acc > u:
                want = v
                break
        assert tok == want and abs(total - 1.0) < 1e-12
    # rejected tokens can never come back, and the rest keeps its proportions
    rejected = [int(np.argmax(g)), 7, 7]
    counts = np.zeros(50)
    us = (np.arange(20000) + 0.5) / 20000
    for u in us:
        tok, total = O.bonus_token(logits, rejected, u)
        counts[tok] += 1
    assert counts[rejected[0]] == 0 and counts[7] == 0
    rest = g.copy()
    rest[rejected] = 0
    assert abs(total - rest.sum()) < 1e-12
    assert np.abs(counts / len(us) - rest / rest.sum()).max() < 2e-4


def test_append_path_kv_writes_the_path_rows_in_order_to_both_cfg_rows():
    B, cap, H, D, T = 2, 12, 1, 2, 5
    k = np.zeros((2 * B, cap, H, D))
    v = np.zeros((2 * B, cap, H, D))
    kt = np.arange(2 * B * T * H * D, dtype=float).reshape(2 * B, T, H, D)
    vt = -kt
    plen = np.array([3, 4, 5, 6])
    new = O.append_path_kv(k, v, plen, kt, vt, [[0, 2, 4], [0]], B)
    assert new.tolist() == [6, 5, 8, 7]
    assert np.array_equal(k[0, 3:6], kt[0, [0, 2, 4]]) and np.array_equal(k[2, 5:8], kt[2, [0, 2, 4]])
    assert np.array_equal(v[1, 4:5], vt[1, [0]]) and np.array_equal(v[3, 6:7], vt[3, [0]])
    assert k[0, 6:].sum() == 0 and k[1, 5:].sum() == 0


# ---- Algorithm 1's correction step: [q - p]+ -------------------------------------------------------------------


def _draw_intervals(fn, n_grid=200001):
    """Lebesgue measure of {u in [0,1) : fn(u) == v} for every v, for a non-decreasing step function fn, found by
    bisection on its jump points (no sampling): returns {v: measure}."""
    out = {}
    lo = 0.0
    v_lo = fn(lo)
    while True:
        hi = 1.0 - 2 ** -53
        if fn(hi) == v_lo:
            out[v_lo] = out.get(v_lo, 0.0) + 1.0 - lo
            return out
        a, b = lo, hi                        # fn(a) == v_lo, fn(b) != v_lo
        for _ in range(80):
            mid = 0.5 * (a + b)
            if fn(mid) == v_lo:
                a = mid
            else:
                b = mid
        out[v_lo] = out.get(v_lo, 0.0) + b - lo
        lo, v_lo = b, fn(b)


def test_accept_test_plus_residual_draw_reproduces_the_target_distribution():
    """The property Section 3 states for Algorithm 1: the emitted token is a sample of the target distribution.
    One draft position, vocabulary of 7, every quantity exact: the draft x is accepted on the set of u with
    u < min(1, q(x)/p(x)) (measured on the checker's own accept test with the relaxation off), otherwise the
    token comes from the residual draw, whose inverse-CDF map is measured interval by interval.
    sum_x p(x) [ acc(x) delta_x + (1 - acc(x)) res(.) ]  must equal q."""
    rng = np.random.default_rng(17)
    V = 7
    for trial in range(5):
        logits = rng.normal(0, 1.5, V)
        q = O.softmax(logits)
        p = rng.dirichlet(np.ones(V) * 0.7)
        if trial == 4:
            p[2] = 0.0                       # a token the drafter never proposes
            p /= p.sum()
        res = _draw_intervals(lambda u: O.residual_token(logits, p, True, u)[0])
        res = np.array([res.get(v, 0.0) for v in range(V)])
        want_res = np.maximum(q - p, 0)
        assert np.allclose(res, want_res / want_res.sum(), atol=1e-12)
        assert abs(O.residual_token(logits, p, True, 0.3)[1] - want_res.sum()) < 1e-15
        emitted = np.zeros(V)
        parent = np.array([-1, 0])
        feat = np.eye(2, 4)
        for x in range(V):
            if p[x] == 0:
                continue
            def accepted(u):
                r = O.relaxed_accept(feat, np.stack([logits, logits]), np.array([0, x]), parent,
                                     np.array([1.0, p[x]]), np.array([0.0, u]), 2.0, 2.0, 0.0, flags=0)
                return int(r["accept"][1])
            m = _draw_intervals(accepted)
            acc = m.get(1, 0.0)
            assert abs(acc - min(1.0, q[x] / p[x])) < 1e-12
            emitted[x] += p[x] * acc
            emitted += p[x] * (1 - acc) * res
        assert np.allclose(emitted, q, atol=1e-11)


def test_residual_draw_special_cases():
    logits = np.log(np.array([0.1, 0.2, 0.3, 0.4]))
    q = O.softmax(logits)
    # nothing rejected: the target row itself, whatever the drafter's row says
    for u, want in ((0.0, 0), (0.0999, 0), (0.1001, 1), (0.2999, 1), (0.3001, 2), (0.61, 3), (0.999999, 3)):
        assert O.residual_token(logits, np.array([1.0, 0, 0, 0]), False, u) == (want, 1.0)
    # drafter = target: nothing lies above p, the target row is used
    assert O.residual_token(logits, q, True, 0.65)[0] == 3
    # p takes all of token 3 and more: only tokens where q > p remain, in proportion to the excess
    p = np.array([0.05, 0.05, 0.1, 0.8])
    r = np.array([0.05, 0.15, 0.2, 0.0])
    tok, total = O.residual_token(logits, p, True, 0.51)
    assert abs(total - r.sum()) < 1e-15 and tok == 2            # cdf 0.125, 0.5, 1.0
    assert O.residual_token(logits, p, True, 0.49)[0] == 1 and O.residual_token(logits, p, True, 0.12)[0] == 0
    assert O.residual_token(logits, p, True, 0.999999)[0] == 2  # token 3 has no residual mass
