"""Helpers shared by the GPU parity tests: move seeded host inputs to the device in the workload's
element type, call the library through the binding, and compare decisions while setting aside
near-threshold cases."""
from __future__ import annotations

import numpy as np
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import binding as cb
from paper_2605_07230_b200 import synth

DEV = "cuda:0"


quantize = synth.quantize


def to_dev(x: np.ndarray, dtype: str) -> torch.Tensor:
    """Exact transfer: x must already be representable in `dtype`."""
    t = torch.from_numpy(np.ascontiguousarray(x, np.float32))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
        assert torch.equal(t.to(torch.float32), torch.from_numpy(np.ascontiguousarray(x, np.float32)))
    return t.to(DEV).contiguous()


def make_ctx(w: synth.Workload, T: int, ffn: int = 0, P_max: int | None = None) -> cb.Context:
    return cb.Context(cb.BF16 if w.dtype == "bf16" else cb.F32, w.B, T, P_max or w.prefix_len, w.h, w.n_heads,
                      w.n_heads, w.head_dim, w.V, ffn)


def attention_inputs(w, rng, T, prefix_len=None):
    d = synth.attention_inputs(w, rng, T)
    plen = d["prefix_len"] if prefix_len is None else np.asarray(prefix_len, np.int32)
    return d["q"], d["k_prefix"], d["v_prefix"], d["k_tree"], d["v_tree"], plen


def tail_inputs(w, rng, parent, noise: float = 0.15):
    d = synth.tail_inputs(w, rng, parent, noise)
    return d["w_head"], d["hidden"], d["gamma_final"], d["tok"], d["draft_p"], d["uniforms"]


def compare_decisions(parent, oracle_rows, accept_gpu, path_nodes_gpu, path_len_gpu, mode, min_node_frac=0.5):
    """Bit-exact comparison of accept masks and paths, setting aside near-threshold cases.

    oracle_rows: per prompt, the checker's result dict (computed from the SAME features/logits the
    device used).  A cosine or budget comparison inside the near band at node x may legitimately go the
    other way on the device; that can change x's own relaxed probability and the running total handed on
    from x, i.e. to x's later siblings and to every descendant of x and of those siblings.  Exactly these
    nodes are set aside; a node whose accept test is inside the band is set aside alone.  All other nodes
    must match bit for bit.  The path is compared when nothing of the prompt was set aside.  Fails if
    fewer than `min_node_frac` of all nodes could be compared.  Returns counts.
    """
    stats = {"prompts": 0, "prompts_set_aside": 0, "nodes": 0, "nodes_compared": 0, "nodes_set_aside": 0,
             "paths_compared": 0}
    T = len(parent)
    for b, res in enumerate(oracle_rows):
        stats["prompts"] += 1
        near = res["near"]
        unstable = np.zeros(T, bool)
        for x in range(1, T):
            if near[x] & 3:
                unstable[x] = True
                for y in range(x + 1, T):          # later siblings follow x in index order
                    if parent[y] == parent[x]:
                        unstable[y] = True
        for y in range(1, T):                      # BFS order: a parent is final before its children
            if unstable[parent[y]]:
                unstable[y] = True
        aside = unstable | ((near & 4) != 0)
        if unstable.any():
            stats["prompts_set_aside"] += 1
        stats["nodes"] += T
        stats["nodes_set_aside"] += int(aside.sum())
        stats["nodes_compared"] += int((~aside).sum())
        got = accept_gpu[b]
        assert np.array_equal(got[~aside], res["accept"][~aside]), f"accept mask differs for prompt {b}"
        if not aside.any():
            path, alpha, _ = O.select_path(res["accept"], parent, res["tvd_out"], mode)
            assert path_len_gpu[b] == alpha, f"alpha differs for prompt {b}"
            assert path_nodes_gpu[b][: alpha + 1].tolist() == path
            assert np.all(path_nodes_gpu[b][alpha + 1:] == -1)
            stats["paths_compared"] += 1
        else:
            # whatever the device decided on the nodes set aside, its path must follow from its own accept bits
            path, alpha, _ = O.select_path(got, parent, None, mode)
            assert path_len_gpu[b] == alpha and path_nodes_gpu[b][: alpha + 1].tolist() == path
    assert stats["nodes_compared"] >= min_node_frac * stats["nodes"], stats
    return stats


def target_sampled_drafts(w, host, parent, rng, temperature=1.5):
    """Draft tokens drawn level by level from the TARGET's own softened distribution (the toy workload's
    definition): children of node j are sampled without replacement from softmax(logits[j] / temperature),
    best first, with that softened probability as the drafter's p.  Needs the checker's forward pass once
    per level (a row's logits depend only on the tokens of its ancestors), so it is only for small cases."""
    T = len(parent)
    kids = O.children_of(parent)
    depth = O.tree_depth(parent)
    tok = host["tok"].copy()
    p = np.ones_like(host["draft_p"])
    for level in range(int(depth.max())):
        out = O.verify_step(host["embed"], host["layers"], host["gamma_final"], host["w_head"], tok, parent,
                            host["k_prefix"], host["v_prefix"], host["prefix_len"], p, host["uniforms"], w.n_heads,
                            w.head_dim, w.eps, w.rope_base, w.cfg_scale, 1.0, w.tau_pos, w.tau_seq, w.tvd_budget,
                            kv_bf16=w.dtype == "bf16")
        logits = out["head"]["logits"]
        for b in range(w.B):
            for j in range(T):
                if depth[j] != level or not kids[j]:
                    continue
                soft = O.softmax(logits[b, j] / temperature)
                g = np.log(np.maximum(soft, 1e-300)) - np.log(-np.log(rng.random(len(soft))))
                pick = np.argsort(-g)[: len(kids[j])]
                pick = pick[np.argsort(-soft[pick], kind="stable")]
                for kid, t in zip(kids[j], pick):
                    tok[b, kid] = t
                    p[b, kid] = soft[t]
    return tok.astype(np.int32), p.astype(np.float32)
