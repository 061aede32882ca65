"""Seeded synthetic inputs for the CASCADE tree-verification step.

This module only *makes data*: draft-tree shapes, codebooks, weights, prefix KV caches, a
target-free stand-in drafter, uniforms, and bf16 <-> fp32 bit conversion.  It contains none of the
verification arithmetic (no attention, no LM head, no acceptance rule), so both the CUDA path and the
CPU checker can be fed from it without sharing any of the method's code.

Everything is numpy on the host and a pure function of its arguments (seeded
``numpy.random.Generator``), so the same call gives the same bytes everywhere.

Shapes follow the paper's workloads (Janus-Pro-7B and Lumina-mGPT-7B-768 sized target models, static
EAGLE-1 style draft trees, classifier-free guidance with a cond/uncond pair); the values are random
and stand in for real prompts, weights and drafters, which are not available offline.
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass, field

import numpy as np

# --------------------------------------------------------------------------------------------
# bf16 storage helpers (data formatting only)
# --------------------------------------------------------------------------------------------


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the 16-bit patterns as uint16."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact up-cast of bf16 bit patterns (uint16) to fp32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 array whose every value is exactly representable in bf16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# --------------------------------------------------------------------------------------------
# draft trees
# --------------------------------------------------------------------------------------------


def complete_tree(branching: int, levels: int) -> np.ndarray:
    """parent[] of a complete tree: root (node 0) plus `levels` draft levels, BFS order.

    complete_tree(2, 3) is the 15-row toy tree (1 + 2 + 4 + 8).
    """
    parent = [-1]
    frontier = [0]
    for _ in range(levels):
        nxt = []
        for p in frontier:
            for _ in range(branching):
                parent.append(p)
                nxt.append(len(parent) - 1)
        frontier = nxt
    return np.asarray(parent, dtype=np.int32)


def chain_tree(n_draft: int) -> np.ndarray:
    """Root followed by a single chain of n_draft nodes (plain speculative decoding)."""
    return np.arange(-1, n_draft, dtype=np.int32)


def static_topk_tree(n_draft: int, branching=(4, 3, 2, 2, 1, 1)) -> np.ndarray:
    """Static EAGLE-1 style pruned tree with `n_draft` draft nodes plus the root row.

    Every node of the full tree with the given per-level branching is named by its rank path
    (r_1..r_d), r_k < branching[k-1].  All nodes are ordered by (sum of ranks, depth, rank path) and
    the first `n_draft` are kept; a node's parent always sorts before it, so the kept set is closed
    under taking ancestors.  Rows are then numbered in BFS order with the children of one parent
    contiguous and in rank order.
    """
    full = []
    for d in range(1, len(branching) + 1):
        for path in itertools.product(*[range(b) for b in branching[:d]]):
            full.append(path)
    if n_draft > len(full):
        raise ValueError(f"at most {len(full)} draft nodes with branching {branching}")
    full.sort(key=lambda p: (sum(p), len(p), p))
    kept = set(full[:n_draft])
    for p in kept:
        assert len(p) == 1 or p[:-1] in kept
    index = {(): 0}
    parent = [-1]
    frontier = [()]
    while frontier:
        nxt = []
        for par in frontier:
            d = len(par)
            if d >= len(branching):
                continue
            for r in range(branching[d]):
                child = par + (r,)
                if child in kept:
                    index[child] = len(parent)
                    parent.append(index[par])
                    nxt.append(child)
        frontier = nxt
    assert len(parent) == n_draft + 1
    return np.asarray(parent, dtype=np.int32)


def random_tree(rng: np.random.Generator, n_rows: int, max_children: int = 4) -> np.ndarray:
    """A random tree in BFS order with contiguous sibling groups (for property tests)."""
    parent = [-1]
    frontier = [0]
    while len(parent) < n_rows and frontier:
        nxt = []
        for p in frontier:
            k = int(rng.integers(0, max_children + 1))
            if p == frontier[-1] and not nxt and k == 0:
                k = 1  # keep the tree growing
            for _ in range(k):
                if len(parent) >= n_rows:
                    break
                parent.append(p)
                nxt.append(len(parent) - 1)
        frontier = nxt
    return np.asarray(parent, dtype=np.int32)


def tree_depth(parent: np.ndarray) -> np.ndarray:
    depth = np.zeros(len(parent), dtype=np.int32)
    for j in range(1, len(parent)):
        depth[j] = depth[parent[j]] + 1
    return depth


def level_widths(parent: np.ndarray) -> list[int]:
    d = tree_depth(parent)
    return [int((d == l).sum()) for l in range(1, int(d.max()) + 1)] if len(parent) > 1 else []


# --------------------------------------------------------------------------------------------
# codebook, weights, caches
# --------------------------------------------------------------------------------------------


def clustered_codebook(rng, V: int, h: int, n_clusters: int, sigma: float, w: float = 0.02) -> np.ndarray:
    """Image-token embedding table E[V,h]: token v sits at w*(mu_{v mod n_clusters} + sigma*xi_v).

    Many codes of one cluster are near-identical, which is the redundancy of image vocabularies the
    paper's relaxation exploits.
    """
    mu = rng.standard_normal((n_clusters, h), dtype=np.float32)
    E = np.empty((V, h), dtype=np.float32)
    for c in range(n_clusters):
        rows = np.arange(c, V, n_clusters)
        E[rows] = w * (mu[c][None, :] + sigma * rng.standard_normal((len(rows), h), dtype=np.float32))
    return E


def gaussian(rng, shape, std: float = 1.0) -> np.ndarray:
    return (std * rng.standard_normal(shape, dtype=np.float32)).astype(np.float32)


@dataclass
class LayerWeights:
    """One pre-norm Llama-style decoder layer; every matrix is [out_features, in_features]."""

    gamma_attn: np.ndarray
    wq: np.ndarray
    wk: np.ndarray
    wv: np.ndarray
    wo: np.ndarray
    gamma_mlp: np.ndarray
    w_gate: np.ndarray
    w_up: np.ndarray
    w_down: np.ndarray


def layer_weights(rng, h: int, n_heads: int, head_dim: int, ffn: int, std: float = 0.02) -> LayerWeights:
    hd = n_heads * head_dim
    return LayerWeights(
        gamma_attn=np.ones(h, np.float32),
        wq=gaussian(rng, (hd, h), std),
        wk=gaussian(rng, (hd, h), std),
        wv=gaussian(rng, (hd, h), std),
        wo=gaussian(rng, (h, hd), std),
        gamma_mlp=np.ones(h, np.float32),
        w_gate=gaussian(rng, (ffn, h), std),
        w_up=gaussian(rng, (ffn, h), std),
        w_down=gaussian(rng, (h, ffn), std),
    )


# --------------------------------------------------------------------------------------------
# stand-in drafter (outside the verification boundary: it only supplies tokens and probabilities)
# --------------------------------------------------------------------------------------------


def cluster_drafter(
    rng,
    parent: np.ndarray,
    B: int,
    V: int,
    n_clusters: int,
    stay: float = 0.75,
    sharp: float = 1.6,
    roots=None,
):
    """Target-free stand-in for a trained drafter.

    For a parent token t the proposal distribution puts mass `stay` on the codes of t's own cluster
    and `1-stay` on one other cluster picked per parent, each spread over the member codes with a
    random per-code weight raised to `sharp`; the children of one parent are drawn from it without
    replacement, best first.  Returns tok[B,T] (row 0 = the pending root token) and draft_p[B,T]
    (probability the stand-in assigned to each drafted token under its parent's context; row 0 = 1).
    `roots` [B] fixes the root tokens (a decode loop's pending tokens) instead of drawing them.
    """
    T = len(parent)
    per = V // n_clusters
    tok = np.zeros((B, T), dtype=np.int32)
    p = np.ones((B, T), dtype=np.float32)
    children = [[] for _ in range(T)]
    for j in range(1, T):
        children[parent[j]].append(j)
    for b in range(B):
        tok[b, 0] = int(rng.integers(0, V)) if roots is None else int(roots[b])
        for j in range(T):
            kids = children[j]
            if not kids:
                continue
            c_own = int(tok[b, j]) % n_clusters
            c_alt = int((c_own + 1 + rng.integers(0, n_clusters - 1)) % n_clusters)
            w_own = rng.random(per) ** sharp
            w_alt = rng.random(per) ** sharp
            prob = np.concatenate([stay * w_own / w_own.sum(), (1.0 - stay) * w_alt / w_alt.sum()])
            ids = np.concatenate([c_own + n_clusters * np.arange(per), c_alt + n_clusters * np.arange(per)])
            # sample without replacement (Gumbel top-k), then order best-first like a top-k drafter
            g = np.log(prob) - np.log(-np.log(rng.random(len(prob))))
            pick = np.argsort(-g)[: len(kids)]
            pick = pick[np.argsort(-prob[pick], kind="stable")]
            for kid, i in zip(kids, pick):
                tok[b, kid] = ids[i]
                p[b, kid] = prob[i]
    return tok, p


# --------------------------------------------------------------------------------------------
# workload descriptions
# --------------------------------------------------------------------------------------------


@dataclass
class Workload:
    """Shape and recipe of one synthetic verify-step workload."""

    name: str
    dtype: str  # "f32" or "bf16"
    B: int
    h: int
    n_heads: int
    head_dim: int
    V: int
    n_clusters: int
    sigma: float
    prefix_len: int
    tree: str  # "binary3" | "topk<N>" | "chain<N>" | "nary<b>x<l>"
    cfg_scale: float
    tau_pos: float
    tau_seq: float
    ffn: int
    tvd_budget: float = 0.5
    seed: int = 0
    eps: float = 1e-6
    rope_base: float = 10000.0
    extra: dict = field(default_factory=dict)

    def parent(self) -> np.ndarray:
        if self.tree == "binary3":
            return complete_tree(2, 3)
        if self.tree.startswith("topk"):
            return static_topk_tree(int(self.tree[4:]))
        if self.tree.startswith("chain"):
            return chain_tree(int(self.tree[5:]))
        if self.tree.startswith("nary"):           # "nary<b>x<l>": complete tree, b children per node, l draft levels
            b, l = self.tree[4:].split("x")
            return complete_tree(int(b), int(l))
        raise ValueError(self.tree)


def workload(name: str, **over) -> Workload:
    """Named workloads.  'toy' is small enough for a CPU check in seconds; 'janus' and 'lumina'
    have the shapes of the two target models the paper measures; 'sweep' cells override B, the tree
    size, prefix length and cluster tightness."""
    table = {
        "toy": dict(dtype="f32", B=1, h=256, n_heads=4, head_dim=64, V=1024, n_clusters=64, sigma=0.1,
                    prefix_len=64, tree="binary3", cfg_scale=4.0, tau_pos=0.85, tau_seq=0.5, ffn=688, seed=0),
        "janus": dict(dtype="bf16", B=1, h=4096, n_heads=32, head_dim=128, V=16384, n_clusters=256, sigma=0.1,
                      prefix_len=384, tree="topk60", cfg_scale=5.0, tau_pos=0.85, tau_seq=0.5, ffn=11008, seed=1),
        "lumina": dict(dtype="bf16", B=1, h=4096, n_heads=32, head_dim=128, V=65536, n_clusters=256, sigma=0.1,
                       prefix_len=2480, tree="topk60", cfg_scale=3.0, tau_pos=0.95, tau_seq=0.925, ffn=11008,
                       seed=2),
        "sweep": dict(dtype="bf16", B=8, h=4096, n_heads=32, head_dim=128, V=16384, n_clusters=256, sigma=0.1,
                      prefix_len=1024, tree="topk64", cfg_scale=5.0, tau_pos=0.85, tau_seq=0.5, ffn=11008, seed=3),
        # LlamaGen-XL-Stage2, the model behind the paper's largest speed-ups.  The paper gives its thresholds, guidance
        # scale and sequence length (1024 image tokens) but no shape; ASSUMED here: width 1280, SwiGLU 3584, vocabulary
        # 16384, a 120-token text prefix (that model's published configuration), with its 20 heads of 64 regrouped as
        # 10 heads of 128 (the bf16 attention kernel takes head size 128), half-way through an image (120 + 512 keys)
        "llamagen": dict(dtype="bf16", B=1, h=1280, n_heads=10, head_dim=128, V=16384, n_clusters=256, sigma=0.1,
                         prefix_len=632, tree="topk60", cfg_scale=3.0, tau_pos=0.85, tau_seq=0.5, ffn=3584, seed=5),
        # reduced-width stand-ins of the same structure for CPU-side and quick GPU tests
        "mini": dict(dtype="bf16", B=2, h=512, n_heads=4, head_dim=128, V=2048, n_clusters=64, sigma=0.1,
                     prefix_len=200, tree="topk32", cfg_scale=5.0, tau_pos=0.85, tau_seq=0.5, ffn=1408, seed=4),
    }
    cfg = dict(table[name])
    cfg.update(over)
    return Workload(name=name, **cfg)


def quantize(x: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 array holding exactly the values a buffer of element type `dtype` will hold."""
    x = np.asarray(x, np.float32)
    return round_to_bf16(x) if dtype == "bf16" else x


def attention_inputs(w: Workload, rng, T: int, n_kv_heads: int | None = None):
    """Stand-alone inputs of the tree attention: q, prefix K/V, tree K/V ~ N(0,1), in the workload's type."""
    R, H, D, P = 2 * w.B, w.n_heads, w.head_dim, w.prefix_len
    hkv = n_kv_heads or H
    g = lambda *shape: quantize(rng.standard_normal(shape, dtype=np.float32), w.dtype)
    return dict(q=g(R, T, H, D), k_prefix=g(R, P, hkv, D), v_prefix=g(R, P, hkv, D), k_tree=g(R, T, hkv, D),
                v_tree=g(R, T, hkv, D), prefix_len=np.full(R, P, np.int32))


def tail_inputs(w: Workload, rng, parent, noise: float = 0.15):
    """Inputs of the head / acceptance / selection pieces: a clustered codebook tied as LM head, hidden
    states that sit near the embedding of each row's token (so a row's target mass falls on that token's
    cluster, spread thinly over near-identical codes), stand-in drafter tokens and probabilities,
    uniforms."""
    T = len(parent)
    E = quantize(clustered_codebook(rng, w.V, w.h, w.n_clusters, w.sigma), w.dtype)
    tok, p = cluster_drafter(rng, parent, w.B, w.V, w.n_clusters)
    base = E[np.concatenate([tok, tok], 0)]                                      # [2B,T,h]
    hidden = quantize(base + noise * 0.02 * rng.standard_normal(base.shape, dtype=np.float32), w.dtype)
    gamma = (1.0 + 0.1 * rng.standard_normal(w.h, dtype=np.float32)).astype(np.float32)
    return dict(w_head=E, hidden=hidden, gamma_final=gamma, tok=tok, draft_p=p, uniforms=uniforms(rng, w.B, T))


def uniforms(rng, B: int, T: int) -> np.ndarray:
    """Pre-drawn acceptance draws r ~ U[0,1) (the verification rule's `random()` made an input)."""
    return rng.random((B, T), dtype=np.float32)


def layer_step_inputs(w: Workload, rng, parent, n_layers: int = 1, out_scale=None):
    """Inputs of a verification step that runs through decoder layers: the clustered codebook as token
    embedding and (tied) LM head, `n_layers` sets of N(0, 0.02) layer weights, an N(0,1) prefix KV cache
    per layer (independent for the cond and uncond rows), stand-in drafter tokens and probabilities,
    uniforms.  Everything is returned in the values the workload's element type can hold.

    out_scale = (s_o, s_down) multiplies the output projection and the MLP down projection.  With plain
    N(0, 0.02) matrices of these widths one layer's update is ~100x the norm of the token embedding, the
    final hidden state forgets its token and no draft is ever accepted; the default for the 7B-shaped
    workloads, (0.05, 0.005), keeps the update at about 0.6x the embedding norm (as in a trained model,
    where a layer nudges the residual stream), so that acceptance and relaxation both take part.  The
    fp32 toy workload keeps the plain weights its definition names."""
    T = len(parent)
    R, H, D, P = 2 * w.B, w.n_heads, w.head_dim, w.prefix_len
    E = quantize(clustered_codebook(rng, w.V, w.h, w.n_clusters, w.sigma), w.dtype)
    if out_scale is None:
        out_scale = (1.0, 1.0) if w.name == "toy" else (0.05, 0.005)
    layers = []
    caches = []
    for _ in range(n_layers):
        lw = layer_weights(rng, w.h, H, D, w.ffn)
        lw.wo = lw.wo * np.float32(out_scale[0])
        lw.w_down = lw.w_down * np.float32(out_scale[1])
        for name in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
            setattr(lw, name, quantize(getattr(lw, name), w.dtype))
        layers.append(lw)
        caches.append((quantize(rng.standard_normal((R, P, H, D), dtype=np.float32), w.dtype),
                       quantize(rng.standard_normal((R, P, H, D), dtype=np.float32), w.dtype)))
    tok, p = cluster_drafter(rng, parent, w.B, w.V, w.n_clusters)
    gamma = (1.0 + 0.1 * rng.standard_normal(w.h, dtype=np.float32)).astype(np.float32)
    return dict(embed=E, w_head=E, layers=layers, k_prefix=[c[0] for c in caches], v_prefix=[c[1] for c in caches],
                gamma_final=gamma, tok=tok, draft_p=p, uniforms=uniforms(rng, w.B, T),
                prefix_len=np.full(R, P, np.int32))
