"""CPU checker for the CASCADE tree-verification step.  TEST INFRASTRUCTURE, NOT THE PRODUCT.

A plain, slow, fp64 numpy statement of what one verification step computes, written from the paper
("CASCADE: Context-Aware Relaxation for Speculative Image Decoding"): Algorithm 1 (speculative
sampling accept test), Section 4.1 (cosine similarity of target hidden states, Eq. 1 interchangeable
set, Eq. 2 convergence set), Section 4.2 (Eq. 3 aggregation under a TVD budget) and Algorithm 2
(relaxed verification).  Only tests, the smoke check and the CPU-baseline leg of the benchmark may
call it.  It shares no code with the CUDA library and imports nothing from it.

No blocking, fusion or reordering: attention is the dense masked softmax, the LM head is a dense
matrix product (numpy's matmul is the library step), acceptance follows Algorithm 2's order of
operations node by node.  Everything is computed in float64 from the given inputs.

Where the paper is silent or inconsistent the reading taken is stated at the function.

Parity pins (tests/test_oracle_*.py): every function below is pinned to something outside itself:
textbook causal / decode attention, CFG end points and linearity, closed-form cosine cases, reduction
to Algorithm 1 with the relaxation off, an independently written sequential walk of Algorithm 2,
brute-force path enumeration, threshold monotonicity with an unbounded budget, hand-computed trees,
exact recovery of the target distribution by accept test + residual draw (Algorithm 1's guarantee), the
library's soft cross-entropy / KL divergence + entropy for the drafter loss of Eq. 4,
the library's top-k and a brute-force nucleus for the truncation of the target distribution.
`decoder_layer` (architecture from the workload definition, not from the paper) is pinned against an
ordinary causal block built from torch's library routines: on a chain with an empty prefix, and on a
branching tree behind prefixes of two lengths, where every root-to-node path must come out as the last
token of the plain causal sequence  prefix + path  (position = prefix length + depth, ancestors only).
"""
from __future__ import annotations

import numpy as np

USE_I = 1  # Eq. 1 relaxation on
USE_C = 2  # Eq. 2 relaxation on
CONV_DIST_SELF = 4  # Eq. 3 read literally: convergence mass taken under the candidate's own row

SELECT_LONGEST = 0
SELECT_FIRST_ACCEPT = 1

NEAR = 1e-3  # scores this close to a threshold are reported, and excluded from exact comparison


# ------------------------------------------------------------------------------------------------
# tree helpers
# ------------------------------------------------------------------------------------------------


def check_tree(parent) -> None:
    """Row 0 is the root (the pending last-emitted token); rows are in BFS order with the children
    of one parent contiguous (the static tree mask of Section 3, 'tree decoding')."""
    parent = np.asarray(parent)
    assert parent[0] == -1
    depth = tree_depth(parent)
    for j in range(1, len(parent)):
        assert 0 <= parent[j] < j
        assert depth[j] >= depth[j - 1]
        assert parent[j] >= parent[j - 1] or j == 1


def tree_depth(parent) -> np.ndarray:
    depth = np.zeros(len(parent), dtype=np.int64)
    for j in range(1, len(parent)):
        depth[j] = depth[parent[j]] + 1
    return depth


def children_of(parent) -> list[list[int]]:
    kids = [[] for _ in range(len(parent))]
    for j in range(1, len(parent)):
        kids[parent[j]].append(j)
    return kids


def ancestor_mask(parent) -> np.ndarray:
    """anc[j, i] = True iff i is j itself or an ancestor of j (root included)."""
    T = len(parent)
    anc = np.zeros((T, T), dtype=bool)
    for j in range(T):
        i = j
        while i >= 0:
            anc[j, i] = True
            i = parent[i]
    return anc


# ------------------------------------------------------------------------------------------------
# (a) tree-masked attention  --  Section 3: the draft tree is verified "via a parallel forward pass"
# ------------------------------------------------------------------------------------------------


def tree_attention(q, k_prefix, v_prefix, prefix_len, k_tree, v_tree, parent, scale):
    """out[r, j, hd] = sum_i softmax_i(scale * q[r,j,hd] . k_i) v_i  over the keys tree row j may see:
    the prefix cache entries 0..prefix_len[r]-1 and the tree rows that are j or its ancestors.

    q [R,T,Hq,D]; k_prefix, v_prefix [R,Pmax,Hkv,D]; prefix_len [R]; k_tree, v_tree [R,T,Hkv,D].
    R = 2B rows of the CFG pair (cond rows first).  Hq is a multiple of Hkv.
    """
    q = np.asarray(q, np.float64)
    R, T, Hq, D = q.shape
    Hkv = k_prefix.shape[2]
    anc = ancestor_mask(parent)
    out = np.zeros((R, T, Hq, D))
    for r in range(R):
        P = int(prefix_len[r])
        allowed = np.concatenate([np.ones((T, P), dtype=bool), anc], axis=1)
        for hq in range(Hq):
            hk = hq // (Hq // Hkv)
            keys = np.concatenate([k_prefix[r, :P, hk], k_tree[r, :, hk]], axis=0).astype(np.float64)
            vals = np.concatenate([v_prefix[r, :P, hk], v_tree[r, :, hk]], axis=0).astype(np.float64)
            s = scale * (q[r, :, hq] @ keys.T)
            s = np.where(allowed, s, -np.inf)
            s = s - s.max(axis=1, keepdims=True)
            w = np.exp(s)
            w = w / w.sum(axis=1, keepdims=True)
            out[r, :, hq] = w @ vals
    return out


# ------------------------------------------------------------------------------------------------
# (b) final norm, LM head, classifier-free guidance, vocabulary softmax
# ------------------------------------------------------------------------------------------------


def rmsnorm(x, gamma, eps):
    x = np.asarray(x, np.float64)
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * np.asarray(gamma, np.float64)


def lm_head_cfg(hidden, gamma, eps, w_head, cfg_scale, temperature=1.0):
    """hidden [2B,T,h] (cond rows 0..B-1, uncond rows B..2B-1) -> dict with

    logits [B,T,V] = (l_u + s (l_c - l_u)) / temperature, l_x = W n_x, n_x = RMSNorm(hidden_x)
    feat   [B,T,h] = n_c      (the target's text-conditioned hidden state that feeds the head)
    feat_norm [B,T], lse [B,T] = log sum_v exp(logits).

    The paper gives only the guidance scale (App. D.2); the mixing rule is the usual one on logits.
    """
    hidden = np.asarray(hidden, np.float64)
    B = hidden.shape[0] // 2
    W = np.asarray(w_head, np.float64)
    n = rmsnorm(hidden, gamma, eps)
    n_c, n_u = n[:B], n[B:]
    l_c = n_c @ W.T
    l_u = n_u @ W.T
    logits = (l_u + cfg_scale * (l_c - l_u)) / temperature
    return {
        "logits": logits,
        "feat": n_c,
        "feat_norm": np.sqrt((n_c * n_c).sum(-1)),
        "lse": log_sum_exp(logits),
    }


def log_sum_exp(logits):
    logits = np.asarray(logits, np.float64)
    m = logits.max(axis=-1, keepdims=True)
    return (m + np.log(np.exp(logits - m).sum(axis=-1, keepdims=True)))[..., 0]


def softmax(logits):
    """gtp of Algorithm 2: the target distribution at a tree row, i.e. for that row's children."""
    logits = np.asarray(logits, np.float64)
    return np.exp(logits - log_sum_exp(logits)[..., None])


def candidate_logits(logits, tok, parent):
    """For every draft node j: its token's logit under its parent's row and under its grandparent's
    row (0 where there is none) -- the only entries of the logits acceptance ever reads."""
    logits = np.asarray(logits, np.float64)
    B, T, _ = logits.shape
    lp = np.zeros((B, T))
    lg = np.zeros((B, T))
    for b in range(B):
        for j in range(1, T):
            pi = parent[j]
            lp[b, j] = logits[b, pi, tok[b, j]]
            if parent[pi] >= 0:
                lg[b, j] = logits[b, parent[pi], tok[b, j]]
    return lp, lg


# ------------------------------------------------------------------------------------------------
# (c) relaxed acceptance  --  Section 4.1-4.2, Eq. 1-3, Algorithm 2
# ------------------------------------------------------------------------------------------------


def cosine(a, b):
    """cos(F_a, F_b) = <F_a, F_b> / (||F_a|| ||F_b||)   (Section 4.1, measurement method)."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(a @ b) / (float(np.sqrt(a @ a)) * float(np.sqrt(b @ b)))


def similarity_scores(feat, parent):
    """cs[(a,b)] for siblings a != b (Eq. 1: same level, same prefix) and cc[(j,c)] for every
    tree edge j -> c (Eq. 2 restricted to continuations of the same sequence, as in the paper's toy
    example where F_3 is compared with its children F_7, F_8)."""
    kids = children_of(parent)
    cs, cc = {}, {}
    for j in range(len(parent)):
        for a in kids[j]:
            cc[(j, a)] = cosine(feat[j], feat[a])
            for b in kids[j]:
                if a != b:
                    cs[(a, b)] = cosine(feat[a], feat[b])
    return cs, cc


def relaxed_accept(feat, logits, tok, parent, draft_p, u, tau_pos, tau_seq, tvd_budget, flags=USE_I | USE_C):
    """Relaxed acceptance for ONE prompt.

    feat [T,h]   F_j: target hidden state at tree row j (after consuming tok[j])
    logits [T,V] row j is the target's (guided) logits for the position after row j
    tok [T], draft_p [T] (drafter probability of tok[j] under its parent's context), u [T] in [0,1)

    Per draft node j >= 1 with parent pi and g = softmax(logits[pi]) (Algorithm 2, gtp):
      q_j   = g[tok_j]
      I_j   = siblings b of j with cos(F_j, F_b) >= tau_pos                       (Eq. 1)
      C_j   = children c of j with cos(F_j, F_c) >= tau_seq                        (Eq. 2)
      mI_j  = sum of g over the distinct tokens of I_j other than tok_j
      mC_j  = sum of g (or of softmax(logits[j]) under CONV_DIST_SELF) over the distinct tokens of
              C_j other than tok_j and the tokens already counted in mI_j          (Eq. 3)
    Budget (Algorithm 2: one running total per verification step, each set added whole or not at
    all, interchangeable mass first): the walk reaches j only after accepting j's ancestors and
    rejecting j's earlier siblings, so the total on arrival at j is fixed by the tree and the masses:
    the first child starts from the total left after its parent, each later sibling from the total
    left after the previous one.
      t = running total;  qR = q_j
      if I_j non-empty and t + mI_j <= budget: qR += mI_j; t += mI_j
      if C_j non-empty and t + mC_j <= budget: qR += mC_j; t += mC_j
      accept_j = u_j < min(1, qR / p_j)                                            (Algorithm 1 test)
    accept_j is the decision Algorithm 2 takes for j if its walk visits j.

    Returns dict: accept [T] uint8, q_relaxed [T], q_plain [T], tvd_out [T], near [T] uint8 (bit 0: a
    cosine within NEAR of its threshold, bit 1: a budget comparison within NEAR, bit 2: the accept
    test within NEAR), set sizes.
    """
    T = len(parent)
    kids = children_of(parent)
    use_i = bool(flags & USE_I)
    use_c = bool(flags & USE_C)
    self_dist = bool(flags & CONV_DIST_SELF)
    feat = np.asarray(feat, np.float64)
    gtp_cache = {}

    def gtp(row):
        if row not in gtp_cache:
            gtp_cache[row] = softmax(np.asarray(logits[row], np.float64))
        return gtp_cache[row]

    accept = np.zeros(T, np.uint8)
    accept[0] = 1
    q_relaxed = np.zeros(T)
    q_plain = np.zeros(T)
    tvd_out = np.zeros(T)
    near = np.zeros(T, np.uint8)
    size_i = np.zeros(T, np.int32)
    size_c = np.zeros(T, np.int32)

    for pi in range(T):  # BFS order: tvd_out[pi] is final before pi's children are visited
        t = tvd_out[pi]
        g = gtp(pi) if kids[pi] else None
        for j in kids[pi]:
            q_j = g[tok[j]]
            set_i, set_c = [], []
            if use_i:
                for b in kids[pi]:
                    if b != j:
                        c = cosine(feat[j], feat[b])
                        if abs(c - tau_pos) < NEAR:
                            near[j] |= 1
                        if c >= tau_pos:
                            set_i.append(b)
            if use_c:
                for c_node in kids[j]:
                    c = cosine(feat[j], feat[c_node])
                    if abs(c - tau_seq) < NEAR:
                        near[j] |= 1
                    if c >= tau_seq:
                        set_c.append(c_node)
            tok_i = sorted({int(tok[b]) for b in set_i} - {int(tok[j])})
            tok_c = sorted({int(tok[c]) for c in set_c} - {int(tok[j])} - set(tok_i))
            m_i = float(sum(g[x] for x in tok_i))
            dist_c = gtp(j) if self_dist else g
            m_c = float(sum(dist_c[x] for x in tok_c))
            qR = q_j
            if set_i:
                if abs(t + m_i - tvd_budget) < NEAR:
                    near[j] |= 2
                if t + m_i <= tvd_budget:
                    qR += m_i
                    t += m_i
            if set_c:
                if abs(t + m_c - tvd_budget) < NEAR:
                    near[j] |= 2
                if t + m_c <= tvd_budget:
                    qR += m_c
                    t += m_c
            tvd_out[j] = t
            q_plain[j] = q_j
            q_relaxed[j] = qR
            size_i[j] = len(set_i)
            size_c[j] = len(set_c)
            p_j = float(draft_p[j])
            if p_j <= 0.0:
                accept[j] = 0
            else:
                ratio = min(1.0, qR / p_j)
                accept[j] = 1 if float(u[j]) < ratio else 0
                if abs(qR / p_j - float(u[j])) < NEAR:
                    near[j] |= 4
    return {
        "accept": accept,
        "q_relaxed": q_relaxed,
        "q_plain": q_plain,
        "tvd_out": tvd_out,
        "near": near,
        "size_i": size_i,
        "size_c": size_c,
    }


# ------------------------------------------------------------------------------------------------
# (d) path selection
# ------------------------------------------------------------------------------------------------


def select_path(accept, parent, tvd_out=None, mode=SELECT_LONGEST):
    """A node is valid if it and all its ancestors are accepted (the root always is).

    FIRST_ACCEPT is Algorithm 2's walk: from the root move to the first (smallest-index) accepted
    child; stop when a level accepts nobody.  LONGEST returns the deepest valid node, the smallest
    index among equals.  Returns (path_nodes root..end, alpha = number of accepted draft tokens,
    tvd_used = the running total when the walk stops: after the last child of the end node, or the
    end node's own if it has no children).
    """
    T = len(parent)
    kids = children_of(parent)
    depth = tree_depth(parent)
    if mode == SELECT_FIRST_ACCEPT:
        end = 0
        while True:
            nxt = [c for c in kids[end] if accept[c]]
            if not nxt:
                break
            end = nxt[0]
    else:
        valid = np.zeros(T, bool)
        valid[0] = True
        for j in range(1, T):
            valid[j] = bool(accept[j]) and valid[parent[j]]
        end = 0
        for j in range(T):
            if valid[j] and depth[j] > depth[end]:
                end = j
    path = []
    i = end
    while i >= 0:
        path.append(i)
        i = parent[i]
    path.reverse()
    tvd_used = 0.0
    if tvd_out is not None:
        tvd_used = float(tvd_out[kids[end][-1]] if kids[end] else tvd_out[end])
    return path, int(depth[end]), tvd_used


def bonus_token(logits_row, rejected_tokens, u):
    """The token that follows the accepted path (Algorithm 1, last step: after a rejection the next token is
    drawn from the target distribution with the rejected proposals removed; after a fully accepted path it is
    drawn from the target distribution itself).  Algorithm 2 leaves this step out; the reading here: the
    children of the path's end node were all rejected, their (distinct) tokens get probability zero, the rest
    of softmax(logits_row) is renormalised, and the token is the inverse-CDF sample at u in [0,1):
    the first v with cumsum(prob)[v] > u * total.  Returns (token, total = remaining mass)."""
    g = softmax(np.asarray(logits_row, np.float64))
    g = g.copy()
    for t in set(int(x) for x in rejected_tokens):
        g[t] = 0.0
    total = float(g.sum())
    c = np.cumsum(g)
    v = int(np.searchsorted(c, float(u) * total, side="right"))
    return min(v, len(g) - 1), total


def residual_token(logits_row, draft_row, any_rejected, u):
    """Algorithm 1's last step, literally: after a rejection the next token is drawn from the positive part of
    (target - drafter), renormalised,  [q - p]+ / sum [q - p]+ , with q = softmax(logits_row) and p the drafter's
    distribution at the same position; after a fully accepted draft (nothing rejected) it is drawn from q.  The
    draw is the inverse-CDF sample at u in [0,1): the first v with cumsum(weight)[v] > u * total.  Where nothing of
    q lies above p (p = q; Algorithm 1 then never rejects) q itself is used.  Returns (token, total), total = the
    sum of [q - p]+ (1.0 where q was used)."""
    q = softmax(np.asarray(logits_row, np.float64))
    w = q
    total = 1.0
    if any_rejected:
        r = np.maximum(q - np.asarray(draft_row, np.float64), 0.0)
        if r.sum() > 0.0:
            w, total = r, float(r.sum())
    c = np.cumsum(w)
    v = int(np.searchsorted(c, float(u) * c[-1], side="right"))
    return min(v, len(w) - 1), total


def drafter_loss(target_logits, draft_logits, feat, tau_seq, c):
    """The drafter's training loss of Section 4.3, Eq. 4: a soft cross-entropy between the target distribution q_k
    and the drafter's distribution p_k at every position k of a target-generated sequence,
        L = - sum_k w_k sum_v q_k(v) log p_k(v),
    re-weighted where consecutive target predictions converge: w_k = c if the pair (k, k+1) satisfies the
    convergence criterion of Eq. 2, cos(F_k, F_{k+1}) >= tau_seq on the target's hidden states, else 1 (the last
    position has no successor: w = 1).  target_logits, draft_logits [K,V]; feat [K,h].
    Returns (per-position weighted loss [K], weights [K], total)."""
    q = softmax(np.asarray(target_logits, np.float64))
    lp = np.asarray(draft_logits, np.float64)
    log_p = lp - log_sum_exp(lp)[..., None]
    K = q.shape[0]
    ce = -(q * log_p).sum(-1)
    w = np.ones(K)
    for k in range(K - 1):
        if cosine(feat[k], feat[k + 1]) >= tau_seq:
            w[k] = c
    return w * ce, w, float((w * ce).sum())


def filter_logits(logits, top_k, top_p):
    """Top-k / nucleus truncation of the target distribution before verification (the sampling settings
    of the paper's experiments, Appendix D.1: temperature 1, top-p 1.0, top-k 2000; the paper gives the
    numbers only, the truncations are the usual ones, stated here so that ties are decided).  Per row:
      top-k (0 < top_k < V): keep every token whose logit is >= the top_k-th largest logit of the row
        (tokens tied with it stay together, so more than top_k can remain);
      top-p (top_p < 1), on the distribution renormalised over what top-k kept: keep a token iff the
        probability of the tokens with a strictly larger logit is < top_p (the smallest set of most
        likely tokens whose mass reaches top_p; ties stay together).
    Dropped tokens get logit -inf, i.e. probability zero after the softmax.  Returns (filtered, kept)."""
    logits = np.asarray(logits, np.float64)
    V = logits.shape[-1]
    flat = logits.reshape(-1, V)
    out = flat.copy()
    kept = np.ones(flat.shape, bool)
    for i, row in enumerate(flat):
        keep = np.ones(V, bool)
        if 0 < top_k < V:
            kth = np.sort(row)[V - top_k]
            keep &= row >= kth
        if top_p < 1.0:
            p = softmax(np.where(keep, row, -np.inf))
            order = np.argsort(-row, kind="stable")
            sorted_l, sorted_p = row[order], p[order]
            before = np.cumsum(sorted_p) - sorted_p              # mass ahead of each position
            first_of_value = np.searchsorted(-sorted_l, -sorted_l, side="left")  # ties share the first position
            larger = np.empty(V)
            larger[order] = before[first_of_value]
            keep &= larger < top_p
        kept[i] = keep
        out[i, ~keep] = -np.inf
    return out.reshape(logits.shape), kept.reshape(logits.shape)


def append_path_kv(k_cache, v_cache, prefix_len, k_tree, v_tree, path, B):
    """Cache update after a step: the tree rows on the accepted path (root first) are appended, in path
    order, to both CFG rows' caches of one layer.  k_cache/v_cache [2B,cap,H,D] are modified in place;
    returns the new prefix lengths."""
    new_len = np.array(prefix_len, np.int64).copy()
    for b, nodes in enumerate(path):
        for r in (b, B + b):
            for i, node in enumerate(nodes):
                k_cache[r, prefix_len[r] + i] = k_tree[r, node]
                v_cache[r, prefix_len[r] + i] = v_tree[r, node]
            new_len[r] = prefix_len[r] + len(nodes)
    return new_len


# ------------------------------------------------------------------------------------------------
# support: the rest of one decoder layer (architecture from the workload definition, not the paper)
# ------------------------------------------------------------------------------------------------


def round_bf16(x):
    """Round to the nearest bf16 value (ties to even); used only where the workload stores bf16."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    bits = x32.view(np.uint32).astype(np.uint64)
    bits = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) << 16
    return bits.astype(np.uint32).view(np.float32).astype(np.float64)


def rope(x, pos, base):
    """Rotary embedding, half-split pairing: (x[i], x[i+D/2]) rotated by pos * base^(-2i/D).
    x [..., T, H, D], pos [T]."""
    x = np.asarray(x, np.float64)
    D = x.shape[-1]
    half = D // 2
    inv = base ** (-2.0 * np.arange(half) / D)
    ang = np.asarray(pos, np.float64)[:, None] * inv[None, :]  # [T, half]
    cos = np.cos(ang)[:, None, :]
    sin = np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def decoder_layer(x, lw, k_prefix, v_prefix, prefix_len, parent, n_heads, head_dim, eps, rope_base,
                  kv_bf16):
    """One pre-norm decoder layer over the tree rows.  x [R,T,h] -> (x_out [R,T,h], q, k_tree, v_tree).

    a = RMSNorm(x); q,k,v = a Wq^T, a Wk^T, a Wv^T; rotary at position prefix_len[r] + depth[j];
    tree attention; x += attn Wo^T; m = RMSNorm(x); x += (silu(m Wg^T) * (m Wu^T)) Wd^T.
    With kv_bf16 the rotated q, k and v are rounded to bf16, the storage type of the KV cache and of
    the attention operands in the bf16 workloads.
    """
    x = np.asarray(x, np.float64)
    R, T, h = x.shape
    depth = tree_depth(parent)
    f64 = lambda w: np.asarray(w, np.float64)
    a = rmsnorm(x, lw.gamma_attn, eps)
    q = (a @ f64(lw.wq).T).reshape(R, T, n_heads, head_dim)
    k = (a @ f64(lw.wk).T).reshape(R, T, n_heads, head_dim)
    v = (a @ f64(lw.wv).T).reshape(R, T, n_heads, head_dim)
    for r in range(R):
        pos = int(prefix_len[r]) + depth
        q[r] = rope(q[r], pos, rope_base)
        k[r] = rope(k[r], pos, rope_base)
    if kv_bf16:
        q, k, v = round_bf16(q), round_bf16(k), round_bf16(v)
    attn = tree_attention(q, k_prefix, v_prefix, prefix_len, k, v, parent, 1.0 / np.sqrt(head_dim))
    x = x + attn.reshape(R, T, n_heads * head_dim) @ f64(lw.wo).T
    m = rmsnorm(x, lw.gamma_mlp, eps)
    x = x + (silu(m @ f64(lw.w_gate).T) * (m @ f64(lw.w_up).T)) @ f64(lw.w_down).T
    return x, q, k, v


# ------------------------------------------------------------------------------------------------
# the whole step
# ------------------------------------------------------------------------------------------------


def verify_tail(hidden, gamma_f, eps, w_head, cfg_scale, temperature, tok, parent, draft_p, u,
                tau_pos, tau_seq, tvd_budget, flags=USE_I | USE_C, mode=SELECT_LONGEST):
    """Pieces (b)-(d) for B prompts: hidden [2B,T,h] -> logits, features, accept bits, paths."""
    head = lm_head_cfg(hidden, gamma_f, eps, w_head, cfg_scale, temperature)
    B = head["logits"].shape[0]
    res = []
    for b in range(B):
        acc = relaxed_accept(head["feat"][b], head["logits"][b], tok[b], parent, draft_p[b], u[b],
                             tau_pos, tau_seq, tvd_budget, flags)
        path, alpha, tvd_used = select_path(acc["accept"], parent, acc["tvd_out"], mode)
        acc.update(path=path, alpha=alpha, tvd_used=tvd_used)
        res.append(acc)
    return head, res


def verify_step(embed, layers, gamma_f, w_head, tok, parent, k_prefix, v_prefix, prefix_len, draft_p, u,
                n_heads, head_dim, eps, rope_base, cfg_scale, temperature, tau_pos, tau_seq, tvd_budget,
                flags=USE_I | USE_C, mode=SELECT_LONGEST, kv_bf16=True):
    """Full verification step: embed the tree tokens, run the decoder layers over the 2B rows of the
    CFG pair (same tokens and weights, different prefix caches), then verify_tail.

    k_prefix / v_prefix: lists (one per layer) of [2B,Pmax,H,D].
    """
    B = tok.shape[0]
    x = np.asarray(embed, np.float64)[np.concatenate([tok, tok], axis=0)]  # [2B,T,h]
    attn_io = []
    for li, lw in enumerate(layers):
        x, q, k, v = decoder_layer(x, lw, k_prefix[li], v_prefix[li], prefix_len, parent, n_heads, head_dim,
                                   eps, rope_base, kv_bf16)
        attn_io.append((q, k, v))
    head, res = verify_tail(x, gamma_f, eps, w_head, cfg_scale, temperature, tok, parent, draft_p, u,
                            tau_pos, tau_seq, tvd_budget, flags, mode)
    return {"hidden": x, "head": head, "accept": res, "attn_io": attn_io}
