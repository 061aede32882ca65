"""Pins for the CPU checker's support pieces (rotary map, decoder layer plumbing, whole step)."""
import numpy as np
import torch

from oracle import cascade_oracle as O
from paper_2605_07230_b200 import synth


def test_rope_is_complex_rotation():
    rng = np.random.default_rng(0)
    T, H, D = 5, 2, 8
    x = rng.standard_normal((T, H, D))
    pos = np.array([0, 3, 3, 10, 77])
    out = O.rope(x, pos, 10000.0)
    z = x[..., : D // 2] + 1j * x[..., D // 2:]
    theta = pos[:, None] * 10000.0 ** (-2.0 * np.arange(D // 2) / D)
    zr = z * np.exp(1j * theta)[:, None, :]
    assert np.allclose(out[..., : D // 2], zr.real) and np.allclose(out[..., D // 2:], zr.imag)
    assert np.allclose(out[0], x[0])                                   # position 0 is the identity
    assert np.allclose(np.linalg.norm(out, axis=-1), np.linalg.norm(x, axis=-1))
    # relative-position property: <rope(q,m), rope(k,n)> depends only on m - n
    q, k = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))
    d1 = (O.rope(q, [5], 100.0) * O.rope(k, [2], 100.0)).sum()
    d2 = (O.rope(q, [13], 100.0) * O.rope(k, [10], 100.0)).sum()
    assert abs(d1 - d2) < 1e-12


def test_silu_and_round_bf16_against_library():
    x = np.linspace(-6, 6, 101)
    assert np.allclose(O.silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy(), atol=1e-15)
    y = np.random.default_rng(1).standard_normal(1000).astype(np.float32)
    ref = torch.from_numpy(y).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(y), ref)


def _layer(rng, h, H, D, ffn, std=0.05):
    return synth.layer_weights(rng, h, H, D, ffn, std)


def test_zero_output_projections_make_the_layer_an_identity():
    rng = np.random.default_rng(2)
    h, H, D, ffn, T, P = 16, 2, 8, 24, 7, 5
    lw = _layer(rng, h, H, D, ffn)
    lw.wo[:] = 0
    lw.w_down[:] = 0
    parent = synth.random_tree(rng, T)
    x = rng.standard_normal((2, T, h))
    kp, vp = rng.standard_normal((2, P, H, D)), rng.standard_normal((2, P, H, D))
    out, *_ = O.decoder_layer(x, lw, kp, vp, [P, P], parent, H, D, 1e-6, 10000.0, False)
    assert np.array_equal(out, x)


def test_layer_matches_torch_modules_on_a_chain():
    """Chain tree + empty prefix: the layer is an ordinary causal pre-norm block (torch as library)."""
    rng = np.random.default_rng(3)
    h, H, D, ffn, T = 16, 2, 8, 24, 6
    lw = _layer(rng, h, H, D, ffn, 0.2)
    lw.gamma_attn = rng.uniform(0.5, 1.5, h).astype(np.float32)
    lw.gamma_mlp = rng.uniform(0.5, 1.5, h).astype(np.float32)
    x = rng.standard_normal((1, T, h))
    empty = np.zeros((1, 0, H, D))
    out, q, k, v = O.decoder_layer(x, lw, empty, empty, [0], synth.chain_tree(T - 1), H, D, 1e-5, 10000.0, False)
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    xt = t(x[0])
    a = torch.nn.functional.rms_norm(xt, (h,), t(lw.gamma_attn), 1e-5)
    qt, kt, vt = (torch.nn.functional.linear(a, t(w)).view(T, H, D) for w in (lw.wq, lw.wk, lw.wv))

    def rot(z):
        inv = 10000.0 ** (-torch.arange(0, D, 2, dtype=torch.float64) / D)
        ang = torch.arange(T, dtype=torch.float64)[:, None] * inv[None]
        cos, sin = torch.cat([ang.cos(), ang.cos()], -1)[:, None], torch.cat([ang.sin(), ang.sin()], -1)[:, None]
        rot_half = torch.cat([-z[..., D // 2:], z[..., : D // 2]], -1)
        return z * cos + rot_half * sin

    qt, kt = rot(qt), rot(kt)
    att = torch.nn.functional.scaled_dot_product_attention(
        qt.permute(1, 0, 2), kt.permute(1, 0, 2), vt.permute(1, 0, 2), is_causal=True).permute(1, 0, 2)
    xt = xt + torch.nn.functional.linear(att.reshape(T, H * D), t(lw.wo))
    m = torch.nn.functional.rms_norm(xt, (h,), t(lw.gamma_mlp), 1e-5)
    xt = xt + torch.nn.functional.linear(
        torch.nn.functional.silu(torch.nn.functional.linear(m, t(lw.w_gate))) * torch.nn.functional.linear(m, t(lw.w_up)),
        t(lw.w_down))
    assert np.allclose(out[0], xt.numpy(), atol=1e-11)
    assert np.allclose(q[0], qt.numpy(), atol=1e-12)


def test_verify_step_composes_the_pieces():
    rng = np.random.default_rng(4)
    w = synth.workload("toy")
    parent = w.parent()
    T = len(parent)
    E = synth.clustered_codebook(rng, w.V, w.h, w.n_clusters, w.sigma)
    lw = synth.layer_weights(rng, w.h, w.n_heads, w.head_dim, w.ffn)
    kp = rng.standard_normal((2, w.prefix_len, w.n_heads, w.head_dim))
    vp = rng.standard_normal((2, w.prefix_len, w.n_heads, w.head_dim))
    tok, p = synth.cluster_drafter(rng, parent, 1, w.V, w.n_clusters)
    u = synth.uniforms(rng, 1, T)
    out = O.verify_step(E, [lw], np.ones(w.h), E, tok, parent, [kp], [vp], [w.prefix_len] * 2, p, u,
                        w.n_heads, w.head_dim, w.eps, w.rope_base, w.cfg_scale, 1.0, w.tau_pos, w.tau_seq,
                        w.tvd_budget, kv_bf16=False)
    x = E[np.concatenate([tok, tok])].astype(np.float64)
    x2, *_ = O.decoder_layer(x, lw, kp, vp, [w.prefix_len] * 2, parent, w.n_heads, w.head_dim, w.eps,
                             w.rope_base, False)
    assert np.array_equal(out["hidden"], x2)
    head = O.lm_head_cfg(x2, np.ones(w.h), w.eps, E, w.cfg_scale)
    assert np.array_equal(out["head"]["logits"], head["logits"])
    acc = O.relaxed_accept(head["feat"][0], head["logits"][0], tok[0], parent, p[0], u[0], w.tau_pos, w.tau_seq,
                           w.tvd_budget)
    assert np.array_equal(out["accept"][0]["accept"], acc["accept"])
    assert out["accept"][0]["path"] == O.select_path(acc["accept"], parent, acc["tvd_out"])[0]


def _causal_block(x_seq, lw, H, D, eps, base):
    """A plain causal pre-norm block over a token sequence, positions 0..n-1, in torch (library routines:
    rms_norm, linear, scaled_dot_product_attention, silu).  Returns (output rows, rotated keys, values)."""
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    n, h = x_seq.shape
    xt = t(x_seq)
    a = torch.nn.functional.rms_norm(xt, (h,), t(lw.gamma_attn), eps)
    qt, kt, vt = (torch.nn.functional.linear(a, t(w)).view(n, H, D) for w in (lw.wq, lw.wk, lw.wv))

    def rot(z):
        inv = base ** (-torch.arange(0, D, 2, dtype=torch.float64) / D)
        ang = torch.arange(n, dtype=torch.float64)[:, None] * inv[None]
        cos, sin = torch.cat([ang.cos(), ang.cos()], -1)[:, None], torch.cat([ang.sin(), ang.sin()], -1)[:, None]
        return z * cos + torch.cat([-z[..., D // 2:], z[..., : D // 2]], -1) * sin

    qt, kt = rot(qt), rot(kt)
    att = torch.nn.functional.scaled_dot_product_attention(
        qt.permute(1, 0, 2), kt.permute(1, 0, 2), vt.permute(1, 0, 2), is_causal=True).permute(1, 0, 2)
    xt = xt + torch.nn.functional.linear(att.reshape(n, H * D), t(lw.wo))
    m = torch.nn.functional.rms_norm(xt, (h,), t(lw.gamma_mlp), eps)
    xt = xt + torch.nn.functional.linear(
        torch.nn.functional.silu(torch.nn.functional.linear(m, t(lw.w_gate))) * torch.nn.functional.linear(m, t(lw.w_up)),
        t(lw.w_down))
    return xt.numpy(), kt.numpy(), vt.numpy()


def test_every_root_to_node_path_is_a_causal_sequence_after_the_prefix():
    """Position rule and masking of the layer on a BRANCHING tree with a NON-EMPTY prefix: tree decoding verifies
    several continuations of one prefix at once (Section 3), so the layer's output at node j must be what an
    ordinary causal block gives for the last token of the sequence  prefix tokens + root-to-j path.  The cache
    rows handed to the layer are the keys / values of the prefix tokens rotated at positions 0..P-1.  Using the
    row index instead of the depth as the position, dropping the prefix length from it, or letting a row see a
    non-ancestor each fail this for some node.  The two rows of the pair get prefixes of different lengths."""
    rng = np.random.default_rng(5)
    h, H, D, ffn = 16, 2, 8, 24
    eps, base = 1e-5, 10000.0
    lw = _layer(rng, h, H, D, ffn, 0.2)
    lw.gamma_attn = rng.uniform(0.5, 1.5, h).astype(np.float32)
    lw.gamma_mlp = rng.uniform(0.5, 1.5, h).astype(np.float32)
    parent = synth.static_topk_tree(11, (3, 2, 2))       # 12 rows, three levels, siblings at every level
    T = len(parent)
    depth = synth.tree_depth(parent)
    assert depth.max() == 3 and any(depth[j] != j for j in range(T))
    P = [5, 3]
    Pmax = max(P)
    x_prefix = [rng.standard_normal((p, h)) for p in P]
    x_tree = rng.standard_normal((2, T, h))
    kp, vp = np.zeros((2, Pmax, H, D)), np.zeros((2, Pmax, H, D))
    for r in range(2):
        _, k, v = _causal_block(x_prefix[r], lw, H, D, eps, base)
        kp[r, :P[r]], vp[r, :P[r]] = k, v
        kp[r, P[r]:], vp[r, P[r]:] = 1e6, -1e6          # rows beyond the prefix length must never be read
    out, q, k, v = O.decoder_layer(x_tree, lw, kp, vp, P, parent, H, D, eps, base, False)
    for r in range(2):
        for j in range(T):
            path = []
            i = j
            while i >= 0:
                path.append(i)
                i = parent[i]
            path.reverse()
            seq = np.concatenate([x_prefix[r], x_tree[r, path]], 0)
            want, k_seq, v_seq = _causal_block(seq, lw, H, D, eps, base)
            assert np.allclose(out[r, j], want[-1], atol=1e-10), (r, j)
            assert np.allclose(k[r, j], k_seq[-1], atol=1e-11) and np.allclose(v[r, j], v_seq[-1], atol=1e-11)
