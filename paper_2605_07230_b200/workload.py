"""Device-resident synthetic workloads for the verification step: moves the seeded host inputs of
`synth` into torch device buffers of the right element type and fills a `binding.Step`.

Data movement and argument marshalling only; all computation happens in libcascade.so.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import binding as cb
from . import synth


def to_device(x: np.ndarray, dtype: str, device) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x, np.float32))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    return t.to(device).contiguous()


@dataclass
class DeviceStep:
    """One set of device buffers for a verification step plus the Step struct that points at them."""

    host: dict
    dev: dict
    out: dict
    step: cb.Step = field(default=None)


class PiecesWorkload:
    """The four hot-path pieces on stand-alone inputs (no decoder-layer glue): tree attention on
    random q / K / V, and LM head + relaxed acceptance + path selection on hidden states that sit near
    their tokens' embeddings.  `n_sets` independent copies of every buffer let a benchmark rotate
    through more bytes than the L2 holds."""

    def __init__(self, w: synth.Workload, device="cuda:0", n_sets: int = 1, keep_logits: bool = False,
                 select_mode: int = cb.SELECT_LONGEST, flags: int = cb.USE_I | cb.USE_C):
        self.w = w
        self.device = device
        self.parent = w.parent()
        T = len(self.parent)
        self.T = T
        self.ctx = cb.Context(cb.BF16 if w.dtype == "bf16" else cb.F32, w.B, T, max(w.prefix_len, 1), w.h, w.n_heads,
                              w.n_heads, w.head_dim, w.V, 0)
        self.tree = cb.Tree(self.ctx, self.parent)
        self.params = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, flags)
        self.sets: list[DeviceStep] = []
        rng = np.random.default_rng(w.seed)
        host = {}
        host.update(synth.attention_inputs(w, rng, T))
        host.update(synth.tail_inputs(w, rng, self.parent))
        for s in range(n_sets):
            if s > 0:
                # fresh per-step inputs for every set; the big read-only tensors keep their values but
                # live at their own addresses
                rng_s = np.random.default_rng(w.seed * 1000 + s)
                tok, p = synth.cluster_drafter(rng_s, self.parent, w.B, w.V, w.n_clusters)
                base = host["w_head"][np.concatenate([tok, tok], 0)]
                hidden = synth.quantize(base + 0.15 * 0.02 * rng_s.standard_normal(base.shape, dtype=np.float32),
                                        w.dtype)
                host_s = dict(host, tok=tok, draft_p=p, hidden=hidden, uniforms=synth.uniforms(rng_s, w.B, T))
            else:
                host_s = host
            self.sets.append(self._make_set(host_s, keep_logits, select_mode))

    def _make_set(self, host, keep_logits, select_mode) -> DeviceStep:
        w, T, dev = self.w, self.T, self.device
        B = w.B
        d = {}
        for k in ("q", "k_prefix", "v_prefix", "k_tree", "v_tree", "hidden", "w_head"):
            d[k] = to_device(host[k], w.dtype, dev)
        d["gamma_final"] = torch.from_numpy(host["gamma_final"]).to(dev)
        d["prefix_len"] = torch.from_numpy(host["prefix_len"]).to(dev)
        d["tok"] = torch.from_numpy(host["tok"]).to(dev)
        d["draft_p"] = torch.from_numpy(host["draft_p"]).to(dev)
        d["uniforms"] = torch.from_numpy(host["uniforms"]).to(dev)
        el = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        o = dict(
            attn_out=torch.zeros((2 * B, T, w.n_heads, w.head_dim), dtype=el, device=dev),
            accept=torch.zeros((B, T), dtype=torch.uint8, device=dev),
            path_nodes=torch.zeros((B, self.tree.depth + 1), dtype=torch.int32, device=dev),
            path_len=torch.zeros(B, dtype=torch.int32, device=dev),
            q_relaxed=torch.zeros((B, T), device=dev),
            tvd_out=torch.zeros((B, T), device=dev),
            tvd_used=torch.zeros(B, device=dev),
            near_count=torch.zeros(B, dtype=torch.int32, device=dev),
            feat=torch.zeros((B, T, w.h), device=dev),
            scores=torch.zeros((B, max(self.tree.num_pairs, 1)), device=dev),
            row_lse=torch.zeros((B, T), device=dev),
        )
        if keep_logits or w.dtype != "bf16":
            o["logits"] = torch.zeros((B, T, w.V), device=dev)
        step = cb.make_step(
            layers=None, gamma_final=d["gamma_final"], w_head=d["w_head"], prefix_cap=w.prefix_len,
            prefix_len=d["prefix_len"], eps=w.eps, rope_base=w.rope_base,
            softmax_scale=float(1.0 / np.sqrt(w.head_dim)), cfg_scale=w.cfg_scale, temperature=1.0,
            tok=d["tok"], draft_p=d["draft_p"], uniforms=d["uniforms"], hidden_in=d["hidden"],
            q=d["q"], k_tree=d["k_tree"], v_tree=d["v_tree"],
            k_prefix=d["k_prefix"] if w.prefix_len > 0 else None, v_prefix=d["v_prefix"] if w.prefix_len > 0 else None,
            attn_out=o["attn_out"], params=self.params, select_mode=select_mode,
            accept=o["accept"], path_nodes=o["path_nodes"], path_len=o["path_len"], q_relaxed=o["q_relaxed"],
            tvd_out=o["tvd_out"], tvd_used=o["tvd_used"], near_count=o["near_count"], logits=o.get("logits"),
            feat=o["feat"], scores=o["scores"], row_lse=o["row_lse"])
        return DeviceStep(host=host, dev=d, out=o, step=step)

    def run(self, i: int = 0) -> DeviceStep:
        s = self.sets[i % len(self.sets)]
        cb.cascade_verify_step(self.ctx, self.tree, s.step)
        return s

    def close(self):
        self.tree.close()
        self.ctx.close()

    # bytes the algorithm has to move per step (each operand once), by piece
    def algorithmic_bytes(self) -> dict:
        w, T = self.w, self.T
        e = 2 if w.dtype == "bf16" else 4
        R = 2 * w.B
        attn = R * (w.prefix_len + T) * w.n_heads * w.head_dim * 2 * e + 2 * R * T * w.n_heads * w.head_dim * e
        head = w.V * w.h * e + R * T * w.h * e
        return {"tree_attn": attn, "lm_head": head}

    def algorithmic_flops(self) -> dict:
        w, T = self.w, self.T
        return {"lm_head": 2.0 * w.B * T * w.h * w.V,
                "tree_attn": 4.0 * 2 * w.B * w.n_heads * T * (w.prefix_len + T) * w.head_dim}


class LayerWorkload:
    """The whole verification step through `n_layers` decoder layers: token embedding, layers (tree
    attention over each layer's prefix cache), final norm, LM head with guidance, relaxed acceptance,
    path selection.  `n_sets` copies of the weights and caches live at their own addresses (a benchmark
    rotates through them so that a step never finds its operands in the L2)."""

    def __init__(self, w: synth.Workload, n_layers: int = 1, device="cuda:0", n_sets: int = 1,
                 keep_logits: bool = False, select_mode: int = cb.SELECT_LONGEST, flags: int = cb.USE_I | cb.USE_C,
                 host: dict | None = None, want_hidden: bool = True):
        self.w, self.device, self.n_layers = w, device, n_layers
        self.want_hidden = want_hidden      # ask the step for the final hidden states (one more kernel)
        self.parent = w.parent()
        T = self.T = len(self.parent)
        self.ctx = cb.Context(cb.BF16 if w.dtype == "bf16" else cb.F32, w.B, T, max(w.prefix_len, 1), w.h, w.n_heads,
                              w.n_heads, w.head_dim, w.V, w.ffn)
        self.tree = cb.Tree(self.ctx, self.parent)
        self.params = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, flags)
        rng = np.random.default_rng(w.seed)
        self.host = host if host is not None else synth.layer_step_inputs(w, rng, self.parent, n_layers)
        self.sets = [self._make_set(self.host if i == 0 else self._fresh_step(i), keep_logits, select_mode)
                     for i in range(n_sets)]

    def _fresh_step(self, i):
        rng = np.random.default_rng(self.w.seed * 1000 + i)
        tok, p = synth.cluster_drafter(rng, self.parent, self.w.B, self.w.V, self.w.n_clusters)
        return dict(self.host, tok=tok, draft_p=p, uniforms=synth.uniforms(rng, self.w.B, self.T))

    def _make_set(self, host, keep_logits, select_mode) -> DeviceStep:
        w, T, dev, B = self.w, self.T, self.device, self.w.B
        el = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        d = dict(embed=to_device(host["embed"], w.dtype, dev), gamma_final=f32(host["gamma_final"]),
                 prefix_len=f32(host["prefix_len"]), tok=f32(host["tok"]), draft_p=f32(host["draft_p"]),
                 uniforms=f32(host["uniforms"]))
        layers = []
        for li, lw in enumerate(host["layers"]):
            # q/k/v and gate/up stacked in memory: the library runs each group as one projection
            qkv = to_device(np.concatenate([lw.wq, lw.wk, lw.wv], 0), w.dtype, dev)
            gu = to_device(np.concatenate([lw.w_gate, lw.w_up], 0), w.dtype, dev)
            hd = w.n_heads * w.head_dim
            layers.append(dict(gamma_attn=f32(lw.gamma_attn), wq=qkv[:hd], wk=qkv[hd:2 * hd], wv=qkv[2 * hd:],
                               wo=to_device(lw.wo, w.dtype, dev), gamma_mlp=f32(lw.gamma_mlp), w_gate=gu[:w.ffn],
                               w_up=gu[w.ffn:], w_down=to_device(lw.w_down, w.dtype, dev),
                               k_prefix=to_device(host["k_prefix"][li], w.dtype, dev),
                               v_prefix=to_device(host["v_prefix"][li], w.dtype, dev), _keep=(qkv, gu)))
        d["layers"] = layers
        o = dict(
            accept=torch.zeros((B, T), dtype=torch.uint8, device=dev),
            path_nodes=torch.zeros((B, self.tree.depth + 1), dtype=torch.int32, device=dev),
            path_len=torch.zeros(B, dtype=torch.int32, device=dev),
            q_relaxed=torch.zeros((B, T), device=dev), tvd_out=torch.zeros((B, T), device=dev),
            tvd_used=torch.zeros(B, device=dev), near_count=torch.zeros(B, dtype=torch.int32, device=dev),
            feat=torch.zeros((B, T, w.h), device=dev), scores=torch.zeros((B, max(self.tree.num_pairs, 1)), device=dev),
            row_lse=torch.zeros((B, T), device=dev),
            hidden_out=torch.zeros((2 * B, T, w.h), device=dev) if self.want_hidden else None,
            k_tree_out=torch.zeros((self.n_layers, 2 * B, T, w.n_heads, w.head_dim), dtype=el, device=dev),
            v_tree_out=torch.zeros((self.n_layers, 2 * B, T, w.n_heads, w.head_dim), dtype=el, device=dev))
        if keep_logits or w.dtype != "bf16":
            o["logits"] = torch.zeros((B, T, w.V), device=dev)
        step = cb.make_step(
            layers=[{k: v for k, v in l.items() if k != "_keep"} for l in layers], embed=d["embed"],
            gamma_final=d["gamma_final"], w_head=d["embed"], prefix_cap=w.prefix_len, prefix_len=d["prefix_len"],
            eps=w.eps, rope_base=w.rope_base, softmax_scale=float(1.0 / np.sqrt(w.head_dim)), cfg_scale=w.cfg_scale,
            temperature=1.0, tok=d["tok"], draft_p=d["draft_p"], uniforms=d["uniforms"], params=self.params,
            select_mode=select_mode, accept=o["accept"], path_nodes=o["path_nodes"], path_len=o["path_len"],
            q_relaxed=o["q_relaxed"], tvd_out=o["tvd_out"], tvd_used=o["tvd_used"], near_count=o["near_count"],
            logits=o.get("logits"), feat=o["feat"], scores=o["scores"], row_lse=o["row_lse"],
            hidden_out=o["hidden_out"], k_tree_out=o["k_tree_out"], v_tree_out=o["v_tree_out"])
        return DeviceStep(host=host, dev=d, out=o, step=step)

    def run(self, i: int = 0) -> DeviceStep:
        s = self.sets[i % len(self.sets)]
        cb.cascade_verify_step(self.ctx, self.tree, s.step)
        return s

    def close(self):
        self.tree.close()
        self.ctx.close()

    def weight_bytes(self) -> dict:
        w = self.w
        e = 2 if w.dtype == "bf16" else 4
        hd = w.n_heads * w.head_dim
        return {"layer": (3 * hd * w.h + w.h * hd + 3 * w.ffn * w.h) * e * self.n_layers, "lm_head": w.V * w.h * e}


class DecodeLoop:
    """A speculative decode loop around the verification step (the last workload of the set: many layers,
    the caches grow by the accepted tokens every step).  Per step: the stand-in drafter proposes a tree
    below each prompt's pending token (host), the library verifies it (cascade_verify_step), draws the
    token after the accepted path (cascade_bonus_token) and appends the accepted rows to every layer's
    cache (cascade_kv_append); the host reads back the path and the new pending token.  Data movement and
    argument marshalling only."""

    def __init__(self, w: synth.Workload, n_layers: int, max_steps: int, device="cuda:0", seed: int = 0,
                 select_mode: int = cb.SELECT_LONGEST, tile_layers: bool = False, cap: int | None = None):
        # tile_layers: every layer gets the values of one seeded layer (its own copy on the device, its own
        # caches): for timing at full depth without generating 30 layers of weights on the host
        self.w, self.n_layers, self.device = w, n_layers, device
        self.parent = w.parent()
        T = self.T = len(self.parent)
        depth = int(synth.tree_depth(self.parent).max())
        # rows per cache: room for `max_steps` steps that each accept a whole path, unless the caller knows better
        # (a run that stops at a token count); a step that does not fit is refused by the library, not written
        self.cap = cap if cap is not None else w.prefix_len + max_steps * (depth + 1)
        B, R = w.B, 2 * w.B
        self.ctx = cb.Context(cb.BF16 if w.dtype == "bf16" else cb.F32, B, T, self.cap, w.h, w.n_heads, w.n_heads,
                              w.head_dim, w.V, w.ffn)
        self.tree = cb.Tree(self.ctx, self.parent)
        self.params = cb.Params(w.tau_pos, w.tau_seq, w.tvd_budget, cb.USE_I | cb.USE_C)
        rng = np.random.default_rng(w.seed)
        if tile_layers:
            host = synth.layer_step_inputs(w, rng, self.parent, 1)
            host["layers"] = host["layers"] * n_layers
            host["k_prefix"] = [host["k_prefix"][0]] * n_layers
            host["v_prefix"] = [host["v_prefix"][0]] * n_layers
        else:
            host = synth.layer_step_inputs(w, rng, self.parent, n_layers)
        # caches with room for the whole run; the first prefix_len rows hold the seeded prompt cache
        for li in range(n_layers):
            for name in ("k_prefix", "v_prefix"):
                full = np.zeros((R, self.cap, w.n_heads, w.head_dim), np.float32)
                full[:, :w.prefix_len] = host[name][li]
                host[name][li] = full
        self.host = host
        self.rng = np.random.default_rng(seed)
        self.roots = host["tok"][:, 0].copy()
        self.prefix_len_host = host["prefix_len"].astype(np.int64).copy()
        wl = LayerWorkload.__new__(LayerWorkload)   # reuse its buffer set-up on this context
        wl.w, wl.device, wl.n_layers, wl.parent, wl.T, wl.ctx, wl.tree, wl.params = (w, device, n_layers, self.parent, T,
                                                                                     self.ctx, self.tree, self.params)
        w_cap = synth.Workload(**{**w.__dict__, "prefix_len": self.cap})
        wl.w = w_cap
        wl.want_hidden = False                      # the loop has no use for the hidden states
        self.set = wl._make_set(host, True, select_mode)
        self.set.step.prefix_cap = self.cap
        self.u_bonus = torch.zeros(B, device=device)
        self.bonus = torch.zeros(B, dtype=torch.int32, device=device)
        self.mass = torch.zeros(B, device=device)
        self.emitted = [[] for _ in range(B)]
        self.graph = None
        self.launches_last_step = 0

    def draft(self):
        """Next tree of the stand-in drafter below the pending tokens, plus this step's uniforms."""
        w = self.w
        tok, p = synth.cluster_drafter(self.rng, self.parent, w.B, w.V, w.n_clusters, roots=self.roots)
        u = synth.uniforms(self.rng, w.B, self.T)
        ub = self.rng.random(w.B, dtype=np.float32)
        return tok, p, u, ub

    def _enqueue(self):
        """The device work of one step: verify, draw the token after the path, append the accepted rows."""
        d, o = self.set.dev, self.set.out
        cb.cascade_verify_step(self.ctx, self.tree, self.set.step)
        n_launch = self.ctx.last_launch_count
        cb.cascade_bonus_token(self.ctx, self.tree, o["logits"], d["tok"], o["path_nodes"], o["path_len"], self.u_bonus,
                               self.bonus, self.mass)
        n_launch += self.ctx.last_launch_count
        cb.cascade_kv_append(self.ctx, self.tree, self.set.step, o["k_tree_out"], o["v_tree_out"], o["path_nodes"],
                             o["path_len"], self.cap, d["prefix_len"])
        self.launches_last_step = n_launch + self.ctx.last_launch_count

    def capture(self):
        """Record the step's device work once as a CUDA graph; later steps replay it (all its pointers are
        fixed, the caches' fill levels live in device memory).  Call after at least one ordinary step."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                self._enqueue()
        torch.cuda.current_stream().wait_stream(side)
        self.graph = g

    def step(self, drafted=None, events_after=None):
        tok, p, u, ub = drafted if drafted is not None else self.draft()
        d, o = self.set.dev, self.set.out
        d["tok"].copy_(torch.from_numpy(tok))
        d["draft_p"].copy_(torch.from_numpy(p))
        d["uniforms"].copy_(torch.from_numpy(u))
        self.u_bonus.copy_(torch.from_numpy(ub))
        if self.graph is not None:
            self.graph.replay()
        else:
            self._enqueue()
        if events_after is not None:
            events_after.record()           # the device work of this step ends here
        plen = o["path_len"].cpu().numpy()
        nodes = o["path_nodes"].cpu().numpy()
        bonus = self.bonus.cpu().numpy()
        self.ctx.check()
        for b in range(self.w.B):
            path = nodes[b][: plen[b] + 1]
            self.emitted[b].extend(int(tok[b, j]) for j in path[1:])
            self.emitted[b].append(int(bonus[b]))
            self.prefix_len_host[[b, self.w.B + b]] += plen[b] + 1
        self.roots = bonus.copy()
        return dict(tok=tok, draft_p=p, uniforms=u, u_bonus=ub, path_len=plen, path_nodes=nodes, bonus=bonus)

    def close(self):
        self.tree.close()
        self.ctx.close()
