"""Thin ctypes binding of libcascade.so (the C ABI declared in include/cascade.h).

Argument marshalling only: every step of the verification path runs inside the library's CUDA
kernels.  Tensors are torch tensors used as device (or pinned host) memory; their data pointers and
the current CUDA stream are passed straight through.  If the shared library is missing the import of
`lib()` raises: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcascade.so")

OK = 0
ERR_INVALID_ARG, ERR_BAD_TREE, ERR_WORKSPACE, ERR_UNSUPPORTED_SHAPE, ERR_CUDA, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6
ERR_OVERFLOW = -7
F32, BF16 = 0, 1
USE_I, USE_C, CONV_DIST_SELF = 1, 2, 4
SELECT_LONGEST, SELECT_FIRST_ACCEPT = 0, 1
KERNEL_COUNT = 32

EXPORTS = [
    "cascade_create", "cascade_destroy", "cascade_workspace_bytes", "cascade_check", "cascade_last_launch_count",
    "cascade_strerror", "cascade_timing_enable", "cascade_timing_read", "cascade_kernel_name", "cascade_tree_create", "cascade_tree_destroy", "cascade_tree_update", "cascade_tree_rows", "cascade_tree_depth",
    "cascade_tree_num_pairs", "cascade_tree_pairs", "cascade_tree_attn", "cascade_lm_head_cfg",
    "cascade_similarity", "cascade_relaxed_accept", "cascade_select_path", "cascade_verify_step",
    "cascade_verify_step_host", "cascade_accept_static", "cascade_bonus_token", "cascade_kv_append",
    "cascade_filter_logits", "cascade_set_wait_limit", "cascade_wait_probe",
    "cascade_tree_update_device", "cascade_tree_download", "cascade_drafter_loss",
]


class Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("dtype", "B", "T_max", "P_max", "h", "Hq", "Hkv", "D", "V", "ffn")]


class Params(C.Structure):
    _fields_ = [("tau_pos", C.c_float), ("tau_seq", C.c_float), ("tvd_budget", C.c_float), ("flags", C.c_uint32)]


class Layer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("gamma_attn", "wq", "wk", "wv", "wo", "gamma_mlp", "w_gate", "w_up",
                                          "w_down", "k_prefix", "v_prefix")]


class Step(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("layers", C.POINTER(Layer)), ("embed", C.c_void_p), ("gamma_final", C.c_void_p),
        ("w_head", C.c_void_p), ("prefix_cap", C.c_int32), ("prefix_len", C.c_void_p),
        ("eps", C.c_float), ("rope_base", C.c_float), ("softmax_scale", C.c_float), ("cfg_scale", C.c_float),
        ("temperature", C.c_float),
        ("tok", C.c_void_p), ("draft_p", C.c_void_p), ("uniforms", C.c_void_p), ("hidden_in", C.c_void_p),
        ("q", C.c_void_p), ("k_tree", C.c_void_p), ("v_tree", C.c_void_p), ("k_prefix", C.c_void_p),
        ("v_prefix", C.c_void_p), ("attn_out", C.c_void_p),
        ("params", Params), ("select_mode", C.c_int32),
        ("accept", C.c_void_p), ("path_nodes", C.c_void_p), ("path_len", C.c_void_p), ("q_relaxed", C.c_void_p),
        ("tvd_out", C.c_void_p), ("tvd_used", C.c_void_p), ("near_count", C.c_void_p),
        ("logits", C.c_void_p), ("feat", C.c_void_p), ("scores", C.c_void_p), ("row_lse", C.c_void_p),
        ("hidden_out", C.c_void_p), ("k_tree_out", C.c_void_p), ("v_tree_out", C.c_void_p),
        ("top_k", C.c_int32), ("top_p", C.c_float),
    ]


_lib = None


def lib() -> C.CDLL:
    """Load libcascade.so (once).  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it first (python -m paper_2605_07230_b200.build)")
        L = C.CDLL(LIB_PATH)
        L.cascade_strerror.restype = C.c_char_p
        L.cascade_workspace_bytes.restype = C.c_int64
        vp = C.c_void_p
        L.cascade_create.argtypes = [C.POINTER(vp), C.POINTER(Shape)]
        L.cascade_destroy.argtypes = [vp]
        L.cascade_workspace_bytes.argtypes = [vp]
        L.cascade_check.argtypes = [vp, vp]
        L.cascade_last_launch_count.argtypes = [vp]
        L.cascade_timing_enable.argtypes = [vp, C.c_int32]
        L.cascade_timing_read.argtypes = [vp, vp, vp]
        L.cascade_kernel_name.argtypes = [C.c_int32]
        L.cascade_kernel_name.restype = C.c_char_p
        L.cascade_tree_create.argtypes = [vp, C.c_int32, vp, C.POINTER(vp)]
        L.cascade_tree_destroy.argtypes = [vp]
        L.cascade_tree_update.argtypes = [vp, C.c_int32, vp, vp]
        for f in ("cascade_tree_rows", "cascade_tree_depth", "cascade_tree_num_pairs"):
            getattr(L, f).argtypes = [vp]
        L.cascade_tree_pairs.argtypes = [vp, vp, vp]
        L.cascade_tree_attn.argtypes = [vp, vp, vp, vp, vp, C.c_int32, vp, vp, vp, vp, C.c_float, vp]
        L.cascade_lm_head_cfg.argtypes = [vp, vp, vp, vp, C.c_float, vp, C.c_float, C.c_float, vp, vp, vp, vp, vp,
                                          vp, vp, vp]
        L.cascade_similarity.argtypes = [vp, vp, vp, C.c_int32, vp, vp, vp]
        L.cascade_relaxed_accept.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, C.POINTER(Params), vp, vp, vp,
                                             vp, vp]
        L.cascade_select_path.argtypes = [vp, vp, vp, vp, C.c_int32, vp, vp, vp, vp]
        L.cascade_verify_step.argtypes = [vp, vp, C.POINTER(Step), vp]
        L.cascade_verify_step_host.argtypes = [vp, vp, C.POINTER(Step), vp, vp, vp, vp, vp, vp, vp]
        L.cascade_accept_static.argtypes = [C.c_int32, C.c_int32, vp, vp, C.c_int32, vp, vp, vp, vp, vp, vp, vp,
                                            C.POINTER(Params), C.c_int32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.cascade_bonus_token.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.cascade_kv_append.argtypes = [vp, vp, C.c_int32, C.POINTER(Layer), vp, vp, vp, vp, C.c_int32, vp, vp]
        L.cascade_filter_logits.argtypes = [vp, vp, C.c_int32, C.c_int32, C.c_float, vp, vp]
        L.cascade_tree_update_device.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, vp, vp]
        L.cascade_tree_download.argtypes = [vp, vp, vp, vp, vp, vp]
        L.cascade_drafter_loss.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_float, vp, vp, vp, vp]
        L.cascade_set_wait_limit.argtypes = [vp, C.c_int64]
        L.cascade_wait_probe.argtypes = [vp, vp, vp]
        _lib = L
    return _lib


class CascadeError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"cascade status {status}: {lib().cascade_strerror(status).decode()}")


def _check(status: int) -> None:
    if status != OK:
        raise CascadeError(status)


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors must be contiguous"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Context:
    """cascade_create / cascade_destroy."""

    def __init__(self, dtype: int, B: int, T_max: int, P_max: int, h: int, Hq: int, Hkv: int, D: int, V: int,
                 ffn: int = 0):
        self.shape = Shape(dtype, B, T_max, P_max, h, Hq, Hkv, D, V, ffn)
        self.handle = C.c_void_p()
        _check(lib().cascade_create(C.byref(self.handle), C.byref(self.shape)))

    def close(self):
        if self.handle:
            lib().cascade_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def workspace_bytes(self) -> int:
        return lib().cascade_workspace_bytes(self.handle)

    @property
    def last_launch_count(self) -> int:
        return lib().cascade_last_launch_count(self.handle)

    def check(self) -> None:
        _check(lib().cascade_check(self.handle, _stream()))

    def set_wait_limit(self, limit_ns: int) -> None:
        _check(lib().cascade_set_wait_limit(self.handle, int(limit_ns)))

    def wait_probe(self, waited_ns=None) -> None:
        """Enqueues the failure-path self-test (a wait that cannot end); check() raises ERR_TIMEOUT afterwards."""
        _check(lib().cascade_wait_probe(self.handle, _ptr(waited_ns), _stream()))

    def timing_enable(self, on: bool) -> None:
        _check(lib().cascade_timing_enable(self.handle, int(on)))

    def timing_read(self) -> dict:
        """{kernel name: (total ms, launches)} accumulated since the last read."""
        n = KERNEL_COUNT
        ms = (C.c_float * n)()
        cnt = (C.c_int32 * n)()
        _check(lib().cascade_timing_read(self.handle, ms, cnt))
        out = {}
        for i in range(n):
            name = lib().cascade_kernel_name(i)
            if name is not None and cnt[i] > 0:
                out[name.decode()] = (float(ms[i]), int(cnt[i]))
        return out


class Tree:
    """cascade_tree_create / cascade_tree_destroy.  `parent` is a host int32 sequence."""

    def __init__(self, ctx: Context, parent):
        self.ctx = ctx
        arr = (C.c_int32 * len(parent))(*[int(x) for x in parent])
        self.handle = C.c_void_p()
        _check(lib().cascade_tree_create(ctx.handle, len(parent), arr, C.byref(self.handle)))
        self.T = lib().cascade_tree_rows(self.handle)
        self.depth = lib().cascade_tree_depth(self.handle)
        self.num_pairs = lib().cascade_tree_num_pairs(self.handle)

    def update(self, parent):
        """A new tree in the same descriptor (no allocation); enqueued on the current stream."""
        arr = (C.c_int32 * len(parent))(*[int(x) for x in parent])
        _check(lib().cascade_tree_update(self.handle, len(parent), arr, _stream()))
        self.T = lib().cascade_tree_rows(self.handle)
        self.depth = lib().cascade_tree_depth(self.handle)
        self.num_pairs = lib().cascade_tree_num_pairs(self.handle)

    def update_device(self, T: int, depth_cap: int, pairs_cap: int, parent_dev):
        """A new tree from a device-resident int32 parent[] (no host round trip); enqueued on the current stream."""
        _check(lib().cascade_tree_update_device(self.handle, T, depth_cap, pairs_cap, _ptr(parent_dev), _stream()))
        self.T = lib().cascade_tree_rows(self.handle)
        self.depth = lib().cascade_tree_depth(self.handle)
        self.num_pairs = lib().cascade_tree_num_pairs(self.handle)

    def download(self):
        """The descriptor's device arrays as host lists: parent, depth, child_begin, child_count, anc (T x 4 words)."""
        T = self.T
        arrs = [(C.c_int32 * T)() for _ in range(4)]
        anc = (C.c_uint64 * (4 * T))()
        _check(lib().cascade_tree_download(self.handle, *arrs, anc))
        return [list(a) for a in arrs] + [[list(anc[4 * j: 4 * j + 4]) for j in range(T)]]

    def pairs(self):
        a = (C.c_int32 * max(self.num_pairs, 1))()
        b = (C.c_int32 * max(self.num_pairs, 1))()
        _check(lib().cascade_tree_pairs(self.handle, a, b))
        return list(a)[: self.num_pairs], list(b)[: self.num_pairs]

    def close(self):
        if self.handle:
            lib().cascade_tree_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def cascade_tree_attn(ctx, tree, q, k_prefix, v_prefix, prefix_cap, prefix_len, k_tree, v_tree, out, softmax_scale):
    _check(lib().cascade_tree_attn(ctx.handle, tree.handle, _ptr(q), _ptr(k_prefix), _ptr(v_prefix), prefix_cap,
                                   _ptr(prefix_len), _ptr(k_tree), _ptr(v_tree), _ptr(out), softmax_scale,
                                   _stream()))


def cascade_lm_head_cfg(ctx, tree, hidden, rms_gamma, eps, w_head, cfg_scale, temperature, tok, logits_out,
                        feat_out, feat_norm_out, row_lse_out, cand_parent_out, cand_gparent_out):
    _check(lib().cascade_lm_head_cfg(ctx.handle, tree.handle, _ptr(hidden), _ptr(rms_gamma), eps, _ptr(w_head),
                                     cfg_scale, temperature, _ptr(tok), _ptr(logits_out), _ptr(feat_out),
                                     _ptr(feat_norm_out), _ptr(row_lse_out), _ptr(cand_parent_out),
                                     _ptr(cand_gparent_out), _stream()))


def cascade_similarity(ctx, tree, feat, feat_dim, feat_norm, scores_out):
    _check(lib().cascade_similarity(ctx.handle, tree.handle, _ptr(feat), feat_dim, _ptr(feat_norm),
                                    _ptr(scores_out), _stream()))


def cascade_relaxed_accept(ctx, tree, scores, logits, row_lse, cand_parent, cand_gparent, tok, draft_p, uniforms,
                           params: Params, accept, q_relaxed, tvd_out, near_count):
    _check(lib().cascade_relaxed_accept(ctx.handle, tree.handle, _ptr(scores), _ptr(logits), _ptr(row_lse),
                                        _ptr(cand_parent), _ptr(cand_gparent), _ptr(tok), _ptr(draft_p),
                                        _ptr(uniforms), C.byref(params), _ptr(accept), _ptr(q_relaxed),
                                        _ptr(tvd_out), _ptr(near_count), _stream()))


def cascade_select_path(ctx, tree, accept, tvd_out, mode, path_nodes, path_len, tvd_used):
    _check(lib().cascade_select_path(ctx.handle, tree.handle, _ptr(accept), _ptr(tvd_out), mode, _ptr(path_nodes),
                                     _ptr(path_len), _ptr(tvd_used), _stream()))


def make_step(**kw) -> Step:
    """Fill a Step from keyword arguments; tensors become pointers, `layers` a list of dicts of tensors.
    The returned struct keeps references to everything it points to."""
    st = Step()
    keep = []
    layers = kw.pop("layers", None) or []
    st.n_layers = len(layers)
    if layers:
        arr = (Layer * len(layers))()
        for i, lw in enumerate(layers):
            for name, _ in Layer._fields_:
                setattr(arr[i], name, _ptr(lw[name]))
                keep.append(lw[name])
        st.layers = arr
        keep.append(arr)
    params = kw.pop("params")
    st.params = params
    for name, ctype in Step._fields_:
        if name in ("n_layers", "layers", "params"):
            continue
        if name not in kw:
            continue
        v = kw.pop(name)
        if ctype is C.c_void_p:
            setattr(st, name, _ptr(v))
            keep.append(v)
        else:
            setattr(st, name, v)
    assert not kw, f"unknown step fields: {sorted(kw)}"
    st._keep = keep
    return st


def cascade_verify_step(ctx, tree, step: Step):
    _check(lib().cascade_verify_step(ctx.handle, tree.handle, C.byref(step), _stream()))


def cascade_verify_step_host(ctx, tree, step: Step, tok_host, draft_p_host, uniforms_host, accept_host,
                             path_nodes_host, path_len_host):
    _check(lib().cascade_verify_step_host(ctx.handle, tree.handle, C.byref(step), _ptr(tok_host),
                                          _ptr(draft_p_host), _ptr(uniforms_host), _ptr(accept_host),
                                          _ptr(path_nodes_host), _ptr(path_len_host), _stream()))


def cascade_accept_static(B, parent, feat, feat_dim, feat_norm, row_lse, cand_parent, cand_gparent, tok, draft_p,
                          uniforms, params: Params, select_mode, accept, q_relaxed, tvd_out, near_count, path_nodes,
                          path_len, tvd_used):
    """Scores + relaxed acceptance + path selection with no context, no tree object and no device
    allocation (the library's static device array is the only scratch).  `parent` is a host sequence."""
    arr = (C.c_int32 * len(parent))(*[int(x) for x in parent])
    _check(lib().cascade_accept_static(B, len(parent), arr, _ptr(feat), feat_dim, _ptr(feat_norm), _ptr(row_lse),
                                       _ptr(cand_parent), _ptr(cand_gparent), _ptr(tok), _ptr(draft_p),
                                       _ptr(uniforms), C.byref(params), select_mode, _ptr(accept), _ptr(q_relaxed),
                                       _ptr(tvd_out), _ptr(near_count), _ptr(path_nodes), _ptr(path_len),
                                       _ptr(tvd_used), _stream()))


def cascade_filter_logits(ctx, logits, top_k, top_p, kept_count=None):
    n_rows = logits.numel() // logits.shape[-1]
    _check(lib().cascade_filter_logits(ctx.handle, _ptr(logits), n_rows, int(top_k), float(top_p), _ptr(kept_count),
                                       _stream()))


def cascade_bonus_token(ctx, tree, logits, tok, path_nodes, path_len, u_bonus, token_out, mass_out=None,
                        draft_row=None):
    _check(lib().cascade_bonus_token(ctx.handle, tree.handle, _ptr(logits), _ptr(tok), _ptr(draft_row),
                                     _ptr(path_nodes), _ptr(path_len), _ptr(u_bonus), _ptr(token_out),
                                     _ptr(mass_out), _stream()))


def cascade_kv_append(ctx, tree, step: Step, k_tree, v_tree, path_nodes, path_len, prefix_cap, prefix_len):
    """Appends the accepted path's rows to the caches named in `step.layers` (a Step made by make_step)."""
    _check(lib().cascade_kv_append(ctx.handle, tree.handle, step.n_layers, step.layers, _ptr(k_tree), _ptr(v_tree),
                                   _ptr(path_nodes), _ptr(path_len), prefix_cap, _ptr(prefix_len), _stream()))


def cascade_drafter_loss(target_logits, draft_logits, feat, tau_seq, c, loss_out, weight_out=None, total_out=None):
    """Eq. 4 of the paper on [K,V] target / drafter logits and [K,h] target hidden states (device tensors)."""
    K, V = target_logits.shape
    _check(lib().cascade_drafter_loss(_ptr(target_logits), _ptr(draft_logits), _ptr(feat), K, V, feat.shape[-1],
                                      float(tau_seq), float(c), _ptr(loss_out), _ptr(weight_out), _ptr(total_out),
                                      _stream()))
