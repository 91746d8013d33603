"""Thin ctypes binding of liblumo_gdn.so: argument marshalling only.

Every step of the path (tree conv, tree scan, commit) runs in the CUDA kernels behind the
C ABI declared in include/lumo_gdn.h; this module turns torch tensors into pointers and
error codes into exceptions.  It raises at import if the shared library is missing: there
is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblumo_gdn.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2609_23900_b200.build` "
        "(the GDN tree verifier has no CPU fallback)")
_lib = ctypes.CDLL(LIB_PATH)

LUMO_F32, LUMO_BF16 = 0, 1
_DTYPE = {torch.float32: LUMO_F32, torch.bfloat16: LUMO_BF16}

SEQ_OK, SEQ_BAD_LEN, SEQ_BAD_NODE, SEQ_BAD_ROOT, SEQ_BAD_LINK, SEQ_BAD_ROW, SEQ_TIMEOUT, SEQ_BAD_CTX = range(8)

TABLES = ["depth", "n_child", "child_off", "child_list", "is_leaf", "leaves", "path_off", "path_nodes",
          "anc_win", "slot_inv", "chain_head", "chain_off", "chain_nodes", "chain_level", "cut_nodes",
          "schedule", "schedule_full", "gram_groups", "attn_vis"]

KERNEL_KINDS = ["conv", "scan", "commit", "path", "attn", "attn_merge", "kv_write", "kv_publish"]

EXPORTS = ["lumo_ctx_create", "lumo_ctx_destroy", "lumo_last_error", "lumo_ctx_scratch_bytes",
           "lumo_ctx_timing_enable", "lumo_ctx_timing_read", "lumo_ctx_set_scan_algo", "lumo_ctx_set_overlap", "lumo_ctx_set_timeout_drill",
           "lumo_tree_desc_create", "lumo_tree_desc_destroy", "lumo_tree_desc_get",
           "lumo_tree_path_from_node", "lumo_gdn_tree_verify", "lumo_gdn_commit",
           "lumo_gdn_tree_scan_static", "lumo_static_stack_bytes", "lumo_conv_rows_per_cta", "lumo_tree_accept", "lumo_select_spine_top3", "lumo_gdn_commit_verify",
           "lumo_kv_write_tree", "lumo_tree_attention", "lumo_kv_publish"]


class LumoError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"lumo status {code}: {msg}")
        self.code = code


class _Args(ctypes.Structure):
    """Mirror of lumo_gdn_args."""
    _fields_ = [
        ("Hk", ctypes.c_int32), ("Hv", ctypes.c_int32), ("d", ctypes.c_int32),
        ("in_dtype", ctypes.c_int32), ("gate_dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
        ("scale", ctypes.c_float), ("qk_l2norm", ctypes.c_int32), ("l2_eps", ctypes.c_float),
        ("n_state_rows", ctypes.c_int32),
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("alpha", ctypes.c_void_p), ("beta", ctypes.c_void_p),
        ("x", ctypes.c_void_p), ("conv_w", ctypes.c_void_p), ("conv_b", ctypes.c_void_p),
        ("conv_hist", ctypes.c_void_p),
        ("state", ctypes.c_void_p), ("state_row", ctypes.c_void_p),
        ("out", ctypes.c_void_p),
        ("snapshot_mode", ctypes.c_int32), ("n_snap", ctypes.c_int32),
        ("snap_nodes", ctypes.c_void_p), ("snap_out", ctypes.c_void_p),
        ("status", ctypes.c_void_p),
        ("gate_mode", ctypes.c_int32), ("a_log", ctypes.c_void_p), ("dt_bias", ctypes.c_void_p),
    ]


class _AcceptArgs(ctypes.Structure):
    """Mirror of lumo_accept_args."""
    _fields_ = [("V", ctypes.c_int32), ("mode", ctypes.c_int32), ("token", ctypes.c_void_p),
                ("p_target", ctypes.c_void_p), ("q_draft", ctypes.c_void_p), ("uniforms", ctypes.c_void_p),
                ("noise", ctypes.c_void_p), ("work", ctypes.c_void_p)]


class _SelectArgs(ctypes.Structure):
    """Mirror of lumo_select_args."""
    _fields_ = [("rows", ctypes.c_int32), ("V", ctypes.c_int32), ("dtype", ctypes.c_int32), ("split", ctypes.c_int32),
                ("logits", ctypes.c_void_p)]


class _AttnArgs(ctypes.Structure):
    """Mirror of lumo_attn_args."""
    _fields_ = [("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("dh", ctypes.c_int32), ("scale", ctypes.c_float),
                ("n_cache_rows", ctypes.c_int32), ("max_positions", ctypes.c_int32),
                ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
                ("ctx_len", ctypes.c_void_p), ("cache_row", ctypes.c_void_p),
                ("q", ctypes.c_void_p), ("k_new", ctypes.c_void_p), ("v_new", ctypes.c_void_p),
                ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p),
                ("kv_layout", ctypes.c_int32), ("n_splits", ctypes.c_int32), ("status", ctypes.c_void_p)]


_lib.lumo_ctx_create.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_void_p)]
_lib.lumo_ctx_destroy.argtypes = [ctypes.c_void_p]
_lib.lumo_ctx_destroy.restype = None
_lib.lumo_last_error.argtypes = [ctypes.c_void_p]
_lib.lumo_last_error.restype = ctypes.c_char_p
_lib.lumo_ctx_scratch_bytes.argtypes = [ctypes.c_void_p]
_lib.lumo_ctx_scratch_bytes.restype = ctypes.c_int64
_lib.lumo_ctx_set_scan_algo.argtypes = [ctypes.c_void_p, ctypes.c_int]
_lib.lumo_ctx_set_overlap.argtypes = [ctypes.c_void_p, ctypes.c_int]
_lib.lumo_ctx_set_timeout_drill.argtypes = [ctypes.c_void_p, ctypes.c_int]
_lib.lumo_ctx_timing_enable.argtypes = [ctypes.c_void_p, ctypes.c_int]
_lib.lumo_ctx_timing_read.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                      ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double)]
_lib.lumo_tree_desc_create.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.POINTER(ctypes.c_void_p)]
_lib.lumo_tree_desc_destroy.argtypes = [ctypes.c_void_p]
_lib.lumo_tree_desc_destroy.restype = None
_lib.lumo_tree_desc_get.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                    ctypes.POINTER(ctypes.POINTER(ctypes.c_int32)),
                                    ctypes.POINTER(ctypes.c_int64)]
_lib.lumo_tree_path_from_node.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
_lib.lumo_gdn_tree_verify.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(_Args), ctypes.c_int,
                                      ctypes.c_void_p]
_lib.lumo_gdn_tree_scan_static.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(_Args), ctypes.c_int,
                                           ctypes.c_void_p]
_lib.lumo_static_stack_bytes.restype = ctypes.c_int64
_lib.lumo_conv_rows_per_cta.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int]
_lib.lumo_gdn_commit_verify.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
_lib.lumo_select_spine_top3.argtypes = [ctypes.c_void_p, ctypes.POINTER(_SelectArgs), ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_void_p]
_lib.lumo_tree_accept.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(_AcceptArgs), ctypes.c_int,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
_lib.lumo_gdn_commit.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(_Args), ctypes.c_int,
                                 ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]


_lib.lumo_kv_write_tree.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(_AttnArgs), ctypes.c_int, ctypes.c_void_p]
_lib.lumo_tree_attention.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(_AttnArgs), ctypes.c_int, ctypes.c_void_p]
_lib.lumo_kv_publish.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(_AttnArgs), ctypes.c_int,
                                 ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("tensors passed to the library must be contiguous CUDA tensors")
    return t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class Context:
    """lumo_ctx: one per device."""

    def __init__(self, device: int = 0):
        h = ctypes.c_void_p()
        rc = _lib.lumo_ctx_create(int(device), ctypes.byref(h))
        if rc != 0:
            raise LumoError(rc, _lib.lumo_last_error(None).decode())
        self._h = h
        self.device = int(device)

    def _check(self, rc: int):
        if rc != 0:
            raise LumoError(rc, _lib.lumo_last_error(self._h).decode())

    @property
    def scratch_bytes(self) -> int:
        return _lib.lumo_ctx_scratch_bytes(self._h)

    def set_scan_algo(self, algo: str = "auto"):
        """"auto" | "rank1" | "gram" | "solve" | "direct" (Gram form with the closed-form tail) | "tensor" (the same with
        the output sum on the tensor core): which scan kernel verify uses."""
        self._check(_lib.lumo_ctx_set_scan_algo(self._h, {"auto": 0, "rank1": 1, "gram": 2, "solve": 3, "direct": 4, "tensor": 5}[algo]))

    def set_timeout_drill(self, on: bool):
        """Test aid: the tensor-core scan issues no tensor-core work, so its bounded wait runs out."""
        self._check(_lib.lumo_ctx_set_timeout_drill(self._h, int(on)))

    def set_overlap(self, on: bool = True):
        """Programmatic dependent launch between conv, scan and commit (default on)."""
        self._check(_lib.lumo_ctx_set_overlap(self._h, int(on)))

    def timing_enable(self, on: bool = True):
        self._check(_lib.lumo_ctx_timing_enable(self._h, int(on)))

    def timing_read(self, reset: bool = True) -> dict:
        """{kernel kind: (launches, total device ms)} of the launches recorded since the last reset."""
        out = {}
        for i, name in enumerate(KERNEL_KINDS):
            n, ms = ctypes.c_int64(), ctypes.c_double()
            last = reset and i == len(KERNEL_KINDS) - 1
            self._check(_lib.lumo_ctx_timing_read(self._h, i, int(last), ctypes.byref(n), ctypes.byref(ms)))
            out[name] = (n.value, ms.value)
        return out

    def close(self):
        if self._h:
            _lib.lumo_ctx_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- entry points -------------------------------------------------------------------
    def tree_desc(self, parent, slot=None, n_slots: Optional[int] = None, depth=None) -> "TreeDesc":
        return TreeDesc(self, parent, slot, n_slots, depth)

    def path_from_node(self, desc: "TreeDesc", node: torch.Tensor, lmax: int, accepted: torch.Tensor,
                       length: torch.Tensor, status: Optional[torch.Tensor] = None, stream=None):
        self._check(_lib.lumo_tree_path_from_node(self._h, desc._h, _ptr(node), int(lmax), _ptr(accepted),
                                                  _ptr(length), _ptr(status), _stream(stream)))

    @staticmethod
    def pack(layers: Sequence["GdnLayer"]):
        """ctypes array of the layers' argument blocks (reusable across calls)."""
        return (_Args * len(layers))(*[l.args for l in layers])

    def verify(self, desc: "TreeDesc", layers, stream=None):
        arr = layers if isinstance(layers, ctypes.Array) else self.pack(layers)
        self._check(_lib.lumo_gdn_tree_verify(self._h, desc._h, arr, len(layers), _stream(stream)))

    def scan_static(self, desc: "TreeDesc", layers, stream=None):
        """The tree scan with the library's built-in, fixed-size stack: for callers that must not
        allocate device memory.  Scan only (no convolution); refuses shapes that need more stack than
        ``static_stack_bytes()``.  Calls that overlap on the GPU race on the shared stack."""
        arr = layers if isinstance(layers, ctypes.Array) else self.pack(layers)
        self._check(_lib.lumo_gdn_tree_scan_static(self._h, desc._h, arr, len(arr), _stream(stream)))

    def conv_rows_per_cta(self, desc: "TreeDesc", Hk: int, Hv: int, d: int, n_layers: int = 1) -> int:
        """Which instantiation of the tree convolution (16, 8 or 4 entries per CTA) this shape launches."""
        return int(_lib.lumo_conv_rows_per_cta(self._h, desc._h, int(Hk), int(Hv), int(d), int(n_layers)))

    @staticmethod
    def static_stack_bytes() -> int:
        return int(_lib.lumo_static_stack_bytes())

    def accept(self, desc: "TreeDesc", *, token, p_target, accepted, length, next_token, final_node,
               mode: str = "greedy", q_draft=None, uniforms=None, noise=None, work=None, stream=None):
        """Acceptance walk on the device: fills accepted [B, lmax], length, next_token, final_node."""
        a = _AcceptArgs()
        a.V, a.mode = int(p_target.shape[-1]), {"greedy": 0, "rejection": 1}[mode]
        for name, t in (("token", token), ("p_target", p_target), ("q_draft", q_draft), ("uniforms", uniforms),
                        ("noise", noise), ("work", work)):
            setattr(a, name, _ptr(t))
        self._check(_lib.lumo_tree_accept(self._h, desc._h, ctypes.byref(a), int(accepted.shape[1]), _ptr(accepted),
                                          _ptr(length), _ptr(next_token), _ptr(final_node), _stream(stream)))

    def commit_verify(self, prev_desc: "TreeDesc", prev_layers, accepted: torch.Tensor, length: torch.Tensor,
                      desc: "TreeDesc", layers, stream=None):
        """commit(prev_desc, prev_layers, accepted, length) then verify(desc, layers), the state read once."""
        parr = prev_layers if isinstance(prev_layers, ctypes.Array) else self.pack(prev_layers)
        arr = layers if isinstance(layers, ctypes.Array) else self.pack(layers)
        self._check(_lib.lumo_gdn_commit_verify(self._h, prev_desc._h, parr, _ptr(accepted), _ptr(length),
                                                int(accepted.shape[1]), desc._h, arr, len(layers), _stream(stream)))

    def select_spine_top3(self, logits: torch.Tensor, spine: torch.Tensor, cand: torch.Tensor, split: int = 0,
                          stream=None):
        """Fused draft selection: spine [R] and cand [R, 3] (int32, device) from logits [R, V] (f32 or bf16)."""
        a = _SelectArgs()
        a.rows, a.V = int(logits.shape[0]), int(logits.shape[1])
        a.dtype = {torch.float32: 0, torch.bfloat16: 1}[logits.dtype]
        a.split = int(split)
        a.logits = _ptr(logits)
        self._check(_lib.lumo_select_spine_top3(self._h, ctypes.byref(a), _ptr(spine), _ptr(cand), _stream(stream)))

    def commit(self, desc: "TreeDesc", layers, accepted: torch.Tensor, length: torch.Tensor, stream=None):
        arr = layers if isinstance(layers, ctypes.Array) else self.pack(layers)
        self._check(_lib.lumo_gdn_commit(self._h, desc._h, arr, len(layers), _ptr(accepted), _ptr(length),
                                         int(accepted.shape[1]), _stream(stream)))


    # ---- attention half ----
    @staticmethod
    def pack_attn(layers: Sequence["AttnLayer"]):
        return (_AttnArgs * len(layers))(*[l.args for l in layers])

    def kv_write_tree(self, desc: "TreeDesc", layers, stream=None):
        arr = layers if isinstance(layers, ctypes.Array) else self.pack_attn(layers)
        self._check(_lib.lumo_kv_write_tree(self._h, desc._h, arr, len(arr), _stream(stream)))

    def tree_attention(self, desc: "TreeDesc", layers, stream=None):
        arr = layers if isinstance(layers, ctypes.Array) else self.pack_attn(layers)
        self._check(_lib.lumo_tree_attention(self._h, desc._h, arr, len(arr), _stream(stream)))

    def kv_publish(self, desc: "TreeDesc", layers, accepted: torch.Tensor, length: torch.Tensor,
                   ctx_len_out: Optional[torch.Tensor] = None, stream=None):
        arr = layers if isinstance(layers, ctypes.Array) else self.pack_attn(layers)
        self._check(_lib.lumo_kv_publish(self._h, desc._h, arr, len(arr), _ptr(accepted), _ptr(length),
                                         int(accepted.shape[1]), _ptr(ctx_len_out), _stream(stream)))


class TreeDesc:
    """lumo_tree_desc built from host arrays parent [B, N] (and optional slot, depth)."""

    def __init__(self, ctx: Context, parent, slot=None, n_slots: Optional[int] = None, depth=None):
        parent = np.ascontiguousarray(parent, dtype=np.int32)
        if parent.ndim != 2:
            raise ValueError("parent must be [B, N]")
        self.B, self.N = parent.shape
        slot_a = None if slot is None else np.ascontiguousarray(slot, dtype=np.int32)
        depth_a = None if depth is None else np.ascontiguousarray(depth, dtype=np.int32)
        self.Ns = int(n_slots) if n_slots is not None else self.N
        h = ctypes.c_void_p()
        rc = _lib.lumo_tree_desc_create(
            ctx._h, self.B, self.N, self.Ns, parent.ctypes.data,
            None if depth_a is None else depth_a.ctypes.data,
            None if slot_a is None else slot_a.ctypes.data, ctypes.byref(h))
        ctx._check(rc)
        self._h = h
        self._ctx = ctx

    def table(self, name: str, b: int = 0) -> np.ndarray:
        data = ctypes.POINTER(ctypes.c_int32)()
        count = ctypes.c_int64()
        rc = _lib.lumo_tree_desc_get(self._h, TABLES.index(name), int(b), ctypes.byref(data), ctypes.byref(count))
        if rc != 0:
            raise LumoError(rc, "bad table request")
        return np.ctypeslib.as_array(data, shape=(count.value,)).copy() if count.value else np.zeros(0, np.int32)

    def close(self):
        if self._h:
            _lib.lumo_tree_desc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class GdnLayer:
    """lumo_gdn_args for one layer; keeps the tensors alive."""

    def __init__(self, *, Hk: int, Hv: int, d: int, q, k, v, alpha, beta, state, state_row, out=None,
                 x=None, conv_w=None, conv_b=None, conv_hist=None, scale: float = 1.0,
                 qk_l2norm: bool = False, l2_eps: float = 1e-6, snapshot_mode: int = 0, snap_nodes=None,
                 snap_out=None, status=None, a_log=None, dt_bias=None):
        """a_log and dt_bias ([Hv] float32) switch to raw gate inputs: alpha and beta are then activated in
        the kernels."""
        self.tensors = dict(q=q, k=k, v=v, alpha=alpha, beta=beta, state=state, state_row=state_row, out=out,
                            x=x, conv_w=conv_w, conv_b=conv_b, conv_hist=conv_hist, snap_nodes=snap_nodes,
                            snap_out=snap_out, status=status, a_log=a_log, dt_bias=dt_bias)
        if (a_log is None) != (dt_bias is None):
            raise ValueError("a_log and dt_bias go together")
        for t in (a_log, dt_bias):
            if t is not None and t.dtype != torch.float32:
                raise ValueError("a_log and dt_bias must be float32")
        if state.dtype != torch.float32:
            raise ValueError("state must be float32")
        for name in ("state_row", "snap_nodes", "status"):
            t = self.tensors[name]
            if t is not None and t.dtype != torch.int32:
                raise ValueError(f"{name} must be int32")
        if alpha.dtype != beta.dtype or q.dtype != k.dtype or q.dtype != v.dtype:
            raise ValueError("q/k/v (and alpha/beta) must share a dtype")
        for name in ("x", "conv_w", "conv_b", "conv_hist"):
            t = self.tensors[name]
            if t is not None and t.dtype != q.dtype:
                raise ValueError(f"{name} must have the dtype of q/k/v")
        a = _Args()
        a.Hk, a.Hv, a.d = Hk, Hv, d
        a.in_dtype = _DTYPE[q.dtype]
        a.gate_dtype = _DTYPE[alpha.dtype]
        a.out_dtype = _DTYPE[out.dtype] if out is not None else LUMO_F32
        a.scale, a.qk_l2norm, a.l2_eps = float(scale), int(qk_l2norm), float(l2_eps)
        a.n_state_rows = int(state.shape[0])
        a.snapshot_mode = int(snapshot_mode)
        a.n_snap = int(snap_nodes.shape[1]) if snap_nodes is not None else 0
        a.gate_mode = 0 if a_log is None else 1
        for name in ("q", "k", "v", "alpha", "beta", "x", "conv_w", "conv_b", "conv_hist", "state",
                     "state_row", "out", "snap_nodes", "snap_out", "status", "a_log", "dt_bias"):
            setattr(a, name, _ptr(self.tensors[name]))
        self.args = a


class AttnLayer:
    """lumo_attn_args for one full-attention layer; keeps the tensors alive."""

    def __init__(self, *, Hq: int, Hkv: int, k_cache, v_cache, ctx_len, cache_row, scale: float, q=None, k_new=None,
                 v_new=None, out=None, lse=None, n_splits: int = 0, status=None, kv_layout: int = 0):
        """kv_layout 0: caches are [rows, positions, Hkv, dh]; 1: [rows, Hkv, positions, dh]."""
        self.tensors = dict(k_cache=k_cache, v_cache=v_cache, ctx_len=ctx_len, cache_row=cache_row, q=q, k_new=k_new,
                            v_new=v_new, out=out, lse=lse, status=status)
        if k_cache.dtype != torch.bfloat16 or v_cache.dtype != torch.bfloat16 or k_cache.shape != v_cache.shape:
            raise ValueError("k_cache and v_cache must be bfloat16 tensors of one shape [rows, positions, Hkv, dh]")
        if k_cache.dim() != 4 or k_cache.shape[1 if kv_layout else 2] != Hkv:
            raise ValueError("cache shape must be [rows, positions, Hkv, dh] (layout 0) or [rows, Hkv, positions, dh] (layout 1)")
        for name in ("q", "k_new", "v_new"):
            t = self.tensors[name]
            if t is not None and t.dtype != torch.bfloat16:
                raise ValueError(f"{name} must be bfloat16")
        for name in ("out", "lse"):
            t = self.tensors[name]
            if t is not None and t.dtype != torch.float32:
                raise ValueError(f"{name} must be float32")
        for name in ("ctx_len", "cache_row", "status"):
            t = self.tensors[name]
            if t is not None and t.dtype != torch.int32:
                raise ValueError(f"{name} must be int32")
        a = _AttnArgs()
        a.Hq, a.Hkv, a.dh, a.scale = int(Hq), int(Hkv), int(k_cache.shape[3]), float(scale)
        a.n_cache_rows, a.max_positions = int(k_cache.shape[0]), int(k_cache.shape[2 if kv_layout else 1])
        a.n_splits = int(n_splits)
        a.kv_layout = int(kv_layout)
        for name in self.tensors:
            setattr(a, name, _ptr(self.tensors[name]))
        self.args = a
