"""Device-side holder of one synthetic case: uploads a ``workload.Case`` and builds the
per-layer argument blocks for the C-ABI calls.  Marshalling only; no arithmetic."""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from paper_2609_23900_b200 import binding
from .workload import Case

_TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16}


class DeviceCase:
    def __init__(self, ctx: binding.Context, case: Case, *, out_dtype: str = "f32", use_conv: bool = True,
                 gate_dtype: Optional[str] = None, snapshot_mode: int = 0, snap_nodes=None,
                 scale: float = 1.0, qk_l2norm: Optional[bool] = None, l2_eps: float = 1e-6,
                 device: Optional[torch.device] = None, pinned_host: bool = False, raw_gates=None):
        """raw_gates: optional list (one entry per layer) of dicts with host arrays alpha_in, beta_in
        [B, Ns, Hv] and a_log, dt_bias [Hv]; the layer then takes raw gate inputs instead of the case's
        post-activation gates."""
        self.ctx, self.case = ctx, case
        # conv outputs are not unit vectors: the pipeline normalises q, k inside the kernels
        # (Sec. "Sequential arithmetic and accepted-path replay": in-kernel query/key normalisation)
        qk_l2norm = use_conv if qk_l2norm is None else qk_l2norm
        self.scale, self.qk_l2norm, self.l2_eps = scale, qk_l2norm, l2_eps
        dev = device or torch.device("cuda", ctx.device)
        self.dev = dev
        dt = _TORCH_DT[case.in_dtype]
        gdt = _TORCH_DT[gate_dtype or case.in_dtype]
        odt = _TORCH_DT[out_dtype]
        self.desc = ctx.tree_desc(case.parent, slot=case.slot, n_slots=case.Ns)
        up = lambda a, t: torch.from_numpy(np.ascontiguousarray(a)).to(t).to(dev)
        self.state_row = torch.from_numpy(case.state_row.copy()).to(dev)
        self.accepted = torch.from_numpy(case.accepted.copy()).to(dev)
        self.accepted_len = torch.from_numpy(case.accepted_len.copy()).to(dev)
        self.snap_nodes = None
        E = 0
        if snapshot_mode == 1:
            self.snap_nodes = torch.from_numpy(np.ascontiguousarray(snap_nodes, dtype=np.int32)).to(dev)
            E = self.snap_nodes.shape[1]
        elif snapshot_mode == 2:
            E = case.N
        self.layers: List[binding.GdnLayer] = []
        self.host = []   # pinned host copies of the per-step inputs (end-to-end timing)
        for L in case.layers:
            t = dict(
                q=up(L.q, dt), k=up(L.k, dt), v=up(L.v, dt), alpha=up(L.alpha, gdt), beta=up(L.beta, gdt),
                state=up(L.state, torch.float32), state_row=self.state_row,
                out=torch.empty((case.B, case.Ns, case.Hv, case.d), dtype=odt, device=dev),
                status=torch.full((case.B,), -1, dtype=torch.int32, device=dev),
            )
            if raw_gates is not None:
                rg = raw_gates[len(self.layers)]
                t.update(alpha=up(rg["alpha_in"], gdt), beta=up(rg["beta_in"], gdt),
                         a_log=up(rg["a_log"], torch.float32), dt_bias=up(rg["dt_bias"], torch.float32))
            if use_conv:
                t.update(x=up(L.x, dt), conv_w=up(L.conv_w, dt), conv_hist=up(L.hist, dt),
                         conv_b=None if L.conv_b is None else up(L.conv_b, dt))
            if snapshot_mode:
                t.update(snap_nodes=self.snap_nodes,
                         snap_out=torch.zeros((case.B, E, case.Hv, case.d, case.d), dtype=torch.float32, device=dev))
            self.layers.append(binding.GdnLayer(Hk=case.Hk, Hv=case.Hv, d=case.d, scale=scale, qk_l2norm=qk_l2norm,
                                                l2_eps=l2_eps, snapshot_mode=snapshot_mode, **t))
            if pinned_host:
                self.host.append({n: t[n].cpu().pin_memory() for n in ("x", "alpha", "beta") if n in t})

    def verify(self, stream=None):
        self.ctx.verify(self.desc, self.layers, stream)

    def commit(self, accepted=None, length=None, stream=None):
        self.ctx.commit(self.desc, self.layers, self.accepted if accepted is None else accepted,
                        self.accepted_len if length is None else length, stream)

    def t(self, name: str, layer: int = 0) -> torch.Tensor:
        return self.layers[layer].tensors[name]

    def np(self, name: str, layer: int = 0) -> np.ndarray:
        """Host float64 (or int) copy of a device tensor."""
        t = self.t(name, layer)
        if t.dtype in (torch.float32, torch.bfloat16):
            return t.to(torch.float64).cpu().numpy()
        return t.cpu().numpy()


class DeviceAttnCase:
    """Device-side holder of one ``workload.AttnCase`` (one or more identical-shape layers that share the
    inputs of layer 0 unless ``cases`` lists one case per layer).  Marshalling only."""

    def __init__(self, ctx: binding.Context, case, *, n_splits: int = 0, cases=None, with_lse: bool = True,
                 device: Optional[torch.device] = None, kv_layout: int = 0):
        self.ctx, self.case = ctx, case
        self.cases = list(cases) if cases is not None else [case]
        dev = device or torch.device("cuda", ctx.device)
        self.dev = dev
        self.desc = ctx.tree_desc(case.parent, slot=case.slot, n_slots=case.Ns)
        up16 = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(dev)
        self.kv_layout = kv_layout
        # the case holds caches as [rows, positions, Hkv, dh]; layout 1 stores them head-major
        upc = lambda a: up16(a).permute(0, 2, 1, 3).contiguous() if kv_layout else up16(a)
        self.ctx_len = torch.from_numpy(case.ctx_len.copy()).to(dev)
        self.ctx_len_out = torch.full_like(self.ctx_len, -1)
        self.cache_row = torch.from_numpy(case.cache_row.copy()).to(dev)
        self.accepted = torch.from_numpy(case.accepted.copy()).to(dev)
        self.accepted_len = torch.from_numpy(case.accepted_len.copy()).to(dev)
        self.layers: List[binding.AttnLayer] = []
        for c in self.cases:
            self.layers.append(binding.AttnLayer(
                Hq=c.Hq, Hkv=c.Hkv, k_cache=upc(c.k_cache), v_cache=upc(c.v_cache), kv_layout=kv_layout, ctx_len=self.ctx_len,
                cache_row=self.cache_row, scale=c.scale, q=up16(c.q), k_new=up16(c.k_new), v_new=up16(c.v_new),
                out=torch.full((c.B, c.N, c.Hq, c.dh), float("nan"), dtype=torch.float32, device=dev),
                lse=torch.full((c.B, c.N, c.Hq), float("nan"), dtype=torch.float32, device=dev) if with_lse else None,
                n_splits=n_splits, status=torch.full((c.B,), -1, dtype=torch.int32, device=dev)))
        self.packed = ctx.pack_attn(self.layers)

    def t(self, name: str, layer: int = 0):
        return self.layers[layer].tensors[name]

    def np(self, name: str, layer: int = 0) -> np.ndarray:
        """Host copy in float64; caches always as [rows, positions, Hkv, dh], whatever the device layout."""
        t = self.t(name, layer)
        if self.kv_layout and name in ("k_cache", "v_cache"):
            t = t.permute(0, 2, 1, 3)
        return t.to(torch.float64).cpu().numpy() if t.is_floating_point() else t.cpu().numpy()

    def write(self, stream=None):
        self.ctx.kv_write_tree(self.desc, self.packed, stream)

    def attend(self, stream=None):
        self.ctx.tree_attention(self.desc, self.packed, stream)

    def publish(self, stream=None):
        self.ctx.kv_publish(self.desc, self.packed, self.accepted, self.accepted_len, self.ctx_len_out, stream)
