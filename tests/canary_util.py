"""Guarded device buffers for the GPU tests: every buffer handed to the library sits between two guard zones filled
with a known byte, and the zones are verified after each call.  The stand-in for a memory checker on machines where
none can be run: a kernel that writes one element outside a buffer it was given changes a guard byte."""
from __future__ import annotations

import numpy as np
import torch

from paper_2502_03805_b200 import binding as B

GUARD = 256          # bytes on each side (keeps the interior 256-byte aligned)
FILL = 0xA5
_TORCH = {"f32": torch.float32, "bf16": torch.bfloat16}


class Guarded:
    """A tensor of `shape` / `dtype` carved out of a byte buffer with guard zones before and after it."""

    def __init__(self, shape, dtype, device="cuda", fill=None):
        nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.nbytes = nbytes
        padded = (nbytes + 255) // 256 * 256
        self.raw = torch.full((GUARD + padded + GUARD,), FILL, dtype=torch.uint8, device=device)
        inner = self.raw[GUARD:GUARD + nbytes]
        self.t = inner.view(dtype).reshape(shape) if nbytes else torch.empty(shape, dtype=dtype, device=device)
        if fill is not None and nbytes:
            self.t.fill_(fill)

    def intact(self) -> bool:
        head = self.raw[:GUARD]
        tail = self.raw[GUARD + self.nbytes:]
        return bool((head == FILL).all().item()) and bool((tail == FILL).all().item())


class GuardedSession:
    """The buffers of one problem shape, each with guard zones, and exactly the workspace sizes the library asks for
    (separate score and select workspaces, so an overrun of either is seen)."""

    def __init__(self, *, nb, Hq, Hkv, dh, dm, n, w, pool_k, dtype, budget_mode, budget, alpha=0.5, eps=1e-4,
                 flags=0, valid_from=None, adaptive_floor=0.0):
        self.desc = B.make_desc(nb=nb, Hq=Hq, Hkv=Hkv, dh=dh, dm=dm, n=n, w=w, pool_k=pool_k, dtype=dtype,
                                budget_mode=budget_mode, budget=budget, alpha=alpha, eps=eps, flags=flags,
                                valid_from=valid_from, adaptive_floor=adaptive_floor)
        self.valid_from = valid_from
        self.handle = B.criticalkv_create(0)
        self.btot = budget * Hkv if budget_mode == "uniform" else budget
        sb, tb = B.criticalkv_workspace_bytes(self.desc)
        cap = max(self.btot, 1)
        self.bufs = {
            "attn": Guarded((nb, Hq, n), torch.float32),
            "vnorm": Guarded((nb, Hq, n), torch.float32),
            "idx": Guarded((nb, cap), torch.int32, fill=-1),
            "offsets": Guarded((nb, Hkv + 1), torch.int32, fill=0),
            "stage": Guarded((nb, cap), torch.uint8, fill=0),
            "K_out": Guarded((nb, cap, dh), _TORCH[dtype], fill=0),
            "V_out": Guarded((nb, cap, dh), _TORCH[dtype], fill=0),
            "ws_score": Guarded((max(sb, 256),), torch.uint8),
            "ws_select": Guarded((max(tb, 256),), torch.uint8),
        }
        self.score_bytes, self.select_bytes = sb, tb

    def __getattr__(self, name):
        bufs = self.__dict__.get("bufs", {})
        if name in bufs:
            return bufs[name].t
        raise AttributeError(name)

    def close(self):
        if self.handle is not None:
            B.criticalkv_destroy(self.handle)
            self.handle = None

    def run(self, Qw, K, V, WO, budgets_in=None):
        """score, select, compact with the exact workspace sizes; returns the device status word."""
        b = self.bufs
        B.criticalkv_score(self.handle, self.desc, Qw, K, V, WO, b["attn"].t, b["vnorm"].t, b["ws_score"].t,
                           ws_bytes=self.score_bytes)
        B.criticalkv_select(self.handle, self.desc, b["attn"].t, b["vnorm"].t, budgets_in, b["idx"].t, b["offsets"].t,
                            b["stage"].t, b["ws_select"].t, ws_bytes=self.select_bytes)
        B.criticalkv_compact(self.handle, self.desc, K, V, b["idx"].t, b["offsets"].t, b["K_out"].t, b["V_out"].t)
        torch.cuda.synchronize()
        return B.criticalkv_device_status(self.handle)

    def damaged(self):
        """Names of the buffers whose guard zones changed."""
        return [k for k, g in self.bufs.items() if not g.intact()]
