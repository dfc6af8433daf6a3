"""Device-buffer plumbing around the C ABI: allocates outputs and workspace with torch and forwards to the binding.

No step of the method runs here; every tensor is produced by the kernels of libcriticalkv.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B

_TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}


def to_device(store: np.ndarray, dtype: str, device="cuda:0") -> torch.Tensor:
    """Upload a stored array (float32, or uint16 bfloat16 bit patterns) without changing a bit."""
    t = torch.from_numpy(np.ascontiguousarray(store))
    if dtype == "bf16":
        t = t.view(torch.bfloat16)
    return t.to(device)


def to_host(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


class CompressionSession:
    """Holds a handle, a descriptor and the device buffers of one problem shape."""

    def __init__(self, *, nb, Hq, Hkv, dh, dm, n, w, pool_k, dtype, budget_mode, budget, alpha=0.5, eps=1e-4,
                 scale=0.0, flags=0, device=0, want_stage=True, adaptive_floor=0.0, norm=0, valid_from=None):
        self.device = torch.device("cuda", device)
        self.dtype = dtype
        self.desc = B.make_desc(nb=nb, Hq=Hq, Hkv=Hkv, dh=dh, dm=dm, n=n, w=w, pool_k=pool_k, dtype=dtype,
                                budget_mode=budget_mode, budget=budget, alpha=alpha, eps=eps, scale=scale,
                                flags=flags, adaptive_floor=adaptive_floor, norm=norm, valid_from=valid_from)
        self.valid_from = valid_from   # keeps the device array alive
        self.handle = B.criticalkv_create(device)
        self.btot = budget * Hkv if budget_mode == "uniform" else budget
        sb, tb = B.criticalkv_workspace_bytes(self.desc)
        dev = self.device
        self.score_bytes, self.select_bytes = sb, tb
        self.ws = torch.empty(max(sb, tb, 256), dtype=torch.uint8, device=dev)
        self.attn = torch.empty((nb, Hq, n), dtype=torch.float32, device=dev)
        self.vnorm = torch.empty((nb, Hkv if flags & B.CKV_FLAG_WO_GROUP_SUM else Hq, n), dtype=torch.float32,
                                 device=dev)
        self.idx = torch.full((nb, max(self.btot, 1)), -1, dtype=torch.int32, device=dev)
        self.offsets = torch.zeros((nb, Hkv + 1), dtype=torch.int32, device=dev)
        self.stage = torch.zeros((nb, max(self.btot, 1)), dtype=torch.uint8, device=dev) if want_stage else None
        self.K_out = torch.zeros((nb, max(self.btot, 1), dh), dtype=_TORCH_DTYPE[dtype], device=dev)
        self.V_out = torch.zeros_like(self.K_out)

    def close(self):
        if self.handle is not None:
            B.criticalkv_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def score(self, Qw, K, V, WO, stream=None):
        return B.criticalkv_score(self.handle, self.desc, Qw, K, V, WO, self.attn, self.vnorm, self.ws,
                                  stream=stream)

    def select(self, attn=None, vnorm=None, budgets_in=None, stream=None):
        return B.criticalkv_select(self.handle, self.desc, self.attn if attn is None else attn,
                                   self.vnorm if vnorm is None else vnorm, budgets_in, self.idx, self.offsets,
                                   self.stage, self.ws, stream=stream)

    def compact(self, K, V, stream=None):
        return B.criticalkv_compact(self.handle, self.desc, K, V, self.idx, self.offsets, self.K_out, self.V_out,
                                    stream=stream)

    def compress(self, Qw, K, V, WO, budgets_in=None, stream=None):
        return B.criticalkv_compress(self.handle, self.desc, Qw, K, V, WO, budgets_in, self.attn, self.vnorm,
                                     self.idx, self.offsets, self.stage, self.K_out, self.V_out, self.ws,
                                     stream=stream)

    def device_status(self, stream=None):
        return B.criticalkv_device_status(self.handle, stream)

    @property
    def launches(self):
        return B.criticalkv_launch_count(self.handle)

    @property
    def last_path(self):
        return B.criticalkv_last_path(self.handle)


def session_for(wl, nb=1, **kw) -> CompressionSession:
    """Session for a gen.Workload-like object (fields Hq, Hkv, dh, dm, n, w, kp, dtype, budget_mode, budget, ...)."""
    return CompressionSession(nb=nb, Hq=wl.Hq, Hkv=wl.Hkv, dh=wl.dh, dm=wl.dm, n=wl.n, w=wl.w, pool_k=wl.kp,
                              dtype=wl.dtype, budget_mode=wl.budget_mode, budget=wl.budget, alpha=wl.alpha,
                              eps=wl.eps, **kw)


class ChunkedPrefillCompressor:
    """Chunked prefill with eviction between chunks: keeps the retained K, V and their original token positions on
    the device; every step appends a chunk, calls criticalkv_compress on [retained ; chunk] and keeps the rows the
    library selected.  Only buffer concatenation and reshaping happen here.

    budget_mode "uniform": `budget` entries per KV head; K, V [Hkv, budget, dh] and pos [Hkv, budget] afterwards.
    budget_mode "adaptive": `budget` entries per layer, shared out by the flattened allocation; the heads then keep
    different numbers of entries, so K, V and pos are per-head lists and the next step passes the ragged cache
    right-aligned with the descriptor's valid_from offsets."""

    def __init__(self, *, Hq, Hkv, dh, dm, w, pool_k, dtype, alpha=0.5, eps=1e-4, scale=0.0, flags=0, device=0,
                 budget_mode="uniform"):
        if budget_mode not in ("uniform", "adaptive"):
            raise ValueError(budget_mode)
        self.kw = dict(Hq=Hq, Hkv=Hkv, dh=dh, dm=dm, w=w, pool_k=pool_k, dtype=dtype, alpha=alpha, eps=eps,
                       scale=scale, flags=flags, device=device)
        self.Hkv, self.dh = Hkv, dh
        self.budget_mode = budget_mode
        self.device = torch.device("cuda", device)
        self.K = self.V = self.pos = None
        self.seen = 0
        self.last = None   # adaptive mode: the padded inputs of the last step (for inspection)

    def step(self, Qw, K_chunk, V_chunk, WO, budget):
        """Qw [Hq,w,dh] (last w queries of the chunk), K_chunk, V_chunk [Hkv,len,dh], WO [Hq,dh,dm]: device tensors.
        Compresses [retained ; chunk] to `budget` entries (per KV head, or per layer with adaptive budgets).
        Returns the session used (its attn, vnorm, idx are valid until the next step)."""
        if self.budget_mode == "adaptive":
            return self._step_adaptive(Qw, K_chunk, V_chunk, WO, int(budget))
        ln = K_chunk.shape[1]
        new_pos = torch.arange(self.seen, self.seen + ln, dtype=torch.int32, device=self.device).expand(self.Hkv, ln)
        if self.K is None:
            Kc, Vc, pc = K_chunk.contiguous(), V_chunk.contiguous(), new_pos.contiguous()
        else:
            Kc = torch.cat([self.K, K_chunk], dim=1)
            Vc = torch.cat([self.V, V_chunk], dim=1)
            pc = torch.cat([self.pos, new_pos], dim=1).contiguous()
        self.seen += ln
        s = CompressionSession(nb=1, n=Kc.shape[1], budget_mode="uniform", budget=int(budget), want_stage=False,
                               **self.kw)
        s.compress(Qw, Kc, Vc, WO)
        pos_out = torch.empty((1, max(s.btot, 1)), dtype=torch.int32, device=self.device)
        B.criticalkv_gather_positions(s.handle, s.desc, pc, s.idx, s.offsets, pos_out)
        self.K = s.K_out[0, : s.btot].reshape(self.Hkv, int(budget), self.dh)
        self.V = s.V_out[0, : s.btot].reshape(self.Hkv, int(budget), self.dh)
        self.pos = pos_out[0, : s.btot].reshape(self.Hkv, int(budget))
        return s

    def _step_adaptive(self, Qw, K_chunk, V_chunk, WO, budget):
        Hkv, ln = self.Hkv, K_chunk.shape[1]
        kept = [0] * Hkv if self.K is None else [int(k.shape[0]) for k in self.K]
        n_max = max(kept) + ln
        if budget > sum(kept) + Hkv * ln:
            raise ValueError("budget exceeds the entries the cache holds")
        # every head right-aligned in a buffer of n_max rows: [padding ; retained ; chunk]
        Kc = torch.zeros((Hkv, n_max, self.dh), dtype=K_chunk.dtype, device=self.device)
        Vc = torch.zeros_like(Kc)
        pc = torch.full((Hkv, n_max), -1, dtype=torch.int32, device=self.device)
        new_pos = torch.arange(self.seen, self.seen + ln, dtype=torch.int32, device=self.device)
        for g in range(Hkv):
            lo = n_max - ln - kept[g]
            if kept[g]:
                Kc[g, lo:n_max - ln] = self.K[g]
                Vc[g, lo:n_max - ln] = self.V[g]
                pc[g, lo:n_max - ln] = self.pos[g]
            Kc[g, n_max - ln:] = K_chunk[g]
            Vc[g, n_max - ln:] = V_chunk[g]
            pc[g, n_max - ln:] = new_pos
        valid_from = torch.tensor([[n_max - ln - k for k in kept]], dtype=torch.int32, device=self.device)
        self.seen += ln
        s = CompressionSession(nb=1, n=n_max, budget_mode="adaptive", budget=budget, valid_from=valid_from, **self.kw)
        s.compress(Qw, Kc, Vc, WO)
        pos_out = torch.empty((1, max(s.btot, 1)), dtype=torch.int32, device=self.device)
        B.criticalkv_gather_positions(s.handle, s.desc, pc, s.idx, s.offsets, pos_out)
        off = s.offsets[0].tolist()          # the per-head counts size the next step's buffers
        self.K = [s.K_out[0, off[g]:off[g + 1]].clone() for g in range(Hkv)]
        self.V = [s.V_out[0, off[g]:off[g + 1]].clone() for g in range(Hkv)]
        self.pos = [pos_out[0, off[g]:off[g + 1]].clone() for g in range(Hkv)]
        self.last = dict(K=Kc, V=Vc, pos=pc, valid_from=valid_from, n=n_max)
        return s
