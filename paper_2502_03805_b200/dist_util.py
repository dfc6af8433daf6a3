"""Multi-rank bookkeeping for the benchmark: which layers a rank owns and the max-over-ranks time.

The compression of one layer is independent of every other layer, so ranks share nothing on the data path; the only
exchanges are a barrier and one MAX all-reduce of the measured time.

A single layer can also be split over ranks by KV head (the tensor-parallel layout of the model around it); then the
flattened adaptive budget allocation needs one all-gather of the group attention scores (ShardedCompressor).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_layer_ids(rank: int, layers_per_rank: int):
    """Seeds of the layers rank `rank` generates: disjoint across ranks, `layers_per_rank` each (weak scaling)."""
    return list(range(rank * layers_per_rank, (rank + 1) * layers_per_rank))


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a host scalar (identity when torch.distributed is not initialised)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank: int, world: int, seconds_max: float) -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return units_per_rank * world / seconds_max


def shard_kv_heads(Hkv: int, world: int, rank: int):
    """KV heads [g0, g1) owned by `rank` when a layer's Hkv heads are split evenly over `world` ranks."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside world of {world}")
    if Hkv % world != 0:
        raise ValueError(f"Hkv={Hkv} is not divisible by world size {world}")
    per = Hkv // world
    return rank * per, (rank + 1) * per


def all_gather_heads(a_local: torch.Tensor) -> torch.Tensor:
    """Concatenates the per-rank [nb, Hkv_local, n] tensors along the head axis in rank order (identity without
    torch.distributed).  The only exchange the sharded path needs: Hkv * n floats per layer."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return a_local
    parts = [torch.empty_like(a_local) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, a_local.contiguous())
    return torch.cat(parts, dim=1)


def local_budget_slice(budgets: torch.Tensor, Hkv: int, world: int, rank: int) -> torch.Tensor:
    """The columns of budgets[nb, Hkv] (the allocation every rank computes on the gathered scores) that belong to the
    KV heads of `rank`, as a contiguous [nb, Hkv / world] tensor for criticalkv_select in given-budget mode."""
    g0, g1 = shard_kv_heads(Hkv, world, rank)
    return budgets[:, g0:g1].contiguous()


class ShardedCompressor:
    """Compression of a layer whose KV heads are split over ranks (a rank holds its KV heads, their query heads and
    their rows of W^O).  Uniform budgets need no communication; flattened adaptive budgets gather the group attention
    scores of all heads once, and every rank repeats the cheap allocation on the gathered scores."""

    def __init__(self, *, nb, Hq, Hkv, dh, dm, n, w, pool_k, dtype, budget_mode, budget, world, rank, alpha=0.5,
                 eps=1e-4, device=0, gather=all_gather_heads, flags=0, adaptive_floor=0.0, norm=0):
        from . import binding as B
        from .session import CompressionSession
        self.B = B
        self.g0, self.g1 = shard_kv_heads(Hkv, world, rank)
        self.Hkv, self.world, self.rank = Hkv, world, rank
        G = Hq // Hkv
        hkv_loc = self.g1 - self.g0
        self.global_desc = B.make_desc(nb=nb, Hq=Hq, Hkv=Hkv, dh=dh, dm=dm, n=n, w=w, pool_k=pool_k, dtype=dtype,
                                       budget_mode=budget_mode, budget=budget, alpha=alpha, eps=eps, flags=flags,
                                       adaptive_floor=adaptive_floor, norm=norm)
        self.adaptive = budget_mode == "adaptive"
        local_mode = "given" if self.adaptive else budget_mode
        local_budget = min(budget, hkv_loc * n) if self.adaptive else budget   # capacity of the local outputs
        self.session = CompressionSession(nb=nb, Hq=hkv_loc * G, Hkv=hkv_loc, dh=dh, dm=dm, n=n, w=w, pool_k=pool_k,
                                          dtype=dtype, budget_mode=local_mode, budget=local_budget, alpha=alpha,
                                          eps=eps, device=device, flags=flags, norm=norm)
        self.gather = gather
        dev = self.session.device
        self.a_local = torch.empty((nb, hkv_loc, n), dtype=torch.float32, device=dev)
        self.budgets = torch.empty((nb, Hkv), dtype=torch.int32, device=dev)

    def group_scores(self, stream=None):
        s = self.session
        self.B.criticalkv_group_scores(s.handle, s.desc, s.attn, s.vnorm, self.a_local, None, stream=stream)
        return self.a_local

    def compress(self, Qw, K, V, WO, stream=None):
        """Local shards: Qw [nb, Hq_loc, w, dh], K, V [nb, Hkv_loc, n, dh], WO [nb, Hq_loc, dh, dm]."""
        s, B = self.session, self.B
        s.score(Qw, K, V, WO, stream=stream)
        local_budgets = None
        if self.adaptive:
            # the gather and the slice are torch operations: they must run on the stream the library calls use,
            # otherwise they could read the scores or the budgets before the kernels have written them
            ctx = torch.cuda.stream(stream) if stream is not None and a_is_cuda(self.a_local) else _NullCtx()
            with ctx:
                a_all = self.gather(self.group_scores(stream=stream))
                B.criticalkv_allocate_budgets(s.handle, self.global_desc, a_all, self.budgets, stream=stream)
                local_budgets = local_budget_slice(self.budgets, self.Hkv, self.world, self.rank)
        s.select(budgets_in=local_budgets, stream=stream)
        s.compact(K, V, stream=stream)
        return s


class _NullCtx:
    def __enter__(self):
        return self

    def __exit__(self, *exc):
        return False


def a_is_cuda(t) -> bool:
    return bool(getattr(t, "is_cuda", False))
