"""CPU oracle for the CriticalKV prefill-time compression step.

TEST INFRASTRUCTURE ONLY.  This file is a slow, plain NumPy restatement of the
method of "Optimizing KV Cache Eviction from an Output Perturbation
Perspective" (Algorithm 1, Algorithm 2, Eq. 2, Theorems 3.2 / 3.3 / 3.5 and the
relaxed-bound theorem of the appendix).  It exists to check the CUDA library;
it shares no code with it and nothing in the product path may import it.

Every floating-point quantity is computed in float64 from the stored inputs
widened exactly, with one exception that is part of the contract with the CUDA
path: the arithmetic that *decides integers* (group reduction of the scores and
everything downstream: budgets, the two top-k stages) runs in IEEE float32 in a
fixed operation order, because that is the precision the kernels decide in.

Pins (tests/test_oracle_*.py): softmax rows sum to one; w = 1, kp = 1 reduces
to a library softmax; max-pool against a library sliding maximum and a loop;
the projection norm against closed forms (identity / one-hot / scaled rows) and
a triple loop; Theorem 3.2 as an identity; Theorem 3.3 by enumerating every
subset on n <= 16; Theorem 3.5's arg-min by enumerating every stage-2
completion; alpha = 1 and constant-norm special cases; tie-breaking and budget
invariants.  The whole-path output on the large synthetic configurations has no
printed worked example in the paper to compare with: beyond those pins it is
"parity unpinned".

Readings of the paper where it is silent or inconsistent (each is an argument,
defaults below): logit scale 1/sqrt(head_dim) (Eq. 2); causal mask inside the
window; both stages use the pooled window mean (Algorithm 2 hands its
accumulated weights to Algorithm 1); GQA groups reduce by the arithmetic mean
of the per-query-head scores; b' = floor(alpha * b); ties go to the lower
index; retained rows keep their original order.
"""
from __future__ import annotations

import math
from itertools import combinations

import numpy as np

F64 = np.float64
F32 = np.float32


# ----------------------------------------------------------------------------
# Step 1: observation-window attention (Algorithm 2: the window slice of the queries,
# the softmax and window-mean step and the max-pooling step;
# Eq. 2 for the softmax and its scale)
# ----------------------------------------------------------------------------
def window_softmax(Qw_h, K_g, scale):
    """Causal softmax of the w window queries of one query head over all n keys.

    Window row j sits at sequence position n - w + j and sees keys i <= n - w + j.
    Returns A [w, n] float64, rows summing to one, masked entries exactly 0.
    """
    Qw_h = np.asarray(Qw_h, dtype=F64)
    K_g = np.asarray(K_g, dtype=F64)
    w, n = Qw_h.shape[0], K_g.shape[0]
    logits = (Qw_h @ K_g.T) * F64(scale)
    pos = n - w + np.arange(w)
    visible = np.arange(n)[None, :] <= pos[:, None]
    logits = np.where(visible, logits, -np.inf)
    m = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - m)
    e[~visible] = 0.0
    return e / e.sum(axis=1, keepdims=True)


def window_mean(A):
    """A_bar[i] = (1/w) sum_j A[j, i]  (Algorithm 2, mean over the window rows)."""
    A = np.asarray(A, dtype=F64)
    return A.sum(axis=0) / F64(A.shape[0])


def max_pool(x, kp):
    """Stride-1 max-pool along the sequence, window kp centred on i, clipped
    at both borders, output length n (Algorithm 2: maxpooling; kernel size
    from Section 4.1)."""
    if kp < 1 or kp % 2 == 0:
        raise ValueError("pool kernel must be odd and >= 1")
    x = np.asarray(x)
    n = x.shape[-1]
    r = (kp - 1) // 2
    out = x.copy()
    for d in range(1, r + 1):
        # neighbour at i + d
        out[..., : n - d] = np.maximum(out[..., : n - d], x[..., d:])
        # neighbour at i - d
        out[..., d:] = np.maximum(out[..., d:], x[..., : n - d])
    return out


def pooled_window_attention(Qw, K, kp, scale=None):
    """P [Hq, n] float64: per query head, max-pooled window-mean attention.

    Qw [Hq, w, dh], K [Hkv, n, dh]; query head h reads KV head h // G.
    """
    Hq, w, dh = Qw.shape
    Hkv, n, _ = K.shape
    G = Hq // Hkv
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(dh)
    P = np.empty((Hq, n), dtype=F64)
    for h in range(Hq):
        A = window_softmax(Qw[h], K[h // G], scale)
        P[h] = max_pool(window_mean(A), kp)
    return P


# ----------------------------------------------------------------------------
# Step 2: projected value-row norm (Algorithm 1: "V_cal = V W^O" and the
# "L1 norm of each row"; Theorem 3.3 for the role of the norm)
# ----------------------------------------------------------------------------
def projection_norm(V, WO, *, rows=None, chunk=2048, norm="l1"):
    """nu [Hq, n] float64 with nu[h, i] = || V[h // G, i, :] @ WO[h] ||_1.

    V [Hkv, n, dh]; WO [Hq, dh, dm] (head h's rows of the output projection).
    The product is materialised chunk by chunk and reduced row-wise.
    ``rows``: optional index array: only these token rows are computed
    (result [Hq, len(rows)]).
    """
    Hkv, n, dh = V.shape
    Hq, _, dm = WO.shape
    G = Hq // Hkv
    sel = np.arange(n) if rows is None else np.asarray(rows)
    nu = np.empty((Hq, sel.size), dtype=F64)
    for h in range(Hq):
        W = np.asarray(WO[h], dtype=F64)
        Vg = V[h // G]
        for s in range(0, sel.size, chunk):
            r = sel[s:s + chunk]
            proj = np.asarray(Vg[r], dtype=F64) @ W          # [rows, dm]
            if norm == "l1":
                nu[h, s:s + chunk] = np.abs(proj).sum(axis=1)
            elif norm == "l2":
                nu[h, s:s + chunk] = np.sqrt((proj * proj).sum(axis=1))
            else:
                raise ValueError(norm)
    return nu


def group_summed_projection(WO, G, storage="f32"):
    """W_tilde [Hkv, dh, dm]: the output-projection slices of a KV group added up (float32, heads in increasing
    order) and rounded once to the storage type.  Variant of step 2 for grouped-query attention: the heads of a
    group share K and V, so their outputs add in o = sum_h A_h V_g W^O_h (Eq. 2 applied per head); projecting a
    value row through the summed slice costs one contraction per KV head instead of one per query head.  The paper
    does not spell this variant out; its memory figure for the projected values (one n x d matrix per KV head)
    is consistent with it.  Returned widened to float32."""
    WO = np.asarray(WO, dtype=F32)
    Hq = WO.shape[0]
    Hkv = Hq // G
    out = np.empty((Hkv,) + WO.shape[1:], dtype=F32)
    for g in range(Hkv):
        acc = WO[g * G].copy()
        for h in range(g * G + 1, (g + 1) * G):
            acc = (acc + WO[h]).astype(F32)
        out[g] = acc
    if storage == "bf16":
        import torch
        out = torch.from_numpy(out).to(torch.bfloat16).to(torch.float32).numpy()
    elif storage != "f32":
        raise ValueError(storage)
    return out


def projection_norm_group_sum(V, WO, G, storage="f32", **kw):
    """nu [Hkv, n]: L1 norm of each value row projected through its group's summed W^O slice."""
    return projection_norm(V, group_summed_projection(WO, G, storage), **kw)


def group_scores_group_sum(P, nu_g, G, eps=1e-4):
    """a as in group_scores; c_g = (a_g + eps) * nu_g with nu_g [Hkv, n] (float32, separately rounded + and *)."""
    a, _ = group_scores(P, np.ones_like(np.asarray(P, dtype=F32)), G, eps)
    nu_g = np.asarray(nu_g).astype(F32)
    c = ((a + F32(eps)).astype(F32) * nu_g).astype(F32)
    return a, c


# ----------------------------------------------------------------------------
# Step 3: scores per KV head and budgets
# (Algorithm 1: "A_cal = (A + eps) * row norms", "b' = b x alpha; b'' = b - b'";
#  Algorithm 2: "allocate budget b across heads")
# Decision arithmetic: IEEE float32, fixed order (see module docstring).
# ----------------------------------------------------------------------------
def group_scores(P, nu, G, eps=1e-4):
    """a [Hkv, n], c [Hkv, n] float32.

    a_g = (P_{gG} + P_{gG+1} + ... ) / G                  (left-to-right float32 sums)
    c_g = ((P_{gG}+eps)*nu_{gG} + (P_{gG+1}+eps)*nu_{gG+1} + ...) / G
    every +, * and / a separately rounded float32 operation.
    """
    P = np.asarray(P).astype(F32)
    nu = np.asarray(nu).astype(F32)
    Hq, n = P.shape
    Hkv = Hq // G
    e = F32(eps)
    Gf = F32(G)
    a = np.empty((Hkv, n), dtype=F32)
    c = np.empty((Hkv, n), dtype=F32)
    for g in range(Hkv):
        sa = P[g * G].copy()
        sc = ((P[g * G] + e).astype(F32) * nu[g * G]).astype(F32)
        for h in range(g * G + 1, (g + 1) * G):
            sa = (sa + P[h]).astype(F32)
            t = ((P[h] + e).astype(F32) * nu[h]).astype(F32)
            sc = (sc + t).astype(F32)
        a[g] = (sa / Gf).astype(F32)
        c[g] = (sc / Gf).astype(F32)
    return a, c


def split_budget(b, alpha):
    """b' = floor(alpha * b) in double precision, b'' = b - b' (Algorithm 1)."""
    b1 = int(math.floor(float(F32(alpha)) * float(b)))
    b1 = min(max(b1, 0), int(b))
    return b1, int(b) - b1


def stable_topk(x, k):
    """Indices of the k largest entries; equal values go to the lower index.
    Returned in rank order (best first)."""
    x = np.asarray(x)
    if k <= 0:
        return np.empty(0, dtype=np.int64)
    order = np.argsort(-x, kind="stable")
    return order[:k]


def allocate_budgets(a, mode, budget, floor=0.0):
    """Per-KV-head budgets b_g (Algorithm 2, budget allocation step).

    uniform : every head gets ``budget``.
    adaptive: the ``budget`` largest entries of the flattened [Hkv * n]
              attention scores are counted per head (ties: lower flattened
              index g * n + i first).
    floor   : adaptive only.  Every head is first guaranteed
              floor_b = floor(floor * budget / Hkv) entries (the safeguard of
              adaptive allocation schemes), the remaining budget - Hkv * floor_b
              entries are allocated by the flattened top-k, and b_g is capped at n.
    """
    Hkv, n = a.shape
    if mode == "uniform":
        return np.full(Hkv, int(budget), dtype=np.int64)
    if mode == "adaptive":
        floor_b = int(math.floor(float(F32(floor)) * float(budget) / float(Hkv)))
        floor_b = min(max(floor_b, 0), int(budget) // Hkv)
        top = stable_topk(a.reshape(-1), int(budget) - Hkv * floor_b)
        counts = np.bincount(top // n, minlength=Hkv).astype(np.int64)
        return np.minimum(counts + floor_b, n)
    raise ValueError(mode)


def protect_window(a, c, w):
    """Variant: the last w entries (the observation window itself) are always kept.  Their scores are raised to the
    largest float32 in both stages, so they fill stage 1 first (lowest index first) and count against the budget."""
    a, c = a.copy(), c.copy()
    big = np.finfo(F32).max
    a[:, a.shape[1] - w:] = big
    c[:, c.shape[1] - w:] = big
    return a, c


# ----------------------------------------------------------------------------
# Step 4: two-stage selection of one head (Algorithm 1, stage 1 and stage 2)
# ----------------------------------------------------------------------------
def two_stage_select(a_g, c_g, b, alpha):
    """Returns (S1, S2): stage-1 indices = top-b' of a_g; stage-2 indices =
    top-b'' of c_g among the entries stage 1 left.  Both ascending."""
    n = a_g.shape[0]
    b1, b2 = split_budget(b, alpha)
    S1 = stable_topk(a_g, b1)
    rest = np.ones(n, dtype=bool)
    rest[S1] = False
    cand = np.nonzero(rest)[0]                      # ascending, so ties keep index order
    S2 = cand[stable_topk(np.asarray(c_g)[cand], b2)]
    return np.sort(S1), np.sort(S2)


def select(P, nu, *, G, budget_mode, budget, alpha=0.5, eps=1e-4, budgets_in=None, group_sum=False,
           adaptive_floor=0.0, protect_w=0):
    """Steps 3+4 for one layer.

    Returns dict(idx [Btot] int32 packed by head, ascending inside a head;
    offsets [Hkv+1] int32; stage [Btot] uint8 (1 or 2); a, c float32; budgets).
    group_sum: nu is [Hkv, n] from projection_norm_group_sum.
    """
    a, c = group_scores_group_sum(P, nu, G, eps) if group_sum else group_scores(P, nu, G, eps)
    if protect_w:
        a, c = protect_window(a, c, protect_w)
    Hkv, n = a.shape
    if budget_mode == "given":
        budgets = np.asarray(budgets_in, dtype=np.int64)
    else:
        budgets = allocate_budgets(a, budget_mode, budget, adaptive_floor)
    idx, stage, offsets = [], [], [0]
    for g in range(Hkv):
        S1, S2 = two_stage_select(a[g], c[g], int(budgets[g]), alpha)
        S = np.concatenate([S1, S2])
        st = np.concatenate([np.ones(S1.size, np.uint8), np.full(S2.size, 2, np.uint8)])
        order = np.argsort(S, kind="stable")
        idx.append(S[order])
        stage.append(st[order])
        offsets.append(offsets[-1] + S.size)
    return dict(idx=np.concatenate(idx).astype(np.int32), stage=np.concatenate(stage),
                offsets=np.asarray(offsets, dtype=np.int32), a=a, c=c, budgets=budgets)


# ----------------------------------------------------------------------------
# Step 5: compaction (Algorithm 1, the steps that append the selected entries to the retained cache)
# ----------------------------------------------------------------------------
def compact(K_store, V_store, idx, offsets):
    """Row gather of the stored (unwidened) K, V: [Btot, dh] each, packed like idx."""
    Hkv = K_store.shape[0]
    Ko = np.empty((idx.size, K_store.shape[2]), dtype=K_store.dtype)
    Vo = np.empty_like(Ko)
    for g in range(Hkv):
        s, e = int(offsets[g]), int(offsets[g + 1])
        Ko[s:e] = K_store[g][idx[s:e]]
        Vo[s:e] = V_store[g][idx[s:e]]
    return Ko, Vo


def compress_layer(Qw, K, V, WO, *, kp, budget_mode, budget, alpha=0.5, eps=1e-4, scale=None,
                   K_store=None, V_store=None, group_sum=False, storage="f32"):
    """The whole path for one layer, step by step."""
    G = Qw.shape[0] // K.shape[0]
    P = pooled_window_attention(Qw, K, kp, scale)
    nu = projection_norm_group_sum(V, WO, G, storage) if group_sum else projection_norm(V, WO)
    out = select(P, nu, G=G, budget_mode=budget_mode, budget=budget, alpha=alpha, eps=eps, group_sum=group_sum)
    Ko, Vo = compact(K if K_store is None else K_store, V if V_store is None else V_store,
                     out["idx"], out["offsets"])
    out.update(P=P, nu=nu, K_hat=Ko, V_hat=Vo)
    return out


def compress_layer_ragged(Qw, K_list, V_list, WO, *, kp, budget_mode, budget, alpha=0.5, eps=1e-4, scale=None):
    """The whole path for one layer whose KV heads hold different numbers of entries (what adaptive budgets leave
    behind between the chunks of a chunked prefill).  K_list[g], V_list[g]: [n_g, dh]; the observation window of
    every head is its own last w entries.  Every step is the per-head definition applied to that head's own list;
    the adaptive allocation ranks the attention scores of all heads' entries together, ties going to the lower
    (head, entry) pair.

    Returns dict(P [Hq] list of [n_g] arrays, nu likewise, a, c [Hkv] lists of float32 arrays, budgets [Hkv],
    idx (entry numbers inside each head's own list, packed by head, ascending), offsets [Hkv+1], stage).
    """
    Hq, w, dh = Qw.shape
    Hkv = len(K_list)
    G = Hq // Hkv
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(dh)
    P, nu = [], []
    for h in range(Hq):
        g = h // G
        P.append(max_pool(window_mean(window_softmax(Qw[h], K_list[g], scale)), kp))
        nu.append(projection_norm(np.asarray(V_list[g])[None], np.asarray(WO[h])[None])[0])
    a, c = [], []
    for g in range(Hkv):
        ag, cg = group_scores(np.stack(P[g * G:(g + 1) * G]), np.stack(nu[g * G:(g + 1) * G]), G, eps)
        a.append(ag[0])
        c.append(cg[0])
    lens = np.array([x.shape[0] for x in a], dtype=np.int64)
    if budget_mode == "uniform":
        budgets = np.full(Hkv, int(budget), dtype=np.int64)
    elif budget_mode == "adaptive":
        start = np.concatenate([[0], np.cumsum(lens)])
        top = stable_topk(np.concatenate(a), int(budget))             # order of the concatenation = (head, entry)
        head_of = np.searchsorted(start, top, side="right") - 1
        budgets = np.bincount(head_of, minlength=Hkv).astype(np.int64)
    else:
        raise ValueError(budget_mode)
    if np.any(budgets > lens):
        raise ValueError("a head's budget exceeds the entries it holds")
    idx, stage, offsets = [], [], [0]
    for g in range(Hkv):
        S1, S2 = two_stage_select(a[g], c[g], int(budgets[g]), alpha)
        S = np.concatenate([S1, S2])
        st = np.concatenate([np.ones(S1.size, np.uint8), np.full(S2.size, 2, np.uint8)])
        order = np.argsort(S, kind="stable")
        idx.append(S[order])
        stage.append(st[order])
        offsets.append(offsets[-1] + S.size)
    return dict(P=P, nu=nu, a=a, c=c, budgets=budgets, idx=np.concatenate(idx).astype(np.int32),
                stage=np.concatenate(stage), offsets=np.asarray(offsets, dtype=np.int32))


def chunked_compress(chunks, WO, *, kp, w, budgets, alpha=0.5, eps=1e-4, scale=None, budget_mode="uniform"):
    """Chunked prefill with eviction between chunks (the paper's long-context deployment, appendix on chunked
    prefill): for every chunk the cache is [retained entries ; the chunk's K, V], the observation window is the last
    w queries of the chunk, and the cache is compressed to ``budgets[c]``: entries per KV head with uniform budgets
    (every head keeps the same number), entries per layer with adaptive budgets (the heads then keep different
    numbers and the next chunk meets a ragged cache).  Later chunks therefore see a smaller cache.

    chunks: list of (Qw [Hq,w,dh], K [Hkv,len,dh], V [Hkv,len,dh]) widened inputs.
    Returns (K_ret, V_ret, pos, history of per-step idx): uniform budgets give arrays [Hkv, B_last, dh] and
    [Hkv, B_last] (original token positions) and idx [Hkv, B]; adaptive budgets give per-head lists of arrays
    and, per step, the list of each head's retained entry numbers.
    """
    if budget_mode == "adaptive":
        return _chunked_compress_adaptive(chunks, WO, kp=kp, budgets=budgets, alpha=alpha, eps=eps, scale=scale)
    K_ret = V_ret = pos = None
    seen = 0
    hist = []
    for c, (Qw, K, V) in enumerate(chunks):
        Hkv, ln, _ = K.shape
        new_pos = np.broadcast_to(np.arange(seen, seen + ln, dtype=np.int64), (Hkv, ln))
        if K_ret is None:
            Kc, Vc, pc = K, V, new_pos
        else:
            Kc = np.concatenate([K_ret, K], axis=1)
            Vc = np.concatenate([V_ret, V], axis=1)
            pc = np.concatenate([pos, new_pos], axis=1)
        seen += ln
        out = compress_layer(Qw, Kc, Vc, WO, kp=kp, budget_mode="uniform", budget=int(budgets[c]), alpha=alpha,
                             eps=eps, scale=scale)
        B = int(budgets[c])
        idx = out["idx"].reshape(Hkv, B)
        K_ret = np.stack([Kc[g][idx[g]] for g in range(Hkv)])
        V_ret = np.stack([Vc[g][idx[g]] for g in range(Hkv)])
        pos = np.stack([pc[g][idx[g]] for g in range(Hkv)])
        hist.append(idx)
    return K_ret, V_ret, pos, hist


def _chunked_compress_adaptive(chunks, WO, *, kp, budgets, alpha, eps, scale):
    K_ret = V_ret = pos = None
    seen = 0
    hist = []
    for c, (Qw, K, V) in enumerate(chunks):
        Hkv, ln, _ = K.shape
        new_pos = np.arange(seen, seen + ln, dtype=np.int64)
        if K_ret is None:
            Kc, Vc, pc = [K[g] for g in range(Hkv)], [V[g] for g in range(Hkv)], [new_pos] * Hkv
        else:
            Kc = [np.concatenate([K_ret[g], K[g]], axis=0) for g in range(Hkv)]
            Vc = [np.concatenate([V_ret[g], V[g]], axis=0) for g in range(Hkv)]
            pc = [np.concatenate([pos[g], new_pos]) for g in range(Hkv)]
        seen += ln
        out = compress_layer_ragged(Qw, Kc, Vc, WO, kp=kp, budget_mode="adaptive", budget=int(budgets[c]),
                                    alpha=alpha, eps=eps, scale=scale)
        off = out["offsets"]
        kept = [out["idx"][off[g]:off[g + 1]] for g in range(Hkv)]
        K_ret = [Kc[g][kept[g]] for g in range(Hkv)]
        V_ret = [Vc[g][kept[g]] for g in range(Hkv)]
        pos = [pc[g][kept[g]] for g in range(Hkv)]
        hist.append(kept)
    return K_ret, V_ret, pos, hist


# ----------------------------------------------------------------------------
# Diagnostics: the quantities of Section 3 (Definition 3.1, Theorems 3.2, 3.3,
# 3.5, Assumption 3.4, relaxed bound).  Single query row, single head.
# ----------------------------------------------------------------------------
def masked_softmax(logits, keep):
    """A' = softmax(M + logits), M_i = -inf for evicted entries (Section 3.3)."""
    logits = np.asarray(logits, dtype=F64)
    keep = np.asarray(keep, dtype=bool)
    z = np.where(keep, logits, -np.inf)
    m = z.max()
    e = np.where(keep, np.exp(z - m), 0.0)
    return e / e.sum()


def perturbation(A, A_prime, Vproj):
    """L = || (A - A') V W^O ||_1 (Definition 3.1 / Section 3.3)."""
    return float(np.abs((np.asarray(A, F64) - np.asarray(A_prime, F64)) @ np.asarray(Vproj, F64)).sum())


def theta_bound(A, nu, keep):
    """theta of Theorem 3.3."""
    A, nu = np.asarray(A, F64), np.asarray(nu, F64)
    keep = np.asarray(keep, dtype=bool)
    C = float((A * nu).sum())
    mass = float(A[keep].sum())
    return C - (2.0 - 1.0 / mass) * float((A[keep] * nu[keep]).sum())


def theta_hat_bound(A, nu, keep1, keep2):
    """theta_hat of Theorem 3.5 (sigma = attention mass of the stage-1 set)."""
    A, nu = np.asarray(A, F64), np.asarray(nu, F64)
    k1, k2 = np.asarray(keep1, bool), np.asarray(keep2, bool)
    sigma = float(A[k1].sum())
    C = float((A * nu).sum())
    f = 2.0 - 1.0 / sigma
    return C - f * float((A[k1] * nu[k1]).sum()) - f * float((A[k2] * nu[k2]).sum())


def theta_relax_bound(A, nu, keep1, keep2):
    """theta_hat^relax of the appendix theorem (M = min_i nu_i)."""
    A, nu = np.asarray(A, F64), np.asarray(nu, F64)
    k1, k2 = np.asarray(keep1, bool), np.asarray(keep2, bool)
    sigma = float(A[k1].sum())
    C = float((A * nu).sum())
    f = 2.0 - 1.0 / sigma
    return C - f * float((A[k1] * nu[k1]).sum()) - float(nu.min()) * f * float(A[k2].sum())


def stage1_mass(a_g, b, alpha):
    """sigma of Assumption 3.4: attention collected by stage 1."""
    b1, _ = split_budget(b, alpha)
    return float(np.sort(np.asarray(a_g, F64))[::-1][:b1].sum())


def post_eviction_output(Qw_h, K_g, V_g, keep_idx, scale):
    """o_hat [w, dh]: window queries attending only to the retained entries
    (causal by original position), before W^O.  ``keep_idx=None`` = full cache."""
    Qw_h, K_g, V_g = (np.asarray(x, dtype=F64) for x in (Qw_h, K_g, V_g))
    w, n = Qw_h.shape[0], K_g.shape[0]
    keep = np.ones(n, bool) if keep_idx is None else np.isin(np.arange(n), keep_idx)
    logits = (Qw_h @ K_g.T) * F64(scale)
    pos = n - w + np.arange(w)
    out = np.zeros((w, V_g.shape[1]), dtype=F64)
    for j in range(w):
        vis = keep & (np.arange(n) <= pos[j])
        if not vis.any():
            continue
        out[j] = masked_softmax(logits[j], vis) @ V_g
    return out


DIAG_FIELDS = ("sigma", "mass_kept", "C", "C_stage1", "C_stage2", "nu_min", "L", "theta", "theta_hat",
               "theta_relax")


def row_diagnostics(Qw_h, K_g, V_g, WO_h, S1, S2, scale):
    """Section 3 quantities of one query head for each of its w window rows and a given selection (S1, S2 = index
    arrays of the two stages): per row j, with A = the row's causal softmax and nu = row L1 norms of V W^O,
      sigma = sum_{S1} A (Assumption 3.4), mass_kept = sum_{S1+S2} A, C = sum_i A_i nu_i, C_stage1/2 = the same sum
      over each stage, nu_min = min_i nu_i, L = || (A - A') V W^O ||_1 (Definition 3.1, A' by Theorem 3.2),
      theta (Theorem 3.3), theta_hat (Theorem 3.5), theta_relax (relaxed bound of the appendix).
    Returns [w, 10] float64 in the order of DIAG_FIELDS."""
    Qw_h, K_g, V_g, WO_h = (np.asarray(x, dtype=F64) for x in (Qw_h, K_g, V_g, WO_h))
    w, n = Qw_h.shape[0], K_g.shape[0]
    A = window_softmax(Qw_h, K_g, scale)
    Vp = V_g @ WO_h
    nu = np.abs(Vp).sum(axis=1)
    k1 = np.zeros(n, bool)
    k1[np.asarray(S1, dtype=np.int64)] = True
    k2 = np.zeros(n, bool)
    k2[np.asarray(S2, dtype=np.int64)] = True
    keep = k1 | k2
    out = np.zeros((w, len(DIAG_FIELDS)), dtype=F64)
    for j in range(w):
        a = A[j]
        sigma, mass = a[k1].sum(), a[keep].sum()
        C, C1, C2 = (a * nu).sum(), (a[k1] * nu[k1]).sum(), (a[k2] * nu[k2]).sum()
        a_kept = np.where(keep, a, 0.0) / mass if mass > 0 else np.zeros(n)
        L = np.abs((a - a_kept) @ Vp).sum()
        f_all = 2.0 - 1.0 / mass if mass > 0 else -np.inf
        f_s1 = 2.0 - 1.0 / sigma if sigma > 0 else -np.inf
        theta = C - f_all * (C1 + C2)
        theta_hat = C - f_s1 * (C1 + C2)
        theta_relax = C - f_s1 * C1 - nu.min() * f_s1 * a[k2].sum()
        out[j] = (sigma, mass, C, C1, C2, nu.min(), L, theta, theta_hat, theta_relax)
    return out


def all_subsets(n, b):
    """Every subset of size b as a boolean mask (tiny n only)."""
    for comb in combinations(range(n), b):
        m = np.zeros(n, dtype=bool)
        m[list(comb)] = True
        yield m
