"""Runs the CUDA path on generated layers and returns host arrays (GPU tests and smoke check)."""
from __future__ import annotations

import numpy as np
import torch

from paper_2502_03805_b200 import session_for, to_device, to_host


def upload_layers(layers, wl, device="cuda:0"):
    """Stack the stored inputs of several layers along nb and upload them bit-exactly."""
    def stack(name):
        return to_device(np.stack([getattr(L, name) for L in layers]), wl.dtype, device)
    return stack("Qw_store"), stack("K_store"), stack("V_store"), stack("WO_store")


def run_layers(layers, wl, *, flags=0, separate_calls=False, valid_from=None, **session_kw):
    """One library call over nb = len(layers).  Returns (list of per-layer dicts of host arrays, session)."""
    Qw, K, V, WO = upload_layers(layers, wl)
    s = session_for(wl, nb=len(layers), flags=flags, valid_from=valid_from, **session_kw)
    if separate_calls:
        s.score(Qw, K, V, WO)
        s.select()
        s.compact(K, V)
    else:
        s.compress(Qw, K, V, WO)
    torch.cuda.synchronize()
    assert s.device_status() == 0
    outs = []
    for b in range(len(layers)):
        outs.append(dict(attn=to_host(s.attn[b]), vnorm=to_host(s.vnorm[b]), idx=to_host(s.idx[b]),
                         offsets=to_host(s.offsets[b]), stage=to_host(s.stage[b]),
                         K_out=to_host(s.K_out[b]), V_out=to_host(s.V_out[b])))
    return outs, s
