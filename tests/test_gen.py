"""The seeded generators: determinism, storage rounding, and the structure the recipe promises
(checked with the CPU oracle: attention concentration, Assumption 3.4)."""
import numpy as np
import torch

from gen import bf16_bits_to_f32, config, f32_to_bf16_bits, make_layer, small_workload
from oracle import criticalkv_oracle as oc


def test_bf16_rounding_matches_library_conversion():
    r = np.random.default_rng(0)
    x = np.concatenate([r.standard_normal(5000).astype(np.float32) * 10.0 ** r.integers(-20, 20, 5000),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 65504.0], np.float32)]).astype(np.float32)
    bits = f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    np.testing.assert_array_equal(bits, ref.view(torch.int16).numpy().view(np.uint16))
    np.testing.assert_array_equal(bf16_bits_to_f32(bits), ref.to(torch.float32).numpy())


def test_layers_are_deterministic_and_distinct():
    wl = small_workload(dtype="bf16", n=200, dh=64, dm=128)
    a, b = make_layer(wl, 3), make_layer(wl, 3)
    for name in ("Qw_store", "K_store", "V_store", "WO_store"):
        np.testing.assert_array_equal(getattr(a, name), getattr(b, name))
    c = make_layer(wl, 4)
    assert not np.array_equal(a.K_store, c.K_store)
    assert a.K_store.dtype == np.uint16 and a.K.dtype == np.float32
    np.testing.assert_array_equal(bf16_bits_to_f32(a.V_store), a.V)


def test_shapes_of_named_configs():
    for cid, (Hq, Hkv, dh, dm, n, w, kp, btot) in {
            0: (4, 2, 64, 256, 512, 16, 5, 256), 1: (32, 8, 128, 4096, 4096, 32, 7, 8 * 819),
            2: (32, 8, 128, 4096, 32768, 32, 7, 8 * 13107), 3: (32, 8, 128, 4096, 32768, 32, 7, 52428),
            4: (40, 8, 128, 5120, 131072, 64, 7, 8 * 13107)}.items():
        wl = config(cid)
        assert (wl.Hq, wl.Hkv, wl.dh, wl.dm, wl.n, wl.w, wl.kp, wl.btot) == (Hq, Hkv, dh, dm, n, w, kp, btot)


def test_config0_structure():
    wl = config(0)
    L = make_layer(wl)
    assert L.Qw.shape == (4, 16, 64) and L.K.shape == (2, 512, 64) and L.WO.shape == (4, 64, 256)
    # four outlier key channels per KV head, eight times the spread of the others
    for g in range(wl.Hkv):
        std = L.K[g].std(axis=0)
        big = np.sort(std)[-4:]
        assert np.all(big > 5) and np.sort(std)[-5] < 2
    # per-head scale of W_O within [0.5, 2] / sqrt(dm)
    s = L.WO.reshape(wl.Hq, -1).std(axis=1) * np.sqrt(wl.dm)
    assert np.all(s > 0.45) and np.all(s < 2.1)


def test_concentration_and_assumption_3_4_on_config1():
    wl = config(1)
    L = make_layer(wl)
    shares, P = [], np.empty((wl.Hq, wl.n))
    for h in range(wl.Hq):
        abar = oc.window_mean(oc.window_softmax(L.Qw[h], L.K[h // wl.G], wl.scale))
        shares.append(np.sort(abar)[::-1][: int(0.05 * wl.n)].sum())
        P[h] = oc.max_pool(abar, wl.kp)
    assert 0.6 < np.mean(shares) < 0.8                       # recipe: ~70% of the mass on the top 5% of keys
    a, _ = oc.group_scores(P, np.ones_like(P), wl.G)
    sig = [oc.stage1_mass(a[g], wl.budget, wl.alpha) for g in range(wl.Hkv)]
    assert min(sig) > 0.5                                    # Assumption 3.4
