"""Pins for the synthetic input generators (the inputs themselves, not the method)."""
import numpy as np

from oracle import decode_bf16, decode_e4m3
from workloads import CONFIGS, make_config


def test_config_table_matches_benchmark_shapes():
    assert CONFIGS["tiny_f32"][1:7] == ("f32", 64, 4096, 8, 64, 256)
    assert CONFIGS["dsa_bf16"][1:7] == ("bf16", 4096, 65536, 64, 128, 2048)
    assert CONFIGS["fp8_ar1"][1:7] == ("e4m3", 8192, 131072, 64, 128, 2048)
    assert CONFIGS["fp8_1m"][1:7] == ("e4m3", 4096, 1048576, 64, 128, 2048)
    inp = make_config("tiny_f32")
    assert (inp.T, inp.N, inp.H, inp.D, inp.topk, inp.causal_offset) == (64, 4096, 8, 64, 256, 4032)
    assert inp.visible(0) == 4033 and inp.visible(63) == 4096
    assert inp.valid_pairs() == 64 * 4096 - 64 * 63 // 2 == 260128


def test_seeded_and_deterministic():
    a = make_config("dsa_bf16", T=32, N=512)
    b = make_config("dsa_bf16", T=32, N=512)
    c = make_config("dsa_bf16", T=32, N=512, seed=5)
    assert np.array_equal(a.q, b.q) and np.array_equal(a.k, b.k) and np.array_equal(a.w, b.w)
    assert not np.array_equal(a.k, c.k)


def test_moments_iid():
    inp = make_config("tiny_f32", T=256, N=8192)
    D, H = inp.D, inp.H
    for x, var in ((inp.q, 1.0 / D), (inp.k, 1.0 / D), (inp.w, 1.0 / H)):
        n = x.size
        assert abs(x.mean()) < 4 * np.sqrt(var / n)
        assert abs(x.var() / var - 1) < 4 * np.sqrt(2.0 / n)


def test_drift_tracks_sine():
    inp = make_config("dsa_bf16", T=16, N=32768)
    u = inp.meta["drift_dir"].astype(np.float64)
    proj = decode_bf16(inp.k) @ u
    s = np.arange(inp.N)
    want = 0.2 * np.sin(s / 4096.0)
    resid = proj - want  # what is left is the iid part along u: variance 1/D
    assert abs(resid.mean()) < 5 * np.sqrt(1.0 / inp.D / inp.N) + 1e-3
    assert abs(resid.var() * inp.D - 1) < 0.1
    assert np.corrcoef(proj, want)[0, 1] > 0.8


def test_ar1_queries_and_fp8_scales():
    inp = make_config("fp8_ar1", T=2048, N=1024, H=8, D=32)
    assert inp.q.dtype == np.uint8 and inp.k.dtype == np.uint8 and inp.k_scale.shape == (inp.N,)
    qd = decode_e4m3(inp.q).reshape(inp.T, -1)
    # per-token scaling distorts amplitudes a little; correlate the raw codes' directions instead
    qn = qd / np.abs(qd).max(axis=1, keepdims=True)
    lag1 = np.mean([np.corrcoef(qn[:-1, j], qn[1:, j])[0, 1] for j in range(0, qn.shape[1], 7)])
    assert abs(lag1 - 0.9) < 0.03
    assert np.all(np.abs(decode_e4m3(inp.k)).max(axis=1) == 448.0)  # absmax maps to the top code
    assert np.all(inp.k_scale > 0)
    assert not np.any((inp.q & 0x7F) == 0x7F) and not np.any((inp.k & 0x7F) == 0x7F)  # no NaN codes


def test_planted_fraction_and_direction():
    inp = make_config("adv_planted", T=64, N=4000, H=8, D=32)
    pos = inp.meta["planted_pos"]
    assert pos.shape[0] == round(0.05 * inp.N) == 200 and np.unique(pos).shape[0] == 200
    kd = decode_bf16(inp.k)
    norms = np.linalg.norm(kd, axis=1)
    assert np.allclose(norms[pos], 3.0, rtol=2e-2)
    others = np.setdiff1d(np.arange(inp.N), pos)
    assert abs(np.median(norms[others]) - 1.0) < 0.1 and norms[others].max() > 4.0  # heavy tail
    inp2 = make_config("adv_cluster", T=64, N=4000, H=8, D=32)
    pos2 = inp2.meta["planted_pos"]
    assert np.all(inp2.k[pos2] == inp2.k[pos2[0]])  # identical keys: exact ties


def test_four_level_inputs_are_exact():
    inp = make_config("adv_ties_exact", T=32, N=2048)
    qd, kd = decode_bf16(inp.q), decode_bf16(inp.k)
    step = 2.0 ** -4  # D = 128
    assert sorted(np.unique(np.abs(kd)).tolist()) == [0.5 * step, 1.5 * step]
    assert sorted(np.unique(np.abs(qd)).tolist()) == [0.5 * step, 1.5 * step]
    assert sorted(np.unique(inp.w).tolist()) == [-0.125, 0.125]  # H = 64
