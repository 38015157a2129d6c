"""Host-side checks of the seeded synthetic generator (input generation only)."""
import numpy as np

import synth


def bf16_to_f32(h):
    return (h.astype(np.uint32) << 16).view(np.float32)


def test_tables():
    g = synth.gauss_table()
    assert g.shape == (65536,) and g.dtype == np.float32
    assert abs(g.astype(np.float64).mean()) < 1e-6 and abs(g.astype(np.float64).std() - 1.0) < 1e-3
    assert np.all(np.diff(g) > 0) and np.allclose(g, -g[::-1])
    r = synth.rank_table(3, 1000)
    assert sorted(r.tolist()) == list(range(1, 1001))
    assert not np.array_equal(r, synth.rank_table(4, 1000))
    assert synth.lnrank_table(3, 1000).dtype == np.float32


def test_rows_are_deterministic_and_follow_the_recipe():
    V, seed = 4096, 9
    b = np.array([0, 1, 1], dtype=np.int32)
    k = np.array([0, 0, 2], dtype=np.int32)
    s = np.array([0.5, 2.0, 6.0], dtype=np.float32)
    tau = np.array([0.1, 1.0, 3.0], dtype=np.float32)
    d1 = synth.rows_cpu(0, seed, 5, b, k, s, None, V, synth.FP32)
    d2 = synth.rows_cpu(0, seed, 5, b, k, s, None, V, synth.FP32)
    assert np.array_equal(d1, d2)
    assert not np.array_equal(d1, synth.rows_cpu(0, seed, 6, b, k, s, None, V, synth.FP32))
    t1 = synth.rows_cpu(1, seed, 5, b, k, s, tau, V, synth.FP32)
    ln = synth.lnrank_table(seed, V).astype(np.float64)
    for r in range(3):
        g1 = (d1[r].astype(np.float64) + ln) / s[r]          # recovered first Gaussian
        assert abs(g1.mean()) < 0.08 and abs(g1.std() - 1.0) < 0.05
        g2 = (t1[r].astype(np.float64) - d1[r]) / tau[r]     # recovered second Gaussian
        assert abs(g2.mean()) < 0.08 and abs(g2.std() - 1.0) < 0.05
        assert abs(np.corrcoef(g1, g2)[0, 1]) < 0.06
    # bf16 output is the RNE rounding of the fp32 output
    h = synth.rows_cpu(1, seed, 5, b, k, s, tau, V, synth.BF16)
    f = bf16_to_f32(h)
    assert np.all(np.abs(f - t1) <= np.abs(t1) * 2.0 ** -8)
    import torch
    assert np.array_equal(torch.from_numpy(t1).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16), h)


def test_uniforms_and_params():
    u = synth.uniforms_cpu(1, synth.U_TARGET, 3, 4, 1000)
    assert u.dtype == np.float32 and u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 0.02
    assert not np.array_equal(u, synth.uniforms_cpu(1, synth.U_ACCEPT, 3, 4, 1000))
    wl = synth.WORKLOADS["C4"].scaled(B=64, rounds=2)
    s, t = wl.params(0)
    assert s.shape == (64, 17) and t.shape == (64, 17)
    assert np.isin(s, [12.0, 0.2]).mean() > 0.1 and s.min() >= 0.2 and s.max() <= 12.0
    assert t.min() >= 0.05 and t.max() <= 4.0
    wl5 = synth.WORKLOADS["C5"].scaled(B=2, rounds=11)
    assert abs(wl5.params(0)[1][0, 0] - 0.2) < 1e-6 and abs(wl5.params(10)[1][0, 0] - 3.0) < 1e-6
    s1, t1 = synth.WORKLOADS["C1"].params(7)
    assert np.allclose(s1[0], [0.5, 2, 6, 0.5, 2, 6]) and np.allclose(t1[0], [0.1, 1, 3, 0.1, 1, 3])


def test_host_round_shapes():
    wl = synth.WORKLOADS["C3"].scaled(B=3, V=2048)
    d, t = synth.host_round(wl, 2, [0, 2])
    assert d.shape == (2, 8, 2048) and t.shape == (2, 9, 2048) and d.dtype == np.uint16
    d_all, t_all = synth.host_round(wl, 2)
    assert np.array_equal(d_all[2], d[1]) and np.array_equal(t_all[0], t[0])
