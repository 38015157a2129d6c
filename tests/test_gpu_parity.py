"""GPU parity tests: the CUDA library, called through its C ABI, against the float64
oracle on the same seeded inputs.  Tolerances: 1e-4 absolute on entropy, log-sum-exp,
JS divergence/distance, T_G and P(A|d); discrete results exact except at counted
near-threshold positions (see tests/lockstep.py)."""
import ctypes
import math

import numpy as np
import pytest

import oracle
import synth

pytestmark = pytest.mark.gpu

TOL = 1e-4


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return torch


@pytest.fixture(scope="module")
def adasd():
    import paper_2512_11280_b200 as m
    m.lib()
    return m


def bf16_bits(t):
    return t.view(__import__("torch").int16).cpu().numpy().view(np.uint16)


def raw(t, torch):
    """Device logits -> the oracle's raw input (bf16 bits or float32)."""
    return bf16_bits(t) if t.dtype == torch.bfloat16 else t.cpu().numpy()


# ------------------------------------------------------------------ generator

def test_generator_host_and_device_rows_are_bit_identical(torch):
    for name, V in (("C1", 32000), ("C3", 5000)):
        wl = synth.WORKLOADS[name].scaled(B=3, V=V, rounds=4)
        gs = synth.GpuSynth(wl)
        tdt = torch.bfloat16 if wl.dtype == synth.BF16 else torch.float32
        zd = torch.empty((wl.B, wl.K, V), dtype=tdt, device="cuda")
        zt = torch.empty((wl.B, wl.K + 1, V), dtype=tdt, device="cuda")
        for r in (0, 3):
            gs.draft_rows(r, zd)
            gs.target_rows(r, zt)
            hd, ht = synth.host_round(wl, r)
            assert np.array_equal(raw(zd, torch).reshape(hd.shape), hd)
            assert np.array_equal(raw(zt, torch).reshape(ht.shape), ht)
        u = torch.empty((wl.B, 7), dtype=torch.float32, device="cuda")
        gs.uniforms(synth.U_ACCEPT, 2, u)
        assert np.array_equal(u.cpu().numpy(), synth.uniforms_cpu(wl.seed, synth.U_ACCEPT, 2, wl.B, 7))
        # the round counter kept on the device gives the same rows
        gs.advance_round(3)
        gs.draft_rows(0, zd, use_round_dev=True)
        assert np.array_equal(raw(zd, torch).reshape(hd.shape), synth.host_round(wl, 3)[0])


# ------------------------------------------------------------------ workloads in lockstep

def run_lockstep(wl, **kw):
    import json
    import os
    import time
    from tests.lockstep import Lockstep
    t0 = time.time()
    ls = Lockstep(wl, **kw)
    rep = ls.run()
    s = rep.summary()
    print(wl.name, s)
    log = os.environ.get("ADASD_PARITY_LOG")       # one JSON line per workload, for the records
    if log:
        with open(log, "a") as f:
            f.write(json.dumps(dict(workload=wl.name, B=wl.B, K=wl.K, V=wl.V, followed=len(ls.follow),
                                    seconds=round(time.time() - t0, 1), **s)) + "\n")
    # every disagreement was checked where it arose (it sat on a flagged decision or followed a
    # sample whose uniform lay on a CDF edge); there cannot be more of them than of those
    assert rep.flips <= rep.near_threshold + rep.tie_flips, s
    return rep


def test_c1_tiny_fp32_full(torch):
    rep = run_lockstep(synth.WORKLOADS["C1"])
    assert rep.rounds == 20 and rep.positions == 20 * 6


@pytest.mark.parametrize("V,dtype,cs", [(4, synth.FP32, 1), (64, synth.BF16, 2), (1000, synth.BF16, 4),
                                        (1003, synth.FP32, 8), (4099, synth.BF16, 8),
                                        (40000, synth.BF16, 0), (32768 + 8, synth.FP32, 2)])
def test_small_and_ragged_vocabularies(torch, V, dtype, cs):
    wl = synth.WORKLOADS["C3"].scaled(name=f"ragged{V}", B=3, K=4, V=V, dtype=dtype, rounds=10)
    run_lockstep(wl, cluster_size=cs, min_kde_samples=3)


@pytest.mark.parametrize("cs", [1, 2, 3, 4, 5, 6, 7, 8])
def test_streaming_kernels_at_every_cluster_size(torch, cs):
    # bf16 rows of a multiple of 8 logits take the warp-specialised kernels: 20008 logits give
    # every cluster size a different split (10 iterations per warp down to 1, ragged last unit),
    # in AdaSD mode and in vanilla mode (C3 runs both)
    wl = synth.WORKLOADS["C3"].scaled(name=f"stream_cs{cs}", B=5, K=3, V=20008, rounds=8)
    rep = run_lockstep(wl, cluster_size=cs, min_kde_samples=3)
    assert len(rep.vanilla_accept_hist) >= 2


@pytest.mark.parametrize("V", [2048, 8200])
def test_scott_bandwidth_and_threshold_rejection_rule(torch, V):
    # the two readings kept behind flags: Scott's bandwidth factor, and rejection when P(A|d) < 1/2
    # instead of the Bernoulli draw; enough rounds for the KDE lists to matter
    wl = synth.WORKLOADS["C3"].scaled(name=f"flags{V}", B=4, K=6, V=V, rounds=60, vanilla=False)
    rep = run_lockstep(wl, kde_bandwidth=1, reject_rule=1, check_lists_every=20)
    assert rep.n_rejections > 10 and len(rep.accept_hist) >= 2


def test_vanilla_mode_with_many_rows_takes_the_three_step_path(torch):
    # enough rows to fill the GPU several times over: log-sum-exps of all rows in a streaming
    # pass, the accept test per sequence, then the sampling of one position per sequence
    wl = synth.WORKLOADS["C3"].scaled(name="manyrows", B=192, K=3, V=8200, rounds=6)
    assert wl.B * (2 * wl.K + 1) >= 2 * 148
    rep = run_lockstep(wl, follow=[0, 5, 77, 130, 191], min_kde_samples=3)
    assert len(rep.vanilla_accept_hist) >= 3


# The four large workloads run EVERY round they state, in lockstep with the oracle: C2 and C3 on
# all their sequences, C4 and C5 on eight sequences spread over the batch (the other sequences
# run on the device all the same; the oracle follows the eight).

def test_c2_single_stream_adaptive_window_all_512_rounds(torch):
    wl = synth.WORKLOADS["C2"]
    rep = run_lockstep(wl, check_lists_every=64)
    assert rep.rounds == 512 and len(rep.window_hist) >= 2      # the stop check produced different windows


def test_c3_batched_with_vanilla_all_256_rounds_all_32_sequences(torch):
    wl = synth.WORKLOADS["C3"]
    rep = run_lockstep(wl, check_lists_every=64)
    assert rep.rounds == 256 and rep.positions == 256 * 32 * 9
    assert len(rep.accept_hist) >= 5 and len(rep.vanilla_accept_hist) >= 5


def test_c4_large_batch_large_vocab_all_128_rounds(torch):
    wl = synth.WORKLOADS["C4"]
    rep = run_lockstep(wl, follow=[0, 18, 37, 55, 73, 91, 110, 127], check_lists_every=32)
    assert rep.rounds == 128 and rep.positions == 128 * 8 * 17


def test_c5_streaming_adaptive_all_1024_rounds(torch):
    # the lists end near 10^4 entries per sequence; the context's capacity covers 1024 * 16 appends
    wl = synth.WORKLOADS["C5"]
    rep = run_lockstep(wl, follow=[0, 36, 73, 109, 146, 182, 219, 255], check_lists_every=128)
    assert rep.rounds == 1024 and max(rep.window_hist) <= 16 and len(rep.window_hist) >= 4


@pytest.mark.parametrize("V,dtype", [(128256, synth.BF16), (32000, synth.FP32)])
@pytest.mark.parametrize("tau", [1e-3, 3e-3, 1e-2, 3e-2])
def test_small_distance_regime_meets_the_plain_tolerance(torch, V, dtype, tau):
    """Draft and target rows that nearly agree (target noise tau of 1e-3 .. 3e-2: distances of
    3e-4 .. 2e-2, where d = sqrt(D_JS / ln 2) amplifies any error of D_JS): the kernels form
    D_JS from non-negative terms there, and d must meet 1e-4 WITHOUT the widening that
    tests/lockstep.py allows where fp32 cannot resolve D_JS."""
    import json
    import os
    from tests.lockstep import Lockstep, TOL as LTOL
    wl = synth.WORKLOADS["C3"].scaled(name=f"near_tau{tau:g}_V{V}", B=3, K=6, V=V, dtype=dtype, rounds=4,
                                      recipe="fixed_tau", tau0=tau, vanilla=False)
    ls = Lockstep(wl)
    rep = ls.run()
    s = rep.summary()
    print(wl.name, s["max_err"])
    log = os.environ.get("ADASD_PARITY_LOG")
    if log:
        with open(log, "a") as f:
            f.write(json.dumps(dict(workload=wl.name, V=V, tau=tau, max_err_dist=s["max_err"]["dist"],
                                    max_err_jsd=s["max_err"]["jsd"], dist_beyond_tol=s["dist_beyond_tol"])) + "\n")
    assert rep.positions == 4 * 3 * 7
    assert s["max_err"]["dist"] <= LTOL and rep.dist_beyond_tol == 0, s["max_err"]
    assert s["max_err"]["jsd"] <= 1e-7, s["max_err"]


def test_long_history_kde(torch):
    """Hundreds of rounds on a small vocabulary: long KDE lists, many rejections."""
    wl = synth.WORKLOADS["C3"].scaled(name="history", B=4, K=8, V=2048, rounds=300, vanilla=False)
    rep = run_lockstep(wl, check_lists_every=50)
    assert rep.n_rejections > 20


# ------------------------------------------------------------------ crafted edge cases

class Case:
    """One verify call on hand-made rows, with the oracle's answer beside it."""

    def __init__(self, torch, adasd, zd, zt, x, ut, ua, draft_len=None, dtype=None, **ctx_kw):
        B, K, V = zd.shape
        dtype = dtype or torch.float32
        self.torch, self.B, self.K, self.V = torch, B, K, V
        self.ctx = adasd.Context(B, V, K, dtype=adasd.ADASD_FP32 if dtype == torch.float32 else adasd.ADASD_BF16,
                                 list_capacity=256, **ctx_kw)
        dev = "cuda"
        self.zd = torch.tensor(zd, dtype=torch.float32).to(dtype).to(dev)
        self.zt = torch.tensor(zt, dtype=torch.float32).to(dtype).to(dev)
        self.x = torch.tensor(x, dtype=torch.int32, device=dev)
        self.ut = torch.tensor(ut, dtype=torch.float32, device=dev)
        self.ua = torch.tensor(ua, dtype=torch.float32, device=dev)
        self.dl = None if draft_len is None else torch.tensor(draft_len, dtype=torch.int32, device=dev)
        self.al = torch.full((B,), -9, dtype=torch.int32, device=dev)
        self.nt = torch.full((B,), -9, dtype=torch.int32, device=dev)
        self.rec = self.ctx.new_record()

    def verify(self, fuse=True):
        self.ctx.verify(self.zd, self.zt, self.x, self.ut, self.ua, self.al, self.nt, draft_len=self.dl,
                        record=self.rec, fuse_update=fuse)
        self.torch.cuda.synchronize()
        return {k: v.cpu().numpy() for k, v in self.rec.items()}

    def oracle_round(self, b, state, update=True):
        K_t = self.K if self.dl is None else int(self.dl[b])
        return oracle.verify_round(state, raw(self.zd[b], self.torch), raw(self.zt[b], self.torch),
                                   self.x[b, :K_t].cpu().numpy(), self.ut[b].cpu().numpy(),
                                   self.ua[b].cpu().numpy(), K_t=K_t, update=update)


# every crafted case runs on the generic kernels (small or fp32 rows) and on the streaming
# kernels (bf16 rows of a multiple of 8 logits, at least 8192 of them)
GENERIC_AND_STREAMING = [(1000, "float32"), (8200, "bfloat16")]


@pytest.mark.parametrize("V,dt", GENERIC_AND_STREAMING)
def test_identical_disjoint_and_onehot_rows(torch, adasd, V, dt):
    K = 4
    rng = np.random.default_rng(0)
    ninf = -np.inf
    zd = rng.normal(size=(1, K, V)).astype(np.float32) * 2
    zt = rng.normal(size=(1, K + 1, V)).astype(np.float32) * 2
    zt[0, 0] = zd[0, 0]                                   # identical rows: d == 0 exactly
    zd[0, 1, : V // 2] = ninf                             # disjoint supports: d == 1 exactly
    zt[0, 1, V // 2:] = ninf
    zd[0, 2, :] = ninf                                    # both one-hot on the same token,
    zt[0, 2, :] = ninf                                    # with different finite values: d == 0
    zd[0, 2, 17] = 5.0
    zt[0, 2, 17] = 7.0
    x = [[3, 600, 17, 5]]
    c = Case(torch, adasd, zd, zt, x, rng.random((1, K + 1)), np.full((1, K), 0.5), dtype=getattr(torch, dt))
    r = c.verify()
    st = oracle.SequenceState(capacity=64)
    o = c.oracle_round(0, st)
    assert r["jsd"][0, 0] == 0.0 and r["dist"][0, 0] == 0.0 and o["dist"][0] == 0.0
    # disjoint supports: exactly 1 on the device; the oracle's float64 sum is within rounding of 1
    assert r["dist"][0, 1] == 1.0 and abs(o["dist"][1] - 1.0) < 1e-12, (r["dist"][0, 1], o["dist"][1])
    assert abs(r["jsd"][0, 1] - math.log(2)) < 1e-6
    assert r["dist"][0, 2] == 0.0 and r["H_d"][0, 2] == 0.0 and r["H_t"][0, 2] == 0.0
    assert r["y"][0, 2] == 17
    for k in ("H_d", "jsd", "dist"):
        assert np.allclose(r[k][0], o[k], atol=TOL), k
    assert np.allclose(r["H_t"][0], o["H_t"], atol=TOL)
    assert list(r["y"][0]) == list(o["y"])
    assert int(c.al[0]) == o["accept_len"] and int(c.nt[0]) == o["next_token"]
    g = c.ctx.state_export(0)
    LE, LA, LR = st.lists()
    assert (len(g["LE"]), len(g["LA"]), len(g["LR"])) == (len(LE), len(LA), len(LR))
    assert c.ctx.status() == 0


def test_entropy_closed_forms_on_device(torch, adasd):
    # fp32 rows take the generic kernel, long bf16 rows the streaming one
    for V, dt in ((4, "float32"), (1000, "float32"), (128256, "float32"), (8200, "bfloat16"), (128256, "bfloat16")):
        ctx = adasd.Context(2, V, 1, dtype=adasd.ADASD_FP32 if dt == "float32" else adasd.ADASD_BF16,
                            list_capacity=8)
        z = torch.zeros((2, V), dtype=getattr(torch, dt), device="cuda")
        z[1, :] = -float("inf")
        z[1, V // 3] = 2.5                                      # one-hot
        H = torch.zeros(2, device="cuda")
        lse = torch.zeros(2, device="cuda")
        tok = torch.zeros(2, dtype=torch.int32, device="cuda")
        u = torch.tensor([0.5, 0.99], device="cuda")
        stop = torch.zeros(2, dtype=torch.uint8, device="cuda")
        ctx.draft_entropy(z, H, u=u, token_out=tok, lse_out=lse, stop_out=stop)
        torch.cuda.synchronize()
        assert abs(float(H[0]) - math.log(V)) < TOL and abs(float(lse[0]) - math.log(V)) < TOL
        assert float(H[1]) == 0.0 and abs(float(lse[1]) - 2.5) < 1e-6
        assert int(tok[0]) == V // 2 and int(tok[1]) == V // 3
        assert int(stop[0]) == 1 and int(stop[1]) == 0           # H > T_G = 0 is strict


@pytest.mark.parametrize("V", [3000, 8200])
def test_windows_zero_to_kmax_and_inactive_rows(torch, adasd, V):
    K, B = 32, 5
    rng = np.random.default_rng(4)
    zd = rng.normal(size=(B, K, V)).astype(np.float32) * 3
    zt = zd[:, :, :] + rng.normal(size=(B, K, V)).astype(np.float32)
    zt = np.concatenate([zt, rng.normal(size=(B, 1, V)).astype(np.float32)], axis=1)
    draft_len = [0, 1, 7, 31, 32]
    x = rng.integers(0, V, size=(B, K))
    c = Case(torch, adasd, zd, zt, x, rng.random((B, K + 1)), rng.random((B, K)), draft_len=draft_len,
             dtype=torch.bfloat16)
    r = c.verify()
    for b in range(B):
        st = oracle.SequenceState(capacity=64)
        o = c.oracle_round(b, st)
        K_t = draft_len[b]
        assert int(c.al[b]) == o["accept_len"] and int(c.nt[b]) == o["next_token"], b
        assert np.allclose(r["dist"][b, :K_t], o["dist"], atol=TOL)
        assert np.isnan(r["dist"][b, K_t:]).all()                # untouched beyond the window
        assert list(r["y"][b, : K_t + 1]) == list(o["y"])
        assert (r["y"][b, K_t + 1:] == -2).all()
        assert int(r["draft_len"][b]) == K_t
    assert c.ctx.status() == 0


@pytest.mark.parametrize("V,dt", [(500, "float32"), (8200, "bfloat16")])
def test_nan_and_all_minus_inf_rows_set_status_not_faults(torch, adasd, V, dt):
    K = 2
    rng = np.random.default_rng(5)
    zd = rng.normal(size=(2, K, V)).astype(np.float32)
    zt = rng.normal(size=(2, K + 1, V)).astype(np.float32)
    zd[0, 1, 100] = np.nan
    zt[1, 0, :] = -np.inf
    c = Case(torch, adasd, zd, zt, [[1, 2], [3, 4]], rng.random((2, K + 1)), rng.random((2, K)),
             dtype=getattr(torch, dt))
    r = c.verify()
    assert np.isnan(r["H_d"][0, 1]) and np.isnan(r["jsd"][0, 1])
    assert np.isnan(r["H_t"][1, 0]) and r["y"][1, 0] == -1
    assert np.isfinite(r["H_d"][0, 0]) and np.isfinite(r["H_t"][1, 1])
    assert c.ctx.status() & adasd.STATUS_NAN
    assert c.ctx.status() == 0                                   # reading clears it


@pytest.mark.parametrize("V,dt", [(500, "float32"), (8200, "bfloat16")])
def test_unusable_row_with_fused_update_leaves_thresholds_finite(torch, adasd, V, dt):
    """A round whose first candidate has a NaN draft row (fused update on): the candidate is
    rejected, nothing of it is recorded, T_G keeps its value; the clean round after it updates
    the state exactly as the oracle does, and the draft-stop check still works."""
    K = 3
    rng = np.random.default_rng(31)
    zd = rng.normal(size=(1, K, V)).astype(np.float32) * 2
    zt = np.concatenate([zd + rng.normal(size=(1, K, V)).astype(np.float32),
                         rng.normal(size=(1, 1, V)).astype(np.float32)], axis=1)
    x = [[1, 2, 3]]
    ut, ua = rng.random((1, K + 1)), np.full((1, K), 0.999)
    st = oracle.SequenceState(capacity=64)
    c = Case(torch, adasd, zd, zt, x, ut, ua, dtype=getattr(torch, dt))
    o = c.oracle_round(0, st)                              # a clean round first: one rejection recorded
    c.verify()
    assert o["rejected"] and st.nE.value == 1
    T0 = st.T_G.value
    clean_d = c.zd.clone()
    c.zd[0, 0, 100] = float("nan")
    o = c.oracle_round(0, st)
    r = c.verify()
    assert c.ctx.status() & adasd.STATUS_NAN
    assert np.isnan(r["H_d"][0, 0]) and int(c.al[0]) == 0 == o["accept_len"] and int(r["rejected"][0]) == 1
    T, nE, nA, nR = (t.cpu().numpy() for t in c.ctx.get_thresholds())
    assert (int(nE[0]), int(nA[0]), int(nR[0])) == (st.nE.value, st.nA.value, st.nR.value) == (1, 0, st.nR.value)
    assert np.isfinite(T[0]) and abs(float(T[0]) - T0) < TOL and st.T_G.value == T0
    c.zd.copy_(clean_d)                                    # a clean round again: the state moves on
    o = c.oracle_round(0, st)
    c.verify()
    T, nE, nA, nR = (t.cpu().numpy() for t in c.ctx.get_thresholds())
    assert (int(nE[0]), int(nA[0]), int(nR[0])) == (st.nE.value, st.nA.value, st.nR.value) and int(nE[0]) == 2
    assert np.isfinite(T[0]) and abs(float(T[0]) - st.T_G.value) < TOL
    assert c.ctx.status() == 0


@pytest.mark.parametrize("V", [4096, 8200])      # generic kernel with the CTA-wide tail; streaming kernel with warp tails
def test_fused_update_equals_verify_then_update(torch, adasd, V):
    wl = synth.WORKLOADS["C3"].scaled(B=6, K=6, V=V, rounds=30)
    gs = synth.GpuSynth(wl)
    B, K, V = wl.B, wl.K, wl.V
    zd = torch.empty((B, K, V), dtype=torch.bfloat16, device="cuda")
    zt = torch.empty((B, K + 1, V), dtype=torch.bfloat16, device="cuda")
    ctxs = [adasd.Context(B, V, K, list_capacity=512) for _ in range(2)]
    outs = [[torch.zeros(B, dtype=torch.int32, device="cuda") for _ in range(2)] for _ in range(2)]
    recs = [c.new_record() for c in ctxs]
    rng = np.random.default_rng(8)
    for r in range(wl.rounds):
        gs.draft_rows(r, zd)
        gs.target_rows(r, zt)
        x = torch.tensor(rng.integers(0, V, size=(B, K)), dtype=torch.int32, device="cuda")
        ut = torch.tensor(rng.random((B, K + 1)), dtype=torch.float32, device="cuda")
        ua = torch.tensor(rng.random((B, K)), dtype=torch.float32, device="cuda")
        # make about half of the draft tokens agree with the target sample
        ctxs[0].verify(zd, zt, x, ut, ua, outs[0][0], outs[0][1], record=recs[0], fuse_update=False)
        x = torch.where(torch.tensor(rng.random((B, K)) < 0.6, device="cuda"), recs[0]["y"][:, :K], x)
        ctxs[0].verify(zd, zt, x, ut, ua, outs[0][0], outs[0][1], record=recs[0], fuse_update=True)
        ctxs[1].verify(zd, zt, x, ut, ua, outs[1][0], outs[1][1], record=recs[1], fuse_update=False)
        ctxs[1].update_thresholds(recs[1])
        assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    for b in range(B):
        a, c = ctxs[0].state_export(b), ctxs[1].state_export(b)
        assert a["T_G"] == c["T_G"]
        for k in ("LE", "LA", "LR"):
            assert np.array_equal(a[k], c[k]), k
    assert sum(len(ctxs[0].state_export(b)["LR"]) for b in range(B)) > 0


def test_state_export_import_reset_roundtrip(torch, adasd):
    ctx = adasd.Context(3, 100, 4, list_capacity=16)
    LE, LA, LR = [1.5, 2.5], [0.1, 0.2, 0.3], [0.7, 0.9]
    ctx.state_import(1, 0.0, LE, LA, LR)
    g = ctx.state_export(1)
    assert np.allclose(g["LE"], LE) and np.allclose(g["LA"], LA) and np.allclose(g["LR"], LR)
    assert abs(g["T_G"] - 2.0) < 1e-7                      # recomputed as mean(L_E^R)
    T, nE, nA, nR = (t.cpu().numpy() for t in ctx.get_thresholds())
    assert list(nE) == [0, 2, 0] and list(nA) == [0, 3, 0] and list(nR) == [0, 2, 0]
    assert abs(T[1] - 2.0) < 1e-7 and T[0] == 0
    with pytest.raises(adasd.AdasdError):
        ctx.state_import(1, 0.0, list(range(17)), [], [])   # beyond the capacity
    with pytest.raises(adasd.AdasdError):
        ctx.state_export(3)
    ctx.reset(torch.tensor([1], dtype=torch.int32, device="cuda"))
    g = ctx.state_export(1)
    assert g["T_G"] == 0.0 and len(g["LE"]) == len(g["LA"]) == len(g["LR"]) == 0


def test_host_detected_errors_launch_nothing(torch, adasd):
    ctx = adasd.Context(2, 1000, 4)
    z = torch.zeros((2, 5, 1000), dtype=torch.bfloat16, device="cuda")
    i = torch.zeros((2, 5), dtype=torch.int32, device="cuda")
    f = torch.zeros((2, 5), dtype=torch.float32, device="cuda")
    h = ctx.handle
    p = lambda t: t.data_ptr()
    assert adasd.adasd_verify(h, None, p(z), 5000, 1000, 5000, 1000, p(i), None, p(f), p(f), p(i), p(i),
                              None, 0, None) == -1
    assert adasd.adasd_verify(h, p(z), p(z), 5000, 999, 5000, 1000, p(i), None, p(f), p(f), p(i), p(i),
                              None, 0, None) == -3
    assert adasd.adasd_verify(h, p(z), p(z), 5000, 1000, 5000, 1000, p(i), None, p(f), p(f), p(i), p(i),
                              None, 8, None) == -3
    assert adasd.adasd_draft_entropy(h, p(z), 1000, p(f), None, p(f), None, None, None, None, None) == -1
    assert adasd.adasd_draft_entropy(h, p(z), 10, None, None, p(f), None, None, None, None, None) == -3
    assert adasd.adasd_vanilla_verify(h, p(z), p(z), 5000, 1000, 5000, 1000, p(i), None, p(f), None,
                                      p(i), p(i), None, None) == -1
    torch.cuda.synchronize()
    assert ctx.status() == 0


def test_unaligned_rows_take_the_scalar_path(torch, adasd):
    """Row stride of 1001 bf16 elements: neither base nor stride is 16-byte aligned."""
    V, K, B = 1001, 3, 2
    rng = np.random.default_rng(6)
    zd = rng.normal(size=(B, K, V)).astype(np.float32) * 2
    zt = np.concatenate([zd + rng.normal(size=(B, K, V)).astype(np.float32) * 0.5,
                         rng.normal(size=(B, 1, V)).astype(np.float32)], axis=1)
    c = Case(torch, adasd, zd, zt, rng.integers(0, V, size=(B, K)), rng.random((B, K + 1)),
             rng.random((B, K)), dtype=torch.bfloat16)
    assert (c.zd.stride(1) * 2) % 16 != 0
    r = c.verify()
    for b in range(B):
        o = c.oracle_round(b, oracle.SequenceState(capacity=64))
        for k in ("H_d", "jsd", "dist"):
            assert np.allclose(r[k][b], o[k], atol=TOL), k
        assert list(r["y"][b]) == list(o["y"])


def test_repeatable_bitwise(torch, adasd):
    wl = synth.WORKLOADS["C3"].scaled(B=8, K=8, V=128256, rounds=2)
    gs = synth.GpuSynth(wl)
    zd = torch.empty((8, 8, wl.V), dtype=torch.bfloat16, device="cuda")
    zt = torch.empty((8, 9, wl.V), dtype=torch.bfloat16, device="cuda")
    gs.draft_rows(0, zd)
    gs.target_rows(0, zt)
    x = torch.zeros((8, 8), dtype=torch.int32, device="cuda")
    ut = torch.rand((8, 9), device="cuda")
    ua = torch.rand((8, 8), device="cuda")
    res = []
    for _ in range(2):
        ctx = adasd.Context(8, wl.V, 8)
        rec = ctx.new_record()
        al = torch.zeros(8, dtype=torch.int32, device="cuda")
        nt = torch.zeros(8, dtype=torch.int32, device="cuda")
        ctx.verify(zd, zt, x, ut, ua, al, nt, record=rec)
        torch.cuda.synchronize()
        res.append({k: v.clone() for k, v in rec.items()})
    for k in res[0]:
        a, b = res[0][k], res[1][k]
        assert torch.equal(a.view(torch.int32), b.view(torch.int32)), k


# ------------------------------------------------------------------ CUDA graph replay

@pytest.mark.parametrize("warpers", [None, (0.8, 40, 0.95)])
def test_adaptive_round_in_a_cuda_graph_replays_like_eager_calls(torch, adasd, warpers):
    """(With and without an adjusted distribution: its cutoff kernels are launches like the others.)
    One whole adaptive round (inputs of the round the device counter names, draft steps
    with the stop check, verification with the fused threshold update) is captured ONCE in a
    CUDA graph; replaying it R times must leave the sequences in exactly the state that the
    same R rounds issued call by call leave them in: the hot calls launch from device-resident
    state only, with nothing decided on the host in between."""
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    # 8200 bf16 logits take the streaming kernels; windows of up to 6 from the stop check
    wl = synth.WORKLOADS["C5"].scaled(name="graph", B=24, K=6, V=8200, rounds=12)
    B, K, V, R = wl.B, wl.K, wl.V, 12

    def build():
        ctx = adasd.Context(B, V, K, dtype=wl.dtype, list_capacity=256, device=0)
        if warpers:
            ctx.set_warpers(*warpers)
        gs = synth.GpuSynth(wl, str(dev))
        f32, i32 = dict(dtype=torch.float32, device=dev), dict(dtype=torch.int32, device=dev)
        zd = torch.empty((B, K, V), dtype=torch.bfloat16, device=dev)
        zt = torch.empty((B, K + 1, V), dtype=torch.bfloat16, device=dev)
        U = gs.new_round_uniforms()
        ud = torch.empty((K, B), **f32)
        Hk, tokk = torch.zeros((K, B), **f32), torch.zeros((K, B), **i32)
        stopk = torch.zeros((K, B), dtype=torch.uint8, device=dev)
        active = torch.ones(B, dtype=torch.uint8, device=dev)
        dlen, x = torch.zeros(B, **i32), torch.zeros((B, K), **i32)
        al, nt = torch.zeros(B, **i32), torch.zeros(B, **i32)
        acc = torch.zeros((3, B), dtype=torch.int64, device=dev)   # sums of windows, accept_len, tokens

        def one_round():
            gs.draft_rows(0, zd, use_round_dev=True)
            gs.target_rows(0, zt, use_round_dev=True)
            gs.round_uniforms(0, U, use_round_dev=True)
            ud.copy_(U["draft"].T)
            dlen.zero_()
            active.fill_(1)
            for k in range(K):
                ctx.draft_entropy(zd[:, k, :], Hk[k], u=ud[k], token_out=tokk[k], active=active,
                                  stop_out=stopk[k], draft_len=dlen, row_stride=K * V)
            x.copy_(tokk.T)
            ctx.verify(zd, zt, x, U["target"], U["accept"], al, nt, draft_len=dlen, fuse_update=True)
            acc[0] += dlen
            acc[1] += al
            acc[2] += nt
            gs.advance_round(1)

        def state():
            torch.cuda.synchronize()
            T, nE, nA, nR = ctx.get_thresholds()
            torch.cuda.synchronize()
            return dict(T=T.cpu(), nE=nE.cpu(), nA=nA.cpu(), nR=nR.cpu(), acc=acc.cpu(), al=al.cpu(),
                        nt=nt.cpu(), dlen=dlen.cpu(), status=ctx.status(), round=int(gs.round_dev.item()))
        return ctx, gs, one_round, state, acc

    # call by call
    ctx, gs, one_round, state, acc = build()
    for _ in range(R):
        one_round()
    eager = state()
    ctx.close()
    assert eager["status"] == 0 and eager["round"] == R
    assert int(eager["nE"].sum()) > 0 and len(set(eager["dlen"].tolist())) >= 2   # rejections and stops happened

    # captured once, replayed R times
    ctx, gs, one_round, state, acc = build()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        one_round()                              # untimed first pass outside the capture
        torch.cuda.synchronize()
        ctx.reset()
        gs.round_dev.zero_()
        acc.zero_()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            one_round()
        for _ in range(R):
            g.replay()
        torch.cuda.synchronize()
    replayed = state()
    ctx.close()
    assert replayed["status"] == 0 and replayed["round"] == R
    for key in ("T", "nE", "nA", "nR", "acc", "al", "nt", "dlen"):
        assert torch.equal(eager[key], replayed[key]), key


# the third case repeats the four sequences 56 times: 224 * 7 rows are enough for the three-step
# path (streaming log-sum-exps, accept test, sampling of one position per sequence)
@pytest.mark.parametrize("V,dt,tile", [(1000, "float32", 1), (8200, "bfloat16", 1), (8200, "bfloat16", 56)])
def test_vanilla_mode_crafted_rows(torch, adasd, V, dt, tile):
    """Vanilla speculative sampling on hand-made rows: identical rows accept with alpha = 1 and
    the bonus row is sampled; a draft token the target gives no mass is rejected and the
    residual is the target distribution; an ordinary rejection resamples from max(0, p - q);
    a shorter window takes its own bonus row."""
    K, B = 3, 4
    tdt = getattr(torch, dt)
    rng = np.random.default_rng(11)
    zd = rng.normal(size=(B, K, V)).astype(np.float32) * 2
    zt = zd + rng.normal(size=(B, K, V)).astype(np.float32)
    zt = np.concatenate([zt, rng.normal(size=(B, 1, V)).astype(np.float32) * 2], axis=1)
    zt[0, :K] = zd[0]                                      # b0: identical rows everywhere
    zd[1, 0, :] = -np.inf                                  # b1: one-hot rows on different tokens
    zt[1, 0, :] = -np.inf
    zd[1, 0, 7] = 1.5
    zt[1, 0, 40] = -3.0
    zt[2, 0] = zd[2, 0]                                    # b2: accepted, then an ordinary rejection
    x = rng.integers(0, V, size=(B, K)).astype(np.int32)
    x[1, 0] = 7
    x[2, 1] = 123
    zd[2, 1, 123] += 8.0                                   # the draft likes its token far more than the target
    ua = np.full((B, K), 0.5, dtype=np.float32)
    ua[2, 1] = 0.9999
    ua[3, 0] = 0.0
    ur = np.array([0.3, 0.9, 0.37, 0.62], dtype=np.float32)
    draft_len = [K, K, K, 1] * tile
    zd, zt, x, ua, ur = (np.concatenate([a] * tile, axis=0) for a in (zd, zt, x, ua, ur))
    B = B * tile
    dev = "cuda"
    ctx = adasd.Context(B, V, K, dtype=adasd.ADASD_FP32 if dt == "float32" else adasd.ADASD_BF16, list_capacity=8)
    zd_g = torch.tensor(zd).to(tdt).to(dev)
    zt_g = torch.tensor(zt).to(tdt).to(dev)
    x_g = torch.tensor(x, device=dev)
    al = torch.full((B,), -9, dtype=torch.int32, device=dev)
    nt = torch.full((B,), -9, dtype=torch.int32, device=dev)
    alpha = torch.full((B, K), float("nan"), dtype=torch.float32, device=dev)
    ctx.vanilla_verify(zd_g, zt_g, x_g, torch.tensor(ua, device=dev), torch.tensor(ur, device=dev), al, nt,
                       draft_len=torch.tensor(draft_len, dtype=torch.int32, device=dev), alpha_out=alpha)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    alpha_h = alpha.cpu().numpy()
    for b in sorted(set(range(4)) | set(range(B - 4, B))):
        K_t = draft_len[b]
        o = oracle.vanilla_round(raw(zd_g[b, :K_t], torch), raw(zt_g[b], torch), x[b, :K_t], ua[b, :K_t], float(ur[b]))
        assert int(al[b]) == o["accept_len"], (b, int(al[b]), o)
        assert o["margin"] > 1e-6 and int(nt[b]) == o["next_token"], (b, int(nt[b]), o)
        n_seen = min(o["accept_len"] + 1, K_t)
        assert np.allclose(alpha_h[b, :n_seen], o["alpha"][:n_seen], atol=TOL), (b, alpha_h[b], o["alpha"])
    assert int(al[0]) == K and (alpha_h[0] == 1.0).all()
    assert int(al[1]) == 0 and alpha_h[1, 0] == 0.0 and int(nt[1]) == 40
    assert int(al[2]) == 1 and int(al[3]) == 1
    # every copy of a sequence gets the same answers
    assert torch.equal(al.view(tile, 4), al[:4].expand(tile, 4)) and torch.equal(nt.view(tile, 4), nt[:4].expand(tile, 4))


def test_vanilla_three_step_path_flags_nan_and_empty_rows(torch, adasd):
    """NaN in a draft row and a target row without a finite logit, among enough rows for the
    three-step path: the position counts as rejected, its alpha is NaN, no token is drawn (-1),
    the status flag is raised, and every other sequence is unaffected."""
    V, K, B = 8200, 3, 224
    rng = np.random.default_rng(21)
    zd = rng.normal(size=(B, K, V)).astype(np.float32) * 2
    zt = np.concatenate([zd + rng.normal(size=(B, K, V)).astype(np.float32),
                         rng.normal(size=(B, 1, V)).astype(np.float32)], axis=1)
    zt[:, :K] = zd                                         # identical rows: everything is accepted ...
    zd[17, 1, 4000] = np.nan                               # ... except where a row is unusable
    zt[200, 0, :] = -np.inf
    dev = "cuda"
    ctx = adasd.Context(B, V, K, list_capacity=8)
    zd_g = torch.tensor(zd).to(torch.bfloat16).to(dev)
    zt_g = torch.tensor(zt).to(torch.bfloat16).to(dev)
    x = torch.tensor(rng.integers(0, V, size=(B, K)).astype(np.int32), device=dev)
    ua = torch.full((B, K), 0.5, device=dev)
    ur = torch.full((B,), 0.25, device=dev)
    al = torch.full((B,), -9, dtype=torch.int32, device=dev)
    nt = torch.full((B,), -9, dtype=torch.int32, device=dev)
    alpha = torch.zeros((B, K), device=dev)
    ctx.vanilla_verify(zd_g, zt_g, x, ua, ur, al, nt, alpha_out=alpha)
    torch.cuda.synchronize()
    assert ctx.status() == adasd.STATUS_NAN
    assert int(al[17]) == 1 and int(nt[17]) == -1 and torch.isnan(alpha[17, 1]) and float(alpha[17, 0]) == 1.0
    assert int(al[200]) == 0 and int(nt[200]) == -1 and torch.isnan(alpha[200, 0])
    ok = torch.ones(B, dtype=torch.bool, device=dev)
    ok[17] = ok[200] = False
    assert (al[ok] == K).all() and (nt[ok] >= 0).all() and (nt[ok] < V).all() and (alpha[ok] == 1.0).all()


def test_padded_rows_on_the_streaming_path(torch, adasd):
    """Rows cut out of a wider buffer (row stride V + 24, a gap between sequences; everything
    still 16-byte aligned) take the streaming kernels with the caller's strides: same results,
    bit for bit, as the contiguous copy."""
    wl = synth.WORKLOADS["C3"].scaled(name="padded", B=3, K=4, V=8200, rounds=2)
    B, K, V = wl.B, wl.K, wl.V
    gs = synth.GpuSynth(wl)
    zd = torch.empty((B, K, V), dtype=torch.bfloat16, device="cuda")
    zt = torch.empty((B, K + 1, V), dtype=torch.bfloat16, device="cuda")
    gs.draft_rows(0, zd)
    gs.target_rows(0, zt)
    wide_d = torch.full((B, K + 1, V + 24), 7.0, dtype=torch.bfloat16, device="cuda")   # one spare row per sequence
    wide_t = torch.full((B, K + 2, V + 24), 7.0, dtype=torch.bfloat16, device="cuda")
    pd, pt = wide_d[:, :K, :V], wide_t[:, :K + 1, :V]
    pd.copy_(zd)
    pt.copy_(zt)
    assert pd.stride() == ((K + 1) * (V + 24), V + 24, 1) and not pd.is_contiguous()
    U = gs.new_round_uniforms()
    gs.round_uniforms(0, U)
    out = []
    for d_, t_ in ((zd, zt), (pd, pt)):
        ctx = adasd.Context(B, V, K, list_capacity=64)
        rec = ctx.new_record()
        i32 = dict(dtype=torch.int32, device="cuda")
        H = torch.zeros((K, B), device="cuda")
        tok = torch.zeros((K, B), **i32)
        for k in range(K):
            ctx.draft_entropy(d_[:, k, :], H[k], u=U["draft"][:, k].contiguous(), token_out=tok[k])
        x = tok.T.contiguous()
        al, nt, val, vnt = (torch.zeros(B, **i32) for _ in range(4))
        ctx.verify(d_, t_, x, U["target"], U["accept"], al, nt, record=rec)
        ctx.vanilla_verify(d_, t_, x, U["vanilla_accept"], U["resample"], val, vnt)
        torch.cuda.synchronize()
        assert ctx.status() == 0
        out.append(dict(H=H, tok=tok, al=al, nt=nt, val=val, vnt=vnt, **{k: v.clone() for k, v in rec.items()}))
    for k in out[0]:
        a, b = out[0][k], out[1][k]
        assert torch.equal(a.view(torch.int32) if a.dtype == torch.float32 else a,
                           b.view(torch.int32) if b.dtype == torch.float32 else b), k
    assert (wide_d[:, K, :] == 7.0).all() and (wide_d[:, :, V:] == 7.0).all()        # nothing written around the rows


def test_full_lists_set_the_capacity_flag_and_keep_running(torch, adasd):
    """A list that is full skips the append and raises ADASD_STATUS_CAPACITY; sizes stay at the
    capacity and later rounds still run."""
    wl = synth.WORKLOADS["C3"].scaled(name="cap", B=4, K=6, V=8200, rounds=40, vanilla=False)
    B, K, V = wl.B, wl.K, wl.V
    cap = 8
    ctx = adasd.Context(B, V, K, list_capacity=cap)
    gs = synth.GpuSynth(wl)
    zd = torch.empty((B, K, V), dtype=torch.bfloat16, device="cuda")
    zt = torch.empty((B, K + 1, V), dtype=torch.bfloat16, device="cuda")
    U = gs.new_round_uniforms()
    i32 = dict(dtype=torch.int32, device="cuda")
    al, nt = torch.zeros(B, **i32), torch.zeros(B, **i32)
    x = torch.zeros((B, K), **i32)
    seen = 0
    for r in range(wl.rounds):
        gs.draft_rows(r, zd)
        gs.target_rows(r, zt)
        gs.round_uniforms(r, U)
        ctx.verify(zd, zt, x, U["target"], U["accept"], al, nt, fuse_update=True)
        seen |= ctx.status()
        assert 0 <= int(al.min()) and int(al.max()) <= K and 0 <= int(nt.min()) and int(nt.max()) < V
    T, nE, nA, nR = ctx.get_thresholds()
    torch.cuda.synchronize()
    assert seen & adasd.STATUS_CAPACITY and not (seen & ~adasd.STATUS_CAPACITY)
    assert int(nR.max()) <= cap and int(nA.max()) <= cap and int(nR.max()) == cap
    # L_E^R is capped the same way, and T_G stays the mean of what it holds: a checkpoint
    # round trip leaves it where it was
    assert int(nE.max()) == cap
    for b in range(B):
        before = ctx.state_export(b)
        ctx.state_import(b, before["T_G"], before["LE"], before["LA"], before["LR"])
        after = ctx.state_export(b)
        assert abs(after["T_G"] - before["T_G"]) < 1e-6 and len(after["LE"]) == len(before["LE"])
        assert abs(before["T_G"] - float(np.mean(before["LE"]))) < 1e-5
