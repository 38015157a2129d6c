"""GPU parity of the adjusted distribution (Sec. 2.1.1: temperature, top-k, top-p) against the
float64 oracle: the same lockstep rounds as the other parity tests, with the oracle working on
the rows `oracle.warp` returns and the library on the raw rows with `adasd_set_warpers`."""
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


def raw(t, torch):
    return t.view(torch.int16).cpu().numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.cpu().numpy()


@pytest.mark.parametrize("V,dtype,warpers", [
    (8200, synth.BF16, (0.7, 0, 1.0)),            # temperature alone
    (8200, synth.BF16, (1.0, 40, 1.0)),           # top-k alone
    (8200, synth.BF16, (1.0, 0, 0.9)),            # top-p alone
    (40000, synth.BF16, (0.8, 50, 0.95)),         # all three, streaming-size rows
    (4099, synth.BF16, (1.3, 17, 0.8)),           # unaligned rows
    (1003, synth.FP32, (0.6, 9, 0.85)),           # fp32 rows
    (32000, synth.FP32, (1.0, 0, 0.92)),
])
def test_lockstep_rounds_under_warpers(torch, V, dtype, warpers):
    from tests.lockstep import Lockstep
    wl = synth.WORKLOADS["C3"].scaled(name=f"warp_{V}_{warpers}", B=5, K=5, V=V, dtype=dtype, rounds=30)
    rep = Lockstep(wl, min_kde_samples=3, check_lists_every=10, warpers=warpers).run()
    s = rep.summary()
    assert s["flips"] <= s["near_threshold"] + s["tie_flips"], s
    assert s["warp_near"] <= 3 and s["positions"] > 600, s
    assert len(rep.accept_hist) >= 3, s


def test_many_rows_take_the_three_kernel_vanilla_path_under_warpers(torch):
    """352 rows a round: adasd_vanilla_verify runs row_lse_kernel, vanilla_accept_kernel and
    vanilla_sample_kernel, adasd_verify the warp-specialised kernel, all on the adjusted rows."""
    from tests.lockstep import Lockstep
    wl = synth.WORKLOADS["C3"].scaled(name="warp_manyrows", B=32, K=5, V=8200, rounds=8)
    rep = Lockstep(wl, follow=[0, 7, 13, 21, 30, 31], min_kde_samples=3, check_lists_every=4,
                   warpers=(0.8, 50, 0.95)).run()
    s = rep.summary()
    assert s["flips"] <= s["near_threshold"] + s["tie_flips"] and s["warp_near"] <= 2, s
    assert len(rep.vanilla_accept_hist) >= 3, s


def test_adaptive_windows_under_warpers(torch):
    from tests.lockstep import Lockstep
    wl = synth.WORKLOADS["C5"].scaled(name="warp_adaptive", B=6, K=8, V=8200, rounds=40)
    rep = Lockstep(wl, min_kde_samples=3, check_lists_every=10, warpers=(0.9, 64, 0.97)).run()
    s = rep.summary()
    assert s["flips"] <= s["near_threshold"] + s["tie_flips"] and len(rep.window_hist) >= 3, s


def test_top_1_puts_every_distance_on_an_exact_end(torch, adasd):
    """Sec. 4.4: many distances are exactly 0 or 1.  With top_k = 1 both rows are one-hot, so the
    distance is exactly 0 where draft and target agree on the most probable token and exactly
    1 where they do not, entropies are exactly 0, and nothing enters the distance lists."""
    B, K, V = 6, 6, 8200
    wl = synth.WORKLOADS["C3"].scaled(name="top1", B=B, K=K, V=V, rounds=4, recipe="fixed_tau", tau0=0.4)
    gs = synth.GpuSynth(wl)
    ctx = adasd.Context(B, V, K, list_capacity=64)
    ctx.set_warpers(1.0, 1, 1.0)
    zd = torch.empty((B, K, V), dtype=torch.bfloat16, device="cuda")
    zt = torch.empty((B, K + 1, V), dtype=torch.bfloat16, device="cuda")
    i32 = dict(dtype=torch.int32, device="cuda")
    seen = set()
    for r in range(wl.rounds):
        gs.draft_rows(r, zd)
        gs.target_rows(r, zt)
        U = synth.round_uniforms_cpu(wl, r)
        x = zd.float().argmax(dim=2).to(torch.int32)
        rec = ctx.new_record()
        al, nt = torch.zeros(B, **i32), torch.zeros(B, **i32)
        ctx.verify(zd, zt, x, torch.tensor(U["target"], device="cuda"), torch.tensor(U["accept"], device="cuda"),
                   al, nt, record=rec, fuse_update=True)
        torch.cuda.synchronize()
        d = rec["dist"].cpu().numpy()
        Hd, Ht = rec["H_d"].cpu().numpy(), rec["H_t"].cpu().numpy()
        zd_h, zt_h = raw(zd, torch), raw(zt, torch)
        for b in range(B):
            for i in range(K):
                q = oracle.softmax(oracle.warp(zd_h[b, i], 1.0, 1, 1.0)[0])[0]
                p = oracle.softmax(oracle.warp(zt_h[b, i], 1.0, 1, 1.0)[0])[0]
                want = oracle.js_distance_rows(p, q)[0]
                if want in (0.0, 1.0):                       # (a tie for the largest logit keeps two tokens)
                    assert d[b, i] == want, (r, b, i, d[b, i], want)
                    seen.add(want)
                else:
                    assert abs(d[b, i] - want) < TOL
                    seen.add(0.5)
                assert abs(Hd[b, i] - oracle.entropy(q)) < TOL and abs(Ht[b, i] - oracle.entropy(p)) < TOL
                if np.count_nonzero(q) == 1 and np.count_nonzero(p) == 1:
                    assert Hd[b, i] == 0.0 and Ht[b, i] == 0.0
    assert {0.0, 1.0} <= seen
    assert ctx.status() == 0


def test_identity_settings_change_nothing_and_bad_settings_are_refused(torch, adasd):
    B, K, V = 4, 4, 40000
    wl = synth.WORKLOADS["C3"].scaled(name="ident", B=B, K=K, V=V, rounds=1)
    gs = synth.GpuSynth(wl)
    zd = torch.empty((B, K, V), dtype=torch.bfloat16, device="cuda")
    zt = torch.empty((B, K + 1, V), dtype=torch.bfloat16, device="cuda")
    gs.draft_rows(0, zd)
    gs.target_rows(0, zt)
    U = synth.round_uniforms_cpu(wl, 0)
    x = zd.float().argmax(dim=2).to(torch.int32)
    outs = []
    for setting in (None, (1.0, 0, 1.0), (1.0, V, 1.0)):
        ctx = adasd.Context(B, V, K, list_capacity=64)
        if setting:
            ctx.set_warpers(*setting)
        rec = ctx.new_record()
        al = torch.zeros(B, dtype=torch.int32, device="cuda")
        nt = torch.zeros(B, dtype=torch.int32, device="cuda")
        ctx.verify(zd, zt, x, torch.tensor(U["target"], device="cuda"), torch.tensor(U["accept"], device="cuda"),
                   al, nt, record=rec, fuse_update=False)
        torch.cuda.synchronize()
        outs.append({k: v.clone() for k, v in rec.items()})
    for k in outs[0]:
        for o in outs[1:]:
            assert torch.equal(torch.nan_to_num(outs[0][k].float(), nan=-7.0), torch.nan_to_num(o[k].float(), nan=-7.0)), k
    ctx = adasd.Context(B, V, K, list_capacity=64)
    for bad in ((0.0, 0, 1.0), (-1.0, 0, 1.0), (float("nan"), 0, 1.0), (float("inf"), 0, 1.0),
                (1.0, 0, 0.0), (1.0, 0, 1.5), (1.0, 0, float("nan"))):
        assert adasd.adasd_set_warpers(ctx.handle, *bad) == adasd.ERR_SHAPE, bad
    assert adasd.adasd_set_warpers(ctx.handle, 1.0, -5, 1.0) == 0          # a negative k is "off"
    assert adasd.adasd_set_warpers(None, 1.0, 0, 1.0) == adasd.ERR_NULL


@pytest.mark.parametrize("warpers", [(1.0, 50, 1.0), (0.9, 0, 0.9), (1.1, 300, 0.97)])
def test_a_value_that_fills_most_of_a_row_does_not_break_the_cut(torch, adasd, warpers):
    """100000 tokens: one logit value taken by more than 65536 of them (the one-pass kernel counts
    occurrences in 16 bits and must hand such a row over), a row that is one value throughout, and
    ordinary rows in between; entropy, log-sum-exp and the sampled token against the oracle."""
    B, V = 5, 100000
    rng = np.random.default_rng(11)
    z = rng.normal(size=(B, V)).astype(np.float32) * 2.0
    z[1, :] = -3.0
    z[1, rng.choice(V, 400, replace=False)] = rng.normal(size=400).astype(np.float32) * 2.0 + 1.0
    z[3, :] = 0.5
    zt = torch.tensor(z, device="cuda").to(torch.bfloat16)
    zh = raw(zt, torch)
    ctx = adasd.Context(B, V, 1, list_capacity=8)
    ctx.set_warpers(*warpers)
    ws = (float(np.float32(warpers[0])), warpers[1], float(np.float32(warpers[2])))
    u = torch.tensor([0.05, 0.35, 0.55, 0.75, 0.95], device="cuda")
    H = torch.zeros(B, device="cuda")
    lse = torch.zeros(B, device="cuda")
    tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    for _ in range(2):
        ctx.draft_entropy(zt, H, u=u, token_out=tok, lse_out=lse)
    torch.cuda.synchronize()
    for b in range(B):
        zw, _, band = oracle.warp(zh[b], *ws, band=5e-7)
        assert band < 1e-6, "pick another seed: a top-p decision of this row is too close to call"
        o = oracle.draft_step(zw, float(u[b]), 0.0)
        assert abs(float(H[b]) - o["H"]) < TOL and abs(float(lse[b]) - o["lse"]) < TOL, (b, float(H[b]), o)
        assert int(tok[b]) == o["token"] or o["margin"] < 2e-6, (b, int(tok[b]), o)
    assert ctx.status() == 0


@pytest.mark.parametrize("V,dtype", [(40000, synth.BF16), (4099, synth.BF16), (3000, synth.FP32)])
def test_unusable_and_sparse_rows_under_a_cut(torch, adasd, V, dtype):
    """Rows the cut has to leave alone or nearly so: a row with a NaN (not cut; reported as
    unusable by the row pass), a row with fewer finite logits than top_k (everything finite
    stays), a row whose finite logits are all equal, next to an ordinary row."""
    B = 4
    rng = np.random.default_rng(5)
    z = (rng.normal(size=(B, V)) * 2.0).astype(np.float32)
    z[0, 17] = np.nan
    z[1, :] = -np.inf
    z[1, rng.choice(V, 10, replace=False)] = rng.normal(size=10).astype(np.float32)
    z[2, :] = -np.inf
    z[2, rng.choice(V, 300, replace=False)] = 1.25
    tdt = torch.bfloat16 if dtype == synth.BF16 else torch.float32
    zt = torch.tensor(z, device="cuda").to(tdt)
    zh = raw(zt, torch)
    ctx = adasd.Context(B, V, 1, dtype=dtype, list_capacity=8)
    ws = (float(np.float32(0.9)), 50, float(np.float32(0.9)))
    ctx.set_warpers(*ws)
    u = torch.tensor([0.2, 0.4, 0.6, 0.8], device="cuda")
    H = torch.zeros(B, device="cuda")
    lse = torch.zeros(B, device="cuda")
    tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.draft_entropy(zt, H, u=u, token_out=tok, lse_out=lse)
    torch.cuda.synchronize()
    assert torch.isnan(H[0]) and int(tok[0]) == -1
    for b in range(1, B):
        zw, _, band = oracle.warp(zh[b], *ws, band=5e-7)
        assert band < 1e-6
        o = oracle.draft_step(zw, float(u[b]), 0.0)
        assert abs(float(H[b]) - o["H"]) < TOL and abs(float(lse[b]) - o["lse"]) < TOL, (b, float(H[b]), o)
        assert int(tok[b]) == o["token"] or o["margin"] < 2e-6, (b, int(tok[b]), o)
    kept1 = np.isfinite(oracle.warp(zh[1], *ws)[0]).sum()
    assert kept1 <= 10 and np.isfinite(oracle.warp(zh[2], *ws)[0]).sum() == 300      # ties stay together
    assert ctx.status() == adasd.STATUS_NAN
