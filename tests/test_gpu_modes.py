"""GPU parity of greedy decoding (Sec. 2.1.3) and of the ablation variants Gen-Only and
Verify-Only (Sec. 5) against the float64 oracle, through the library's own calls."""
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


@pytest.mark.parametrize("V,dtype,B,K", [(128256, synth.BF16, 6, 5), (8200, synth.BF16, 9, 7),
                                         (1003, synth.FP32, 5, 4), (4099, synth.BF16, 4, 3)])
def test_greedy_drafting_and_verification(torch, adasd, V, dtype, B, K):
    """Draft tokens are argmax q (adasd_draft_entropy without a uniform), verification accepts
    the longest prefix that equals argmax p, the next token is the target's choice there."""
    wl = synth.WORKLOADS["C3"].scaled(name="greedy", B=B, K=K, V=V, dtype=dtype, rounds=3,
                                      recipe="fixed_tau", tau0=0.6)
    gs = synth.GpuSynth(wl)
    tdt = torch.bfloat16 if dtype == synth.BF16 else torch.float32
    ctx = adasd.Context(B, V, K, dtype=dtype, list_capacity=64)
    zd = torch.empty((B, K, V), dtype=tdt, device="cuda")
    zt = torch.empty((B, K + 1, V), dtype=tdt, device="cuda")
    i32 = dict(dtype=torch.int32, device="cuda")
    seen = set()
    for r in range(wl.rounds):
        gs.draft_rows(r, zd)
        gs.target_rows(r, zt)
        if r == 1:                                   # a tie between two tokens of one target row
            zt[0, 0, 7] = zt[0, 0].max() + 1
            zt[0, 0, 3] = zt[0, 0, 7]
        H = torch.zeros((K, B), device="cuda")
        tok = torch.full((K, B), -9, **i32)
        for k in range(K):
            ctx.draft_entropy(zd[:, k, :], H[k], token_out=tok[k], row_stride=K * V)     # no uniform: argmax q
        x = tok.T.contiguous()
        dlen = torch.tensor([(b + r) % (K + 1) for b in range(B)], **i32)
        al, nt = torch.full((B,), -9, **i32), torch.full((B,), -9, **i32)
        am = torch.full((B, K + 1), -7, **i32)
        ctx.greedy_verify(zt, x, al, nt, draft_len=dlen, argmax_out=am)
        torch.cuda.synchronize()
        zd_h, zt_h, x_h = raw(zd, torch), raw(zt, torch), x.cpu().numpy()
        for b in range(B):
            for k in range(K):
                assert int(x_h[b, k]) == oracle.argmax(zd_h[b, k]), (r, b, k)
            K_t = int(dlen[b])
            o = oracle.greedy_round(zt_h[b], x_h[b, :K_t])
            assert (int(al[b]), int(nt[b])) == (o["accept_len"], o["next_token"]), (r, b, o)
            w = o["accept_len"]
            assert list(am[b, : w + 1].cpu().numpy()) == list(o["argmax"][: w + 1])
            assert (am[b, K_t + 1:] == -7).all()                 # untouched beyond the window
            seen.add(w)
        if r == 1:
            assert int(am[0, 0]) == 3                            # the tie went to the lower index
    assert len(seen) >= 2
    assert ctx.status() == 0


def test_greedy_unusable_target_row_matches_nothing(torch, adasd):
    V, K, B = 1000, 3, 2
    rng = np.random.default_rng(2)
    zt = torch.tensor(rng.normal(size=(B, K + 1, V)).astype(np.float32), device="cuda")
    zt[0, 1, 5] = float("nan")
    zt[1, 0, :] = float("-inf")
    ctx = adasd.Context(B, V, K, dtype=adasd.ADASD_FP32, list_capacity=8)
    am0 = zt.nan_to_num(nan=-1e30).argmax(dim=2).to(torch.int32)
    x = am0[:, :K].contiguous()
    al = torch.zeros(B, dtype=torch.int32, device="cuda")
    nt = torch.zeros(B, dtype=torch.int32, device="cuda")
    ctx.greedy_verify(zt, x, al, nt)
    torch.cuda.synchronize()
    assert (int(al[0]), int(nt[0])) == (1, -1) and (int(al[1]), int(nt[1])) == (0, -1)
    assert ctx.status() == adasd.STATUS_NAN


def test_verify_only_is_adasd_verification_on_a_window_of_five(torch):
    """Sec. 5: Verify-Only fixes the number of candidates at five, as Vanilla does, and keeps
    the JS-distance acceptance rule; the stop flags of the draft steps are ignored."""
    from tests.lockstep import Lockstep
    wl = synth.WORKLOADS["C3"].scaled(name="verify_only", B=6, K=5, V=8200, rounds=60, vanilla=False)
    rep = Lockstep(wl, min_kde_samples=3, check_lists_every=20).run()
    assert rep.window_hist == {5: 60 * 6} and rep.n_rejections > 10 and len(rep.accept_hist) >= 3


@pytest.mark.parametrize("V", [8200, 40000])
def test_gen_only_round_by_round(torch, adasd, V):
    """Sec. 5: Gen-Only = the entropy stop check of Sec. 4.3 with vanilla verification; the
    rejected candidate's entropy feeds T_G.  Windows, accept lengths, list sizes exact; T_G
    and entropies within 1e-4; a stop check within 1e-4 of its threshold may go either way,
    after which the device state is set to the oracle's."""
    B, K, R = 6, 8, 50
    wl = synth.WORKLOADS["C5"].scaled(name="gen_only", B=B, K=K, V=V, rounds=R)
    gs = synth.GpuSynth(wl)
    ctx = adasd.Context(B, V, K, list_capacity=R + 8)
    states = [oracle.SequenceState(capacity=R + 8) for _ in range(B)]
    zd = torch.empty((B, K, V), dtype=torch.bfloat16, device="cuda")
    zt = torch.empty((B, K + 1, V), dtype=torch.bfloat16, device="cuda")
    f32, i32 = dict(dtype=torch.float32, device="cuda"), dict(dtype=torch.int32, device="cuda")
    windows, near_flips, rejections = set(), 0, 0
    for r in range(R):
        U = synth.round_uniforms_cpu(wl, r)
        gs.draft_rows(r, zd)
        gs.target_rows(r, zt)
        hd, ht = synth.host_round(wl, r)
        ud = torch.tensor(U["draft"].T.copy(), device="cuda")
        Hk, tokk = torch.zeros((K, B), **f32), torch.zeros((K, B), **i32)
        active = torch.ones(B, dtype=torch.uint8, device="cuda")
        dlen = torch.zeros(B, **i32)
        for k in range(K):
            ctx.draft_entropy(zd[:, k, :], Hk[k], u=ud[k], token_out=tokk[k], active=active,
                              draft_len=dlen, row_stride=K * V)
        x = tokk.T.contiguous()
        al, nt = torch.zeros(B, **i32), torch.zeros(B, **i32)
        ctx.vanilla_verify(zd, zt, x, torch.tensor(U["vanilla_accept"], device="cuda"),
                           torch.tensor(U["resample"], device="cuda"), al, nt, draft_len=dlen)
        H_bk = Hk.T.contiguous()
        ctx.gen_only_update(H_bk, al, draft_len=dlen)
        torch.cuda.synchronize()
        T, nE, nA, nR = (t.cpu().numpy() for t in ctx.get_thresholds())
        for b in range(B):
            st = states[b]
            steps, near = [], False
            for k in range(K):
                d = oracle.draft_step(hd[b, k], float(U["draft"][b, k]), st.T_G.value)
                steps.append(d)
                near |= abs(d["H"] - st.T_G.value) < TOL
                if d["stop"]:
                    break
            K_t = len(steps)
            xs = [d["token"] for d in steps]
            ov = oracle.vanilla_round(hd[b][:K_t], ht[b], xs, U["vanilla_accept"][b, :K_t], float(U["resample"][b]))
            oracle.gen_only_update(st, [d["H"] for d in steps], K_t, ov["accept_len"])
            ok = int(dlen[b]) == K_t and int(al[b]) == ov["accept_len"] and int(nE[b]) == st.nE.value
            if not ok:
                n_seen = min(ov["accept_len"] + 1, K_t)
                tie = (any(d["margin"] < 2e-6 for d in steps) or ov["margin"] < 2e-6 or
                       any(abs(float(U["vanilla_accept"][b, i]) - ov["alpha"][i]) < TOL for i in range(n_seen)))
                assert near or tie, (r, b, int(dlen[b]), K_t, int(al[b]), ov)
                near_flips += 1
                LE, LA, LR = st.lists()
                ctx.state_import(b, st.T_G.value, LE, LA, LR)
                continue
            windows.add(K_t)
            rejections += ov["accept_len"] < K_t
            for k in range(K_t):
                assert abs(float(Hk[k, b]) - steps[k]["H"]) < TOL
            assert abs(float(T[b]) - st.T_G.value) < TOL and (int(nA[b]), int(nR[b])) == (0, 0)
    assert len(windows) >= 3 and rejections > R and near_flips <= 3
    assert ctx.status() == 0


def test_expired_wait_is_reported_and_the_context_stays_usable(torch, adasd):
    """The give-up path of the bounded device waits, made to run without a fault: one warp of
    one row never asks for its first chunk and waits for it only briefly.  The call returns,
    the status word says TIMEOUT, that row's outputs are NaN / -1, the other rows are right, and
    the next ordinary call on the same context is right for every row."""
    B, V = 5, 40000
    wl = synth.WORKLOADS["C3"].scaled(name="expire", B=B, K=1, V=V, rounds=1)
    gs = synth.GpuSynth(wl)
    ctx = adasd.Context(B, V, 1, list_capacity=8)
    zd = torch.empty((B, 1, V), dtype=torch.bfloat16, device="cuda")
    gs.draft_rows(0, zd)
    z = zd[:, 0, :]
    u = torch.tensor([0.1, 0.3, 0.5, 0.7, 0.9], device="cuda")
    want = [oracle.draft_step(raw(z[b], torch), float(u[b]), 0.0) for b in range(B)]
    row = 2
    H = torch.zeros(B, device="cuda")
    tok = torch.full((B,), -5, dtype=torch.int32, device="cuda")
    rc = adasd.adasd_selftest_expired_wait(ctx.handle, z.data_ptr(), z.stride(0), row, u.data_ptr(), H.data_ptr(),
                                           tok.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    torch.cuda.synchronize()
    st = ctx.status()
    assert st & adasd.STATUS_TIMEOUT and not (st & adasd.STATUS_CAPACITY)
    assert torch.isnan(H[row]) and int(tok[row]) == -1
    for b in range(B):
        if b != row:
            assert abs(float(H[b]) - want[b]["H"]) < TOL and int(tok[b]) == want[b]["token"], b
    # an ordinary call afterwards: every row right, status clean
    H2 = torch.zeros(B, device="cuda")
    tok2 = torch.full((B,), -5, dtype=torch.int32, device="cuda")
    ctx.draft_entropy(z, H2, u=u, token_out=tok2)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    for b in range(B):
        assert abs(float(H2[b]) - want[b]["H"]) < TOL and int(tok2[b]) == want[b]["token"], b
    # refused where the streaming kernel does not apply (fp32 rows)
    ctx32 = adasd.Context(2, 1000, 1, dtype=adasd.ADASD_FP32, list_capacity=8)
    z32 = torch.zeros((2, 1000), device="cuda")
    assert adasd.adasd_selftest_expired_wait(ctx32.handle, z32.data_ptr(), 1000, 0, None, H.data_ptr(), None, None) == -3
