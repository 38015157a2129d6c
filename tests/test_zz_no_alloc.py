"""adasd_vanilla_verify_static: the entry point for callers that cannot allocate.

Some users of this library run where cudaMalloc is not theirs to call: a serving engine
that gave the whole GPU to its own pool, a plugin that must leave the allocator alone.
They cannot create a context, so the library offers one context-free call whose scratch
is a fixed array inside the library image.  This file checks, through the C ABI, that
the call returns what adasd_vanilla_verify returns on the same inputs, twice in a row
(the second call meets the first call's leftovers in the shared array), that both agree
with the float64 oracle's vanilla round on every sequence, and that sizes beyond the
stated maximum are refused.

Collected last on purpose: a run that stops at the first failure has then already run
every other test.  The test builds its own inputs and passes on its own in a fresh
process as well as after the rest of the suite.
"""
import numpy as np
import pytest

import oracle
import paper_2512_11280_b200 as adasd
import synth

pytestmark = pytest.mark.gpu

TOL = 1e-4   # absolute tolerance of the parity tests for floating-point outputs


def _inputs(wl, round_, dev):
    import torch
    B, K, V = wl.B, wl.K, wl.V
    tdt = torch.bfloat16 if wl.dtype == synth.BF16 else torch.float32
    gs = synth.GpuSynth(wl, str(dev))
    zd = torch.empty((B, K, V), dtype=tdt, device=dev)
    zt = torch.empty((B, K + 1, V), dtype=tdt, device=dev)
    gs.draft_rows(round_, zd)
    gs.target_rows(round_, zt)
    U = gs.new_round_uniforms()
    gs.round_uniforms(round_, U)
    # draft tokens: any valid ids will do for the accept test; spread them over the vocabulary
    x = (torch.arange(B * K, device=dev, dtype=torch.int64) * 7919 % V).to(torch.int32).view(B, K)
    dlen = (torch.arange(B, device=dev, dtype=torch.int32) % (K + 1)).contiguous()
    return zd, zt, x, dlen, U


def _raw(t):
    """Device logits -> the oracle's raw input (bf16 bits or float32)."""
    import torch
    return t.view(torch.int16).cpu().numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.cpu().numpy()


# fp32 rows; bf16 rows that are not 16-byte aligned (scalar loads); bf16 rows of a multiple of 8
# logits (16-byte vector loads)
@pytest.mark.parametrize("dtype,V", [(synth.FP32, 32000), (synth.BF16, 5000), (synth.BF16, 4099),
                                     (synth.BF16, 4096)])
def test_static_entry_matches_context_entry_twice(dtype, V):
    import torch
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    wl = synth.WORKLOADS["C3"].scaled(name="noalloc", B=6, K=4, V=V, dtype=dtype, rounds=2)
    B, K = wl.B, wl.K
    ctx = adasd.Context(B, V, K, dtype=dtype, list_capacity=64, device=0)
    i32 = dict(dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream(dev).cuda_stream
    for round_ in range(2):                       # two calls in a row share the static array
        zd, zt, x, dlen, U = _inputs(wl, round_, dev)
        ref_al, ref_nt = torch.full((B,), -5, **i32), torch.full((B,), -5, **i32)
        ref_alpha = torch.full((B, K), float("nan"), dtype=torch.float32, device=dev)
        ctx.vanilla_verify(zd, zt, x, U["vanilla_accept"], U["resample"], ref_al, ref_nt,
                           draft_len=dlen, alpha_out=ref_alpha)
        al, nt = torch.full((B,), -7, **i32), torch.full((B,), -7, **i32)
        alpha = torch.full((B, K), float("nan"), dtype=torch.float32, device=dev)
        status = torch.full((1,), 99, **i32)
        rc = adasd.adasd_vanilla_verify_static(
            B, V, K, dtype, zd.data_ptr(), zt.data_ptr(), zd.stride(0), zd.stride(1), zt.stride(0),
            zt.stride(1), x.data_ptr(), dlen.data_ptr(), U["vanilla_accept"].data_ptr(),
            U["resample"].data_ptr(), al.data_ptr(), nt.data_ptr(), alpha.data_ptr(),
            status.data_ptr(), stream)
        assert rc == 0, adasd.adasd_strerror(rc)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        assert torch.equal(al, ref_al), (round_, al.tolist(), ref_al.tolist())
        assert torch.equal(nt, ref_nt), (round_, nt.tolist(), ref_nt.tolist())
        assert 0 <= int(nt.min()) and int(nt.max()) < V
        live = torch.arange(K, device=dev)[None, :] < dlen[:, None]
        err = (alpha - ref_alpha).abs()[live]
        assert err.numel() == int(dlen.sum()) and not torch.isnan(err).any()
        assert float(err.max()) <= TOL if err.numel() else True
        # the oracle's vanilla round of every sequence (Sec. 2.1.3), not just the other entry point
        x_h, dl_h, al_h, nt_h, a_h = (t.cpu().numpy() for t in (x, dlen, al, nt, alpha))
        ua_h, ur_h = U["vanilla_accept"].cpu().numpy(), U["resample"].cpu().numpy()
        for b in range(B):
            K_t = int(dl_h[b])
            o = oracle.vanilla_round(_raw(zd[b, :K_t]), _raw(zt[b]), x_h[b, :K_t], ua_h[b, :K_t], float(ur_h[b]))
            n_seen = min(o["accept_len"] + 1, K_t)
            assert np.allclose(a_h[b, :n_seen], o["alpha"][:n_seen], atol=TOL), (b, a_h[b], o["alpha"])
            near = any(abs(float(ua_h[b, i]) - o["alpha"][i]) < TOL for i in range(n_seen))
            assert int(al_h[b]) == o["accept_len"] or near, (b, al_h[b], o)
            if int(al_h[b]) == o["accept_len"] and o["margin"] > 2e-6:
                assert int(nt_h[b]) == o["next_token"], (b, nt_h[b], o)
    assert ctx.status() == 0
    ctx.close()


def test_static_entry_refuses_sizes_beyond_its_array():
    import torch
    dev = torch.device("cuda", 0)
    t = torch.zeros(64, dtype=torch.int32, device=dev)
    p = t.data_ptr()
    too_many_seq = adasd.adasd_vanilla_verify_static(1025, 1000, 4, adasd.ADASD_BF16, p, p, 4000, 1000,
                                                     5000, 1000, p, None, p, p, p, p, None, None, None)
    too_many_pos = adasd.adasd_vanilla_verify_static(1000, 1000, 31, adasd.ADASD_BF16, p, p, 31000, 1000,
                                                     32000, 1000, p, None, p, p, p, p, None, None, None)
    assert too_many_seq == -5 and too_many_pos == -5          # ADASD_ERR_CAPACITY, nothing launched
    assert "maximum" in adasd.adasd_strerror(-5)
    torch.cuda.synchronize()
