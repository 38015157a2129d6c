"""CPU-side checks of the C-ABI library: it builds, loads and exports every symbol the
header declares, and host-detectable errors come back as negative codes."""
import ctypes
import os
import re

import paper_2512_11280_b200 as adasd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(adasd_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_library_builds_and_exports_every_declared_symbol():
    lib = adasd.lib()
    names = declared_functions()
    assert "adasd_verify" in names and "adasd_draft_entropy" in names
    assert "adasd_update_thresholds" in names and "adasd_vanilla_verify" in names
    for n in names:
        assert hasattr(lib, n), n
    assert os.path.exists(adasd.library_path())


def test_strerror_and_null_arguments():
    assert adasd.adasd_strerror(0) == "ok"
    assert "NULL" in adasd.adasd_strerror(-1)
    lib = adasd.lib()
    assert lib.adasd_create(None, None) == -1
    assert lib.adasd_destroy(None) == -1
    assert lib.adasd_status(None, None) == -1
    assert lib.adasd_update_thresholds(None, None, None) == -1
    assert adasd.adasd_set_warpers(None, 1.0, 0, 1.0) == -1


def test_error_codes_of_the_header_have_messages_and_match_the_binding():
    text = open(os.path.join(ROOT, "include", "adasd.h")).read()
    codes = dict((n, int(v)) for n, v in re.findall(r"#define (ADASD_ERR_[A-Z]+) \((-\d+)\)", text))
    assert codes == {"ADASD_ERR_NULL": adasd.ERR_NULL, "ADASD_ERR_ALIGN": adasd.ERR_ALIGN,
                     "ADASD_ERR_SHAPE": adasd.ERR_SHAPE, "ADASD_ERR_DTYPE": adasd.ERR_DTYPE,
                     "ADASD_ERR_CAPACITY": adasd.ERR_CAPACITY, "ADASD_ERR_CUDA": adasd.ERR_CUDA,
                     "ADASD_ERR_DEVICE": adasd.ERR_DEVICE}
    msgs = {c: adasd.adasd_strerror(c) for c in codes.values()}
    assert all(m != "unknown error" for m in msgs.values()) and len(set(msgs.values())) == len(msgs)
    assert "device" in msgs[adasd.ERR_DEVICE] and "aligned" in msgs[adasd.ERR_ALIGN]
    assert adasd.adasd_strerror(-6) == "unknown error" and adasd.adasd_strerror(-8) == "unknown error"


def test_misaligned_pointers_are_refused_before_anything_runs():
    """float / int32 arrays must sit on 4-byte boundaries, bf16 logits on 2-byte ones: the
    context-free entry point checks that before it asks CUDA anything, so it shows here."""
    ok = 0x10000                         # never dereferenced: every case below is refused on the host
    def call(zd=ok, zt=ok, x=ok, dlen=None, ua=ok, ur=ok, al=ok, nt=ok, alpha=None, status=None,
             dtype=adasd.ADASD_BF16):
        return adasd.adasd_vanilla_verify_static(2, 1000, 4, dtype, zd, zt, 4000, 1000, 5000, 1000, x, dlen,
                                                 ua, ur, al, nt, alpha, status, None)
    assert call(zd=ok + 1) == adasd.ERR_ALIGN and call(zt=ok + 1) == adasd.ERR_ALIGN
    assert call(zd=ok + 2, dtype=adasd.ADASD_FP32) == adasd.ERR_ALIGN      # fp32 logits: 4 bytes
    for name in ("x", "dlen", "ua", "ur", "al", "nt", "alpha", "status"):
        assert call(**{name: ok + 2}) == adasd.ERR_ALIGN, name
    assert call(x=None) == adasd.ERR_NULL


def test_create_validates_before_touching_cuda():
    for field, value, want in (("B", 0, -3), ("V", 0, -3), ("Kmax", 0, -3), ("Kmax", 33, -3),
                               ("list_capacity", 0, -3), ("dtype", 7, -4), ("kde_bandwidth", 2, -4),
                               ("reject_rule", -1, -4), ("cluster_size", 9, -3)):
        cfg = adasd.AdasdConfig(4, 1000, 8, adasd.ADASD_BF16, 64, 0, 0, 2, 0, 0)
        setattr(cfg, field, value)
        rc, h = adasd.adasd_create(cfg)
        assert rc == want, (field, rc)
        assert not h.value


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        return
    cfg = adasd.AdasdConfig(4, 1000, 8, adasd.ADASD_BF16, 64, 0, 0, 2, 0, 0)
    rc, h = adasd.adasd_create(cfg)
    assert rc == -7 and not h.value            # ADASD_ERR_CUDA: no device, no result
    try:
        adasd.Context(4, 1000, 8)
    except RuntimeError:
        pass
    else:
        raise AssertionError("Context() must fail without a CUDA device")
