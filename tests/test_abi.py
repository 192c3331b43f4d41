"""CPU checks of the boundary: the C-ABI library builds, loads and exports every symbol that
include/hifa4.h declares; argument validation answers without a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_04302_b200 import build, binding
    build.build()
    return binding.lib()


def _declared():
    src = open(os.path.join(ROOT, "include", "hifa4.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(hifa4_[a-z_0-9]+)\s*\(", src)))


def test_exports_every_declared_symbol(lib):
    names = _declared()
    assert "hifa4_attention_fwd" in names and "hifa4_quantize_qkv" in names and "hifa4_smooth_calibrate" in names
    for n in names:
        assert hasattr(lib, n), n
    from paper_2607_04302_b200 import binding
    assert set(binding.EXPORTS) <= set(names)


def test_size_queries_and_validation_without_gpu(lib):
    from paper_2607_04302_b200 import binding as hb
    # 4.5 bits per value: codes + metadata
    nb = [hb.quant_bytes(1, 32, 8, 4096, 128, hb.BF16, hb.Q, p) for p in (hb.CODES, hb.META, hb.MMA)]
    n = 32 * 4096 * 128
    assert (nb[0] + nb[1]) * 8 / n == 4.5 and nb[2] == 2 * n
    assert hb.quant_bytes(1, 32, 8, 4096, 128, hb.BF16, hb.K, hb.CODES) == 8 * 4096 * 128 // 2
    assert hb.quant_bytes(1, 32, 8, 4000, 128, hb.BF16, hb.Q, hb.CODES) == 0       # N % 64
    assert hb.quant_bytes(1, 32, 8, 4096, 96, hb.BF16, hb.Q, hb.CODES) == 0        # d
    assert hb.status_string(0) == "ok" and "timed out" in hb.status_string(6)
    sh = hb._shape(1, 4, 3, 128, 128, hb.BF16)                                      # Hq % Hkv != 0
    st = hb._QKV(*[1] * 9)
    one = C.c_void_p(256)
    rc = lib.hifa4_quantize_qkv(C.byref(sh), one, one, one, None, None, C.byref(st), None, None)
    assert rc == 1
    sh = hb._shape(1, 4, 2, 128, 128, hb.BF16)
    prm = hb._params(True, 96, hb.F32)                                              # Bc
    assert lib.hifa4_attention_fwd(C.byref(sh), C.byref(st), C.byref(prm), one, None, None, None, None) == 2
    prm = hb._params(True, 128, hb.F32, qmean=1)                                    # Q-Mean vectors missing
    assert lib.hifa4_attention_fwd(C.byref(sh), C.byref(st), C.byref(prm), one, None, None, None, None) == 1
    prm = hb._params(True, 128, hb.F32, normalizer=2)                               # no such normaliser mode
    assert lib.hifa4_attention_fwd(C.byref(sh), C.byref(st), C.byref(prm), one, None, None, None, None) == 1
    prm = hb._params(True, 128, hb.F32, p_dtype=hb.F32)                             # FP32 P: built for 64-key tiles only
    assert lib.hifa4_attention_fwd(C.byref(sh), C.byref(st), C.byref(prm), one, None, None, None, None) == 2
    prm = hb._params(True, 128, hb.F32)                                             # histogram request without bins
    assert lib.hifa4_attention_fwd_stats(C.byref(sh), C.byref(st), C.byref(prm), one, None, None, None, None) == 1
    # no sm_100 device here: a well-formed call is refused with ARCH or CUDA, never run on the CPU
    import torch
    if not torch.cuda.is_available():
        prm = hb._params(True, 128, hb.F32)
        rc = lib.hifa4_attention_fwd(C.byref(sh), C.byref(st), C.byref(prm), one, None, None, None, None)
        assert rc in (4, 5)
    assert hb.attention_raw_workspace_bytes(1, 4, 2, 128, 128, hb.BF16, True, 128) > 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2607_04302_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "lib_path", lambda: str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        binding.lib()
