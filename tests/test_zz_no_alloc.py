"""GPU test of hifa4_smooth_calibrate_static, the calibration entry point for callers that are
not allowed to allocate device memory (its scratch is a fixed array inside the library).

The file name makes pytest collect it last, so that a run that stops at the first failure has
already run every other test.  It passes both alone in a fresh process and after the others."""
import pytest
import torch

from paper_2607_04302_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_static_scratch_entry_point_matches_workspace_entry_point():
    from paper_2607_04302_b200 import binding as hb
    hb.lib()
    cfg_a = synth.config("C2", Hq=8, Hkv=2, cal_samples=6, cal_tokens=192)
    cfg_b = synth.config("C4", Hq=4, Hkv=2, cal_samples=3, cal_tokens=128)        # d = 256, mild branch
    # preallocated outputs: the call under test gets every buffer from its caller
    for call, cfg in enumerate((cfg_a, cfg_b, cfg_a)):
        qc, kc = synth.make_calibration(cfg)
        if call == 2:                       # same shape as the first call, different data: the array
            kc = (kc.float() * 0.25).to(kc.dtype)   # still holds larger maxima that must be cleared
        qc, kc = qc.to(DEV), kc.to(DEV)
        s = torch.full((cfg.Hkv, cfg.d), -1.0, dtype=torch.float32, device=DEV)
        inv_s = torch.full_like(s, -1.0)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(DEV)
        free_before = torch.cuda.mem_get_info(DEV)[0]
        hb.smooth_calibrate_static(qc, kc, cfg.smooth_mode, s=s, inv_s=inv_s)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(DEV) == before          # torch saw no allocation
        # and neither did the driver: by the third call every kernel of the entry point is loaded, so the
        # device's free memory cannot move unless the library itself allocated (cudaMalloc, a stream-ordered
        # allocation) -- which torch's own counter above would not see
        if call == 2:
            assert torch.cuda.mem_get_info(DEV)[0] == free_before
        s_ref, inv_ref = hb.smooth_calibrate(qc, kc, cfg.smooth_mode)
        torch.cuda.synchronize()
        # same kernels on the same data: identical bits, which is inside the 1e-6 relative tolerance
        # the calibration tests use
        assert torch.equal(s, s_ref) and torch.equal(inv_s, inv_ref), f"call {call}"
        assert torch.allclose(s, s_ref, rtol=1e-6, atol=0) and bool((s > 0).all())


def test_static_scratch_rejects_oversized_requests():
    from paper_2607_04302_b200 import binding as hb
    # 2 * S * Hkv * d floats must fit the fixed array: 2 * 64 * 64 * 256 = 2 Mi floats does not
    S, Hq, Hkv, T, d = 64, 64, 64, 8, 256
    assert 2 * S * Hkv * d > hb.STATIC_CALIB_MAX_FLOATS
    qc = torch.zeros((S, Hq, T, d), dtype=torch.bfloat16, device=DEV)
    kc = torch.zeros((S, Hkv, T, d), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(hb.Hifa4Error) as e:
        hb.smooth_calibrate_static(qc, kc, hb.MODE_STRONG)
    assert e.value.status == 3 and "workspace" in str(e.value)
    hb.smooth_calibrate(qc, kc, hb.MODE_STRONG)                    # the workspace entry point still takes it
    torch.cuda.synchronize()
