"""GPU parity: Smooth-QK calibration and the fused smooth + HIF4 quantize kernels against the CPU
oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2607_04302_b200 import synth

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def hb():
    from paper_2607_04302_b200 import binding
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def par():
    from tests import parity
    return parity


CASES = {
    "c1": synth.config("C1"),
    "c2-small": synth.config("C2", N=256, Hq=4, Hkv=2, cal_samples=4, cal_tokens=128),
    "d256-mild": synth.config("C4", N=128, Hq=4, Hkv=2, cal_samples=3, cal_tokens=64),
    "d64-bypass": synth.config("C3", N=192, Hq=2, Hkv=1, d=64),
    "batch": synth.config("C5", B=2, N=128, Hq=4, Hkv=2, cal_samples=2, cal_tokens=64),
}


@pytest.mark.parametrize("name", list(CASES))
def test_calibrate_matches_oracle(hb, par, oracle, name):
    cfg = CASES[name]
    if cfg.smooth_mode == 0:
        pytest.skip("bypass")
    qc, kc = synth.make_calibration(cfg)
    s, inv_s = hb.smooth_calibrate(qc.to(DEV), kc.to(DEV), cfg.smooth_mode)
    ref = oracle.smooth_calibrate(par.np32(qc), par.np32(kc), cfg.smooth_mode)
    assert np.allclose(par.np32(s), ref["s"], rtol=1e-6, atol=0)
    # the reciprocal is the correctly rounded fp32 reciprocal of the s the library produced
    assert np.array_equal(par.np32(inv_s), (np.float32(1) / par.np32(s)).astype(np.float32))
    b, _ = hb.smooth_calibrate(qc.to(DEV), kc.to(DEV), hb.MODE_BYPASS)
    assert torch.all(b == 1)
    c, _ = hb.smooth_calibrate(qc.to(DEV), kc.to(DEV), hb.MODE_CUSTOM, alpha=0.5)
    st, _ = hb.smooth_calibrate(qc.to(DEV), kc.to(DEV), hb.MODE_STRONG)
    assert torch.equal(c, st)
    with pytest.raises(hb.Hifa4Error):
        hb.smooth_calibrate(qc.to(DEV), kc.to(DEV), hb.MODE_AUTO)


@pytest.mark.parametrize("name", list(CASES))
def test_quantize_bit_exact(hb, par, name):
    cfg = CASES[name]
    q, k, v = synth.make_qkv(cfg)
    s, inv_s = par.calibrate(cfg, DEV)
    qkv = hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s)
    torch.cuda.synchronize()
    par.check_quantized(cfg, q, k, v, s, inv_s, qkv)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_quantize_adversarial_groups(hb, par, oracle, dtype):
    """Zero groups, single outliers, exact rounding ties, maxima sitting exactly on the scale and
    shift thresholds, tiny and huge magnitudes."""
    rng = np.random.default_rng(5)
    N, d = 128, 128
    x = rng.standard_normal((1, 1, N, d))
    x[0, 0, 0] = 0                                                # all-zero groups
    x[0, 0, 1] = 0; x[0, 0, 1, 5] = 100                           # lone outlier
    x[0, 0, 2] = 1.0                                              # flat
    x[0, 0, 3] = rng.integers(-28, 29, d) * 0.125                 # ties on a coarse grid
    for r in range(4, 40):                                        # maxima on thresholds of random scales
        S = oracle.e6m2_value(int(rng.integers(170, 215)))
        x[0, 0, r] = rng.choice([7 * S, 1.75 * S, 3.5 * S, 0.5 * S / 4, 1.5 * S / 4, 2.5 * S / 2, 6.5 * S / 4,
                                 6.5 * S, 0.0, -3.5 * S], d)
    x[0, 0, 40] *= 2.0 ** -20
    x[0, 0, 41] *= 2.0 ** 12 if dtype == torch.float16 else 2.0 ** 30
    x[0, 0, 42] *= 2.0 ** -14 if dtype == torch.float16 else 2.0 ** -100
    xt = torch.tensor(x, dtype=torch.float32).to(dtype)
    cfg = synth.config("C3", B=1, Hq=1, Hkv=1, N=N, d=d, dtype="fp16" if dtype == torch.float16 else "bf16")
    s = torch.tensor(np.exp(rng.standard_normal((1, d)) * 0.5), dtype=torch.float32, device=DEV)
    inv_s = (1.0 / s).to(torch.float32)
    qkv = hb.quantize_qkv(xt.to(DEV), xt.to(DEV), xt.to(DEV), s, inv_s)
    torch.cuda.synchronize()
    par.check_quantized(cfg, xt, xt, xt, s, inv_s, qkv)
    # bypass path too
    qkv = hb.quantize_qkv(xt.to(DEV), xt.to(DEV), xt.to(DEV))
    torch.cuda.synchronize()
    par.check_quantized(cfg, xt, xt, xt, None, None, qkv)


def test_explicit_head_map(hb, par):
    cfg = synth.config("C2", N=128, Hq=4, Hkv=2, cal_samples=2, cal_tokens=64)
    q, k, v = synth.make_qkv(cfg)
    s, inv_s = par.calibrate(cfg, DEV)
    a = hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s)
    b = hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s, q_to_kv=[0, 0, 1, 1])
    assert torch.equal(a.q_codes, b.q_codes) and torch.equal(a.q_meta, b.q_meta)
    c = hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s, q_to_kv=[1, 1, 0, 0])
    assert not torch.equal(a.q_codes, c.q_codes)
    with pytest.raises(hb.Hifa4Error):
        hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s, q_to_kv=[0, 0, 1, 2])
