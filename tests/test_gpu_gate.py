"""GPU parity of the applicability gate ("Adaptive Applicability Gate"): rho_K, T_K/Q, the branch and
the resulting Smooth-QK factors from hifa4_smooth_calibrate_auto against the CPU oracle's mode 3,
on calibration sets built to land in each of the three branches."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def hb():
    from paper_2607_04302_b200 import binding
    binding.lib()
    return binding


def _cal(S, Hq, Hkv, T, d, dtype, k_gain, q_gain, n_out, seed):
    """N(0,1) calibration activations; n_out K channels per KV head x k_gain, all of Q x q_gain."""
    gen = torch.Generator().manual_seed(seed)
    q = (torch.randn((S, Hq, T, d), generator=gen) * q_gain).to(dtype)
    k = torch.randn((S, Hkv, T, d), generator=gen)
    for g in range(Hkv):
        ch = torch.randperm(d, generator=gen)[:n_out]
        k[:, g, :, ch] *= k_gain
    return q, k.to(dtype)


SETS = {
    # 1 of 128 channels x30: concentrated and dominant -> strong
    "strong-bf16": dict(args=(4, 4, 2, 256, 128, torch.bfloat16, 30.0, 1.0, 1, 1), branch=1),
    # same stripe, Q three times larger: T falls between 2 and 3 -> mild
    "mild-fp16": dict(args=(3, 4, 2, 128, 128, torch.float16, 12.0, 3.2, 1, 2), branch=2),
    # 4 of 64 channels x20: more than 1 % of K is large, P99 sits inside the stripe -> bypass
    "diffuse-bypass": dict(args=(2, 2, 1, 128, 64, torch.bfloat16, 20.0, 1.0, 4, 3), branch=0),
    # no outliers at all -> bypass
    "plain-bypass": dict(args=(2, 2, 2, 64, 256, torch.bfloat16, 1.0, 1.0, 0, 4), branch=0),
}


@pytest.mark.parametrize("name", list(SETS))
def test_gate_matches_oracle(hb, oracle, name):
    spec = SETS[name]
    q, k = _cal(*spec["args"])
    ref = oracle.smooth_calibrate(q.float().numpy(), k.float().numpy(), 3)
    assert ref["branch"] == spec["branch"], (ref["rho_K"], ref["T_KQ"])       # the set lands where it was built to
    s, inv_s, stats = hb.smooth_calibrate_auto(q.to(DEV), k.to(DEV))
    torch.cuda.synchronize()
    st = stats.cpu().numpy()
    assert st[0] == np.float32(ref["rho_K"]) and st[1] == np.float32(ref["T_KQ"])   # same doubles, rounded once
    assert int(st[2]) == ref["branch"] and st[3] == np.float32(ref["alpha"])
    assert np.allclose(s.cpu().numpy(), ref["s"], rtol=1e-6, atol=0)
    assert np.array_equal(inv_s.cpu().numpy(), (np.float32(1) / s.cpu().numpy()).astype(np.float32))
    # the factors are those of the fixed-mode call for the branch the gate took
    fixed, _ = hb.smooth_calibrate(q.to(DEV), k.to(DEV), spec["branch"])
    assert torch.equal(s, fixed)


def test_gate_percentile_is_exact_on_ties_and_edges(hb, oracle):
    """All of K equal (P99 = max, rho = 1), and a K whose 99th-percentile rank falls on the last
    element below a jump."""
    q = torch.ones((1, 1, 64, 64), dtype=torch.bfloat16)
    k = torch.full((1, 1, 64, 64), 2.0, dtype=torch.bfloat16)
    _, _, st = hb.smooth_calibrate_auto(q.to(DEV), k.to(DEV))
    assert st.cpu().tolist() == [1.0, 2.0, 0.0, 0.0]
    n = 64 * 64
    flat = torch.ones(n)
    rank = int(np.ceil(0.99 * n))
    flat[rank:] = 64.0                                  # ranks rank+1.. hold the large value: P99 is still 1
    k2 = flat.reshape(1, 1, 64, 64).to(torch.bfloat16)
    ref = oracle.smooth_calibrate(q.float().numpy(), k2.float().numpy(), 3)
    _, _, st2 = hb.smooth_calibrate_auto(q.to(DEV), k2.to(DEV))
    assert st2.cpu().tolist() == [64.0, 64.0, 1.0, 0.5] and ref["branch"] == 1 and ref["rho_K"] == 64.0
    flat[rank - 1] = 64.0                               # now the rank itself is large: P99 = 64, rho = 1
    k3 = flat.reshape(1, 1, 64, 64).to(torch.bfloat16)
    _, _, st3 = hb.smooth_calibrate_auto(q.to(DEV), k3.to(DEV))
    assert st3.cpu().tolist() == [1.0, 64.0, 0.0, 0.0]


@pytest.mark.parametrize("agg", ["rms", "mean", "p99"])
def test_calibration_aggregators_match_the_oracle(hb, oracle, agg):
    """Mean and 99th-percentile aggregation of the per-sample channel maxima (the alternatives of the paper's
    aggregator comparison) beside the adopted root-mean-square: factors equal to the oracle's to 1e-6."""
    gen = torch.Generator().manual_seed(31)
    S, Hq, Hkv, Ncal, d = 120, 4, 2, 8, 128
    spread = torch.exp(torch.randn((S, 1, 1, 1), generator=gen) * 0.4)
    q = (torch.randn((S, Hq, Ncal, d), generator=gen) * spread).to(torch.bfloat16)
    k = (torch.randn((S, Hkv, Ncal, d), generator=gen) * spread * 3).to(torch.bfloat16)
    flag_o = {"rms": oracle.AGG_RMS, "mean": oracle.AGG_MEAN, "p99": oracle.AGG_P99}[agg]
    flag_g = {"rms": hb.AGG_RMS, "mean": hb.AGG_MEAN, "p99": hb.AGG_P99}[agg]
    ref = oracle.smooth_calibrate(q.float().numpy(), k.float().numpy(), 1, aggregator=flag_o)
    s, inv_s = hb.smooth_calibrate(q.to(DEV), k.to(DEV), 1, aggregator=flag_g)
    assert np.allclose(s.cpu().numpy(), ref["s"], rtol=1e-6)
    assert torch.equal(inv_s, 1.0 / s)
    if agg != "rms":
        base, _ = hb.smooth_calibrate(q.to(DEV), k.to(DEV), 1)
        assert not torch.equal(base, s)
    with pytest.raises(hb.Hifa4Error):
        hb.smooth_calibrate(q.to(DEV), k.to(DEV), 1, aggregator=0x300)
