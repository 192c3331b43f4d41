"""Pins for the oracle's Algorithm 1 (C4V16-Aux) and Smooth-QK: brute force,
Theorem 1's closed forms, and the invariants the method states."""
import numpy as np
import pytest
import torch

from paper_2607_04302_b200 import synth


def _np(t):
    return t.float().numpy()


def _brute(q, k, v, causal, q_pos=None, scale=None):
    """softmax(q k^T / sqrt(d)) v in float64; q [R,d], k,v [N,d]."""
    q, k, v = (np.asarray(a, np.float64) for a in (q, k, v))
    s = q @ k.T * (scale if scale else 1.0 / np.sqrt(q.shape[1]))
    if causal:
        mask = np.arange(k.shape[0])[None, :] > np.asarray(q_pos)[:, None]
        s = np.where(mask, -np.inf, s)
    s = s - s.max(1, keepdims=True)
    p = np.exp(s)
    return (p / p.sum(1, keepdims=True)) @ v


def _small(seed=0, N=256, d=128, R=48, outl=True):
    rng = np.random.default_rng(seed)
    f = lambda *sh: rng.standard_normal(sh).astype(np.float16).astype(np.float32)
    q, k, v = f(R, d), f(N, d), f(N, d)
    if outl:
        k[:, [3, 17, 64, 101]] = (k[:, [3, 17, 64, 101]] * 20).astype(np.float16).astype(np.float32)
    pos = np.sort(rng.choice(N, R, replace=False)).astype(np.int32)
    return q, k, v, pos


# ---- check 1: identity quantizer == exact softmax attention -------------------------------
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("Bc", [64, 128])
def test_identity_quantizer_is_exact_attention(oracle, causal, Bc):
    q, k, v, pos = _small(1)
    out = oracle.attention_rows(q, pos, k, v, causal=causal, Bc=Bc, quant=(0, 0, 0, 0), state=1,
                                in_dtype=oracle.F16, out_dtype=oracle.F64)
    ref = _brute(q, k, v, causal, pos)
    assert np.max(np.abs(out - ref)) <= 1e-12 * max(1.0, np.abs(ref).max())


def test_fp16_state_stays_close_to_exact(oracle):
    q, k, v, pos = _small(2, outl=False)
    out = oracle.attention_rows(q, pos, k, v, causal=True, Bc=64, quant=(0, 0, 0, 0), state=0,
                                in_dtype=oracle.F16)
    ref = _brute(q, k, v, True, pos)
    assert np.linalg.norm(out - ref) / np.linalg.norm(ref) < 1e-3


# ---- check 2: Smooth-QK leaves QK^T unchanged; alpha = 0.5 equalises; bypass is identity ---
def test_smooth_qk_invariance_and_equalisation(oracle):
    cfg = synth.config("C1")
    qc, kc = synth.make_calibration(cfg)
    cal = oracle.smooth_calibrate(_np(qc), _np(kc), mode=1)
    s, inv_s = cal["s"], cal["inv_s"]
    # calibration aggregate: |K|/s == |Q| s == sqrt(|K||Q|) per channel (Eq. "sqk", alpha = .5)
    geo = np.sqrt(cal["kagg"] * cal["qagg"])
    assert np.allclose(cal["kagg"] / s, geo, rtol=2e-7) and np.allclose(cal["qagg"] * s, geo, rtol=2e-7)
    # the outlier channels get the large scales
    top = set(np.argsort(-s[0])[:4].tolist())
    assert top == {3, 17, 64, 101}
    q, k, v = (_np(t)[0, 0] for t in synth.make_qkv(cfg))
    sd = s[0].astype(np.float64)
    qt = oracle.smooth_apply(q, s[0], oracle.F64)
    kt = oracle.smooth_apply(k, (1.0 / sd).astype(np.float32), oracle.F64)
    # exact arithmetic: use the true reciprocal in double
    kt = k.astype(np.float64) / sd
    ref = q.astype(np.float64) @ k.astype(np.float64).T
    assert np.max(np.abs(qt @ kt.T - ref)) <= 1e-13 * np.abs(ref).max()
    # through the whole operator with the identity quantizer and no intermediate rounding
    pos = np.arange(q.shape[0], dtype=np.int32)
    kw = dict(causal=False, Bc=64, quant=(0, 0, 0, 0), state=1, in_dtype=oracle.F64, out_dtype=oracle.F64)
    a = oracle.attention_rows(q, pos, k, v, **kw)
    b = oracle.attention_rows(q, pos, k, v, s[0], inv_s[0], **kw)
    assert np.max(np.abs(a - b)) < 1e-6            # inv_s is a rounded fp32 reciprocal
    # bypass: s = 1 is bit-identical to no smoothing, quantizers on
    one = np.ones(cfg.d, np.float32)
    kw = dict(causal=False, Bc=64, in_dtype=oracle.F16)
    assert np.array_equal(oracle.attention_rows(q, pos, k, v, **kw),
                          oracle.attention_rows(q, pos, k, v, one, one, **kw))


def test_calibration_aggregators_against_numpy(oracle):
    """The three ways of combining the per-sample channel maxima over the calibration set (the paper's
    aggregator comparison: RMS adopted, mean and 99th percentile as alternatives), pinned against numpy
    reductions of the per-sample maxima (np.percentile's inverted-CDF method is the nearest-rank rule)."""
    rng = np.random.default_rng(21)
    S, Hq, Hkv, Ncal, d = 120, 2, 1, 4, 64
    qc = (rng.standard_normal((S, Hq, Ncal, d)) * np.exp(rng.standard_normal((S, 1, 1, 1)) * 0.4)).astype(np.float32)
    kc = (rng.standard_normal((S, Hkv, Ncal, d)) * np.exp(rng.standard_normal((S, 1, 1, 1)) * 0.4)).astype(np.float32)
    kmax = np.abs(kc.astype(np.float64)).max(axis=2)[:, 0]              # [S, d]
    qmax = np.abs(qc.astype(np.float64)).max(axis=(1, 2))               # [S, d], both query heads share the KV head
    want = {oracle.AGG_RMS: (np.sqrt((kmax ** 2).mean(0)), np.sqrt((qmax ** 2).mean(0))),
            oracle.AGG_MEAN: (kmax.mean(0), qmax.mean(0)),
            oracle.AGG_P99: (np.percentile(kmax, 99, axis=0, method="inverted_cdf"),
                             np.percentile(qmax, 99, axis=0, method="inverted_cdf"))}
    got = {}
    for agg, (kw, qw) in want.items():
        cal = oracle.smooth_calibrate(qc, kc, mode=2, aggregator=agg)
        assert np.allclose(cal["kagg"][0], kw, rtol=1e-13) and np.allclose(cal["qagg"][0], qw, rtol=1e-13)
        s_want = kw ** 0.25 / qw ** 0.75
        assert np.allclose(cal["s"][0], s_want, rtol=1e-6) and np.array_equal(cal["inv_s"], (1.0 / cal["s"]).astype(np.float32))
        got[agg] = cal["kagg"][0]
    # the three differ on this data, in the order mean < RMS < 99th percentile (second largest of 120 samples)
    assert np.all(got[oracle.AGG_MEAN] < got[oracle.AGG_RMS]) and np.all(got[oracle.AGG_RMS] < got[oracle.AGG_P99])
    assert np.array_equal(got[oracle.AGG_P99], np.sort(kmax, axis=0)[-2])


def test_calibration_modes_and_gate(oracle):
    rng = np.random.default_rng(5)
    qc = rng.standard_normal((3, 4, 64, 64)).astype(np.float32)
    kc = rng.standard_normal((3, 2, 64, 64)).astype(np.float32)
    kc[..., 5] *= 40
    byp = oracle.smooth_calibrate(qc, kc, mode=0)
    assert np.all(byp["s"] == 1) and np.all(byp["inv_s"] == 1)
    mild = oracle.smooth_calibrate(qc, kc, mode=2)
    strong = oracle.smooth_calibrate(qc, kc, mode=1)
    cust = oracle.smooth_calibrate(qc, kc, mode=4, alpha=0.25)
    assert np.array_equal(mild["s"], cust["s"]) and not np.array_equal(mild["s"], strong["s"])
    # statistics written independently: rho_K = max|K| / P99(|K|) (nearest rank), T = max|K| / max|Q|
    ak = np.sort(np.abs(kc).ravel())
    p99 = ak[int(np.ceil(0.99 * ak.size)) - 1]
    auto = oracle.smooth_calibrate(qc, kc, mode=3)
    assert np.isclose(auto["rho_K"], ak[-1] / p99) and np.isclose(auto["T_KQ"], ak[-1] / np.abs(qc).max())
    # 1 of 64 channels x40: concentrated (rho >= 6) and dominant (T > 3) -> strong branch
    assert auto["branch"] == 1 and np.array_equal(auto["s"], strong["s"])
    # no outliers -> bypass
    auto2 = oracle.smooth_calibrate(qc, rng.standard_normal((3, 2, 64, 64)).astype(np.float32), mode=3)
    assert auto2["branch"] == 0 and np.all(auto2["s"] == 1)
    # per-sample max then RMS over samples (not a global max): a one-sample spike is damped
    kc2 = kc.copy(); kc2[0, 0, 0, 9] = 1000.0
    c2 = oracle.smooth_calibrate(qc, kc2, mode=1)
    m = np.abs(kc2[:, 0, :, 9]).max(1)
    assert np.isclose(c2["kagg"][0, 9], np.sqrt(np.mean(m ** 2)))
    # degenerate channel (all-zero K) keeps s = 1
    kc3 = kc.copy(); kc3[..., 11] = 0
    assert np.all(oracle.smooth_calibrate(qc, kc3, mode=1)["s"][:, 11] == 1)
    # GQA: Q statistics pool the query heads that share a KV head
    qc4 = qc.copy(); qc4[:, 3, :, 2] *= 50             # head 3 belongs to kv head 1
    c4 = oracle.smooth_calibrate(qc4, kc, mode=1)
    assert c4["qagg"][1, 2] > 10 * c4["qagg"][0, 2]


# ---- check 3: P-Reordering: O = (sum P-hat V-hat) / rowsum(P-hat), across tiles ---------------
@pytest.mark.parametrize("state", [1, 0])
def test_p_reordering_identity(oracle, state):
    q, k, v, pos = _small(3)
    out, d = oracle.attention_rows(q, pos, k, v, causal=True, Bc=64, in_dtype=oracle.F16,
                                   state=state, out_dtype=oracle.F64 if state else oracle.F32, dumps=True)
    _, _, vh = oracle.hif4_quantize_rows(np.ascontiguousarray(v.T.astype(np.float64)))   # groups along tokens
    vh = vh.T
    mt = d["m_trace"]                                    # running max after each tile
    m_fin = np.nanmax(mt, axis=1)
    w = np.exp(np.repeat(mt, 64, axis=1) - m_fin[:, None])      # rescale factor each tile ends up with
    w = np.where(np.isnan(w), 0.0, w)
    ph = d["p_hat"] * w
    num, den = ph @ vh, ph.sum(1)
    tol = 1e-12 if state else 2e-3
    assert np.max(np.abs(out - num / den[:, None])) <= tol * np.abs(out).max()
    # P-hat really is a HIF4 tensor: re-decoding the dumped codes with the dumped steps gives it back
    nib = d["p_codes"]
    assert np.array_equal((nib & 7) * np.repeat(d["p_step"], 4, axis=1).astype(np.float64), d["p_hat"])
    assert not (nib & 8).any()                           # softmax weights are non-negative
    # masked keys are exact zeros
    for r, p_ in enumerate(pos):
        assert not d["p_hat"][r, p_ + 1:].any() and not d["p_raw"][r, p_ + 1:].any()


# ---- check 4: Theorem 1, both identities ------------------------------------------------------
@pytest.mark.parametrize("N,Bc", [(128, 128), (256, 64)])
def test_theorem1_closed_forms(oracle, N, Bc):
    rng = np.random.default_rng(11)
    d = 64
    q = rng.standard_normal((8, d)).astype(np.float32) * 1.5
    k = rng.standard_normal((N, d)).astype(np.float32)
    v = rng.standard_normal((N, d)).astype(np.float32)
    pos = np.full(8, N - 1, np.int32)
    kw = dict(causal=False, Bc=Bc, quant=(0, 0, 0, 1), state=1, in_dtype=oracle.F64, out_dtype=oracle.F64)
    o_con, dc = oracle.attention_rows(q, pos, k, v, normalizer=0, dumps=True, **kw)
    o_mis, dm = oracle.attention_rows(q, pos, k, v, normalizer=1, dumps=True, **kw)
    m_fin = np.nanmax(dc["m_trace"], axis=1)
    w = np.exp(np.repeat(dc["m_trace"], Bc, axis=1) - m_fin[:, None])
    a = dc["p_raw"] * w                 # a_j = exp(S_j - m)
    ah = dc["p_hat"] * w                # quantized weights under the same offset
    Z = a.sum(1, keepdims=True)
    wj = a / Z
    eps = ah / a - 1
    eps_bar = (wj * eps).sum(1, keepdims=True)
    delta = eps - eps_bar
    v64 = v.astype(np.float64)
    o_star = wj @ v64
    assert np.max(np.abs(o_star - _brute(q, k, v, False))) < 1e-13
    e_t = np.einsum("rj,rjc->rc", wj * delta, v64[None] - o_star[:, None, :])
    assert np.max(np.abs((o_con - o_star) - e_t / (1 + eps_bar))) < 5e-15
    assert np.max(np.abs((o_mis - o_star) - (e_t + eps_bar * o_star))) < 5e-15
    assert np.all(eps_bar < 0)          # net probability-mass loss on these rows
    # the mismatched normalizer is the sum of the unquantized weights
    assert np.allclose(dm["l"], (dm["p_raw"] * w).sum(1), rtol=1e-13)
    assert np.allclose(dc["l"], ah.sum(1), rtol=1e-13)


def test_eps_bar_sign_and_size_on_gaussian_scores(oracle):
    """Statistical sanity (paper: every measured tile loses mass, median -0.064)."""
    rng = np.random.default_rng(4)
    s = rng.standard_normal((4000, 64)) * 2.5
    p = np.exp(s - s.max(1, keepdims=True)).astype(np.float16).astype(np.float64)
    _, _, ph = oracle.hif4_quantize_rows(p)
    eps = ph.sum(1) / p.sum(1) - 1
    assert -0.12 < np.median(eps) < -0.03 and np.mean(eps < 0) > 0.9


# ---- structure: causal prefix, GQA broadcast, whole-tensor driver -----------------------------
def test_causal_equals_prefix_noncausal(oracle):
    q, k, v, _ = _small(6, N=256)
    pos = np.array([63, 127, 191, 255], np.int32)        # row ends exactly on a 64-key group
    kw = dict(Bc=64, in_dtype=oracle.F16)
    c = oracle.attention_rows(q[:4], pos, k, v, causal=True, **kw)
    for r, p_ in enumerate(pos):
        n = oracle.attention_rows(q[r:r + 1], pos[r:r + 1], k[:p_ + 1], v[:p_ + 1], causal=False, **kw)
        assert np.array_equal(c[r], n[0])


def test_gqa_equals_repeated_mha(oracle):
    cfg = synth.config("C2", N=128, Hq=4, Hkv=2)
    q, k, v = (_np(t) for t in synth.make_qkv(cfg))
    rng = np.random.default_rng(0)
    s = np.exp(rng.standard_normal((2, cfg.d)) * 0.3).astype(np.float32)
    inv_s = (1.0 / s).astype(np.float32)
    kw = dict(causal=True, Bc=64, in_dtype=oracle.BF16)
    a = oracle.attention(q, k, v, s, inv_s, **kw)
    b = oracle.attention(q, np.repeat(k, 2, 1), np.repeat(v, 2, 1), np.repeat(s, 2, 0),
                         np.repeat(inv_s, 2, 0), **kw)
    assert np.array_equal(a, b) and not np.isnan(a).any()
    # explicit head map reproduces the default grouping; sampled rows equal the full run
    c = oracle.attention(q, k, v, s, inv_s, q_to_kv=[0, 0, 1, 1], rows=[(0, 3, 5), (0, 0, 127)], **kw)
    assert np.array_equal(c[0, 3, 5], a[0, 3, 5]) and np.array_equal(c[0, 0, 127], a[0, 0, 127])
    assert np.isnan(c[0, 1]).all()


def test_smoothing_helps_on_outlier_inputs(oracle):
    """Method-level sanity on the tiny configuration: with x20 K channels, Smooth-QK lowers the
    error against exact attention (the paper's motivation for the transform)."""
    cfg = synth.config("C1")
    q, k, v = (_np(t)[0, 0] for t in synth.make_qkv(cfg))
    qc, kc = synth.make_calibration(cfg)
    cal = oracle.smooth_calibrate(_np(qc), _np(kc), mode=1)
    pos = np.arange(cfg.N, dtype=np.int32)
    ref = _brute(q, k, v, False)
    kw = dict(causal=False, Bc=64, in_dtype=oracle.F16)
    on = oracle.attention_rows(q, pos, k, v, cal["s"][0], cal["inv_s"][0], **kw)
    off = oracle.attention_rows(q, pos, k, v, **kw)
    rel = lambda x: np.linalg.norm(x - ref) / np.linalg.norm(ref)
    assert rel(on) < rel(off) and rel(on) < 0.5


def test_qmean_is_exact_without_quantization(oracle):
    """Algorithm 1 lines 2 and 6: subtracting the per-token mean of q and adding mu_i * sum_c k_jc
    back leaves the scores unchanged in exact arithmetic."""
    q, k, v, pos = _small(8)
    q = q + 0.7
    kw = dict(causal=True, Bc=64, quant=(0, 0, 0, 0), state=1, in_dtype=oracle.F64, out_dtype=oracle.F64)
    a = oracle.attention_rows(q, pos, k, v, qmean=0, **kw)
    b = oracle.attention_rows(q, pos, k, v, qmean=1, **kw)
    assert np.max(np.abs(a - b)) < 1e-11


def _cast16(x32: np.ndarray, dtype: str) -> np.ndarray:
    """float32 array -> 16-bit format and back, by the library casts (numpy float16, torch bfloat16)."""
    if dtype == "fp16":
        return x32.astype(np.float16).astype(np.float64)
    return torch.from_numpy(np.ascontiguousarray(x32)).to(torch.bfloat16).to(torch.float64).numpy()


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_smooth_apply_rounds_the_fp32_product_once_to_the_activation_dtype(oracle, dtype):
    """Algorithm 1 line 1 with a 16-bit activation: the smoothed value is the FP32 product of the stored
    activation and the factor, rounded once to the activation dtype (Appendix: the smoothed tensor is a
    transient 16-bit activation).  Pinned against numpy's float32 multiply and the library casts, on
    inputs where the rounding matters: skipping it, or rounding to the other 16-bit format, fails."""
    rng = np.random.default_rng(11)
    x = _cast16(rng.standard_normal((96, 128)).astype(np.float32) * 3.0, dtype).astype(np.float32)
    s = np.exp(rng.standard_normal(128) * 0.7).astype(np.float32)
    want = _cast16(x * s, dtype)                                   # numpy multiplies float32 in float32
    got = oracle.smooth_apply(x, s, oracle.F16 if dtype == "fp16" else oracle.BF16)
    assert np.array_equal(got, want)
    exact = x.astype(np.float64) * s.astype(np.float64)
    assert (want != exact).mean() > 0.9                            # the rounding is not a no-op here
    other = _cast16(x * s, "bf16" if dtype == "fp16" else "fp16")
    assert (want != other).mean() > 0.5                            # and the two formats differ on this data
    # no factor: the activation passes through untouched
    assert np.array_equal(oracle.smooth_apply(x, None, oracle.F16), x.astype(np.float64))


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_qmean_vectors_in_fp16_and_mean_free_query_in_the_activation_dtype(oracle, dtype):
    """Algorithm 1 lines 2 and 6 in the deployed precision (Appendix, "Q-Mean GEMV and coordinate
    consistency"): mu_i = FP16(mean_c q~_ic) and ksum_j = FP16(sum_c k~_jc) from exact sums of the smoothed
    16-bit activations, Q_z = q~ - mu rounded once to the activation dtype.  Pinned against numpy double
    sums and the library casts."""
    rng = np.random.default_rng(12)
    odt = oracle.F16 if dtype == "fp16" else oracle.BF16
    x = _cast16(rng.standard_normal((80, 128)).astype(np.float32) + 0.6, dtype).astype(np.float32)
    s = np.exp(rng.standard_normal(128) * 0.5).astype(np.float32)
    xt = _cast16(x * s, dtype)                                     # smoothed activation (line 1), float64 holder
    mu_want = xt.sum(1) / 128
    mu_want = mu_want.astype(np.float16).astype(np.float64)
    qz_want = _cast16((xt - mu_want[:, None]).astype(np.float32), dtype)
    # the difference of a 16-bit value and an FP16 value fits float32 exactly here (|values| < 2^5, bits > 2^-24)
    assert np.array_equal((xt - mu_want[:, None]).astype(np.float32).astype(np.float64), xt - mu_want[:, None])
    qz, mu = oracle.qmean_rows(x, s, odt)
    assert np.array_equal(mu, mu_want) and np.array_equal(qz, qz_want)
    assert np.abs(mu_want).min() > 0.05                            # the mean matters on this data
    assert (qz_want != xt - mu_want[:, None]).mean() > 0.2         # so does the rounding of Q_z
    ks_want = xt.sum(1).astype(np.float16).astype(np.float64)
    assert np.array_equal(oracle.ksum_rows(x, s, odt), ks_want)
    assert (ks_want != xt.sum(1)).mean() > 0.5                     # FP16 rounding of the key sums is visible
    # qmean_quantize = the same Q_z through the HIF4 encoder
    c, m, dq, mu2 = oracle.qmean_quantize(x, s, odt)
    c2, m2, dq2 = oracle.hif4_quantize_rows(qz_want)
    assert np.array_equal(c, c2) and np.array_equal(m, m2) and np.array_equal(dq, dq2) and np.array_equal(mu2, mu_want)


def test_p_dtype_flag_is_one_fp16_rounding(oracle):
    """The FP16-P default and the FP32-P variant differ by exactly one rounding of P: with the same scores
    and running maxima (the maxima do not depend on P), P16 = float16(P32) element by element (numpy's
    cast), P32 is an FP32 value, and P32 = fl32(exp2(t)) to FP32 accuracy."""
    q, k, v, pos = _small(5)
    kw = dict(causal=True, Bc=64, in_dtype=oracle.F16, dumps=True)
    _, d16 = oracle.attention_rows(q, pos, k, v, p_dtype=oracle.F16, **kw)
    _, d32 = oracle.attention_rows(q, pos, k, v, p_dtype=oracle.F32, **kw)
    assert np.array_equal(d16["m_trace"], d32["m_trace"], equal_nan=True)
    p16, p32 = d16["p_raw"], d32["p_raw"]
    assert np.array_equal(p32, p32.astype(np.float32).astype(np.float64))
    assert np.array_equal(p16, p32.astype(np.float16).astype(np.float64))
    assert (p16 != p32)[p32 > 0].mean() > 0.9            # the flag does something (masked keys are 0 in both)
    # and the codes differ in a small fraction of elements only (the two are different functions)
    frac = (d16["p_codes"] != d32["p_codes"]).mean()
    assert 0 < frac < 5e-3, frac
