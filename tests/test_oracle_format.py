"""Pins for the oracle's number formats: FP16/BF16 rounding and the HIF4 group
encoding (Background, "HIF4").  Nothing here touches the CUDA path."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hif4_reading_examples.txt")


# ---------------------------------------------------------------- roundings
def test_rn_f16_matches_numpy(oracle):
    rng = np.random.default_rng(0)
    xs = np.concatenate([
        rng.standard_normal(2000) * 10.0 ** rng.integers(-9, 5, 2000),
        [0.0, 1.0, 65504.0, 65519.9, 65520.0, 7e4, 2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -25,
         2.0 ** -14, 2.0 ** -14 - 2.0 ** -26, 1 + 2.0 ** -11, 1 + 3 * 2.0 ** -11, -1 - 2.0 ** -11],
    ])
    with np.errstate(over="ignore"):
        want = xs.astype(np.float16).astype(np.float64)
    got = np.array([oracle.rn_f16(x) for x in xs])
    assert np.array_equal(got, want)


def test_rn_bf16_matches_torch(oracle):
    rng = np.random.default_rng(1)
    xs = np.concatenate([rng.standard_normal(2000) * 10.0 ** rng.integers(-30, 30, 2000),
                         [1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -9, 3.0e38]])
    # torch rounds a double to bf16 through float32 only if asked; go straight from float64
    want = torch.tensor(xs, dtype=torch.float64).to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([oracle.rn_bf16(x) for x in xs])
    assert np.array_equal(got, want)


def test_e6m2_table(oracle):
    vals = [oracle.e6m2_value(c) for c in range(256)]
    assert vals[0] == 2.0 ** -48 and vals[255] == 1.75 * 2.0 ** 15
    assert vals[48 * 4] == 1.0 and vals[45 * 4 + 1] == 0.15625
    assert all(b > a for a, b in zip(vals, vals[1:]))           # strictly increasing codes
    # 6-bit exponent, 2-bit mantissa: four values per binade
    assert vals[4] / vals[0] == 2.0 and [v / vals[8] for v in vals[8:12]] == [1, 1.25, 1.5, 1.75]


# ---------------------------------------------------------------- golden examples
def _parse_sparse(txt, n=64):
    parts = txt.split()
    base = float(parts[0].split("=")[1])
    arr = np.full(n, base)
    for p in parts[1:]:
        v, i = p.split("@")
        arr[int(i)] = float(v)
    return arr


def _golden():
    rows = []
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, xin, meta, codes, dec = [f.strip() for f in line.split("|")]
        rows.append((name, _parse_sparse(xin), int(meta, 16), _parse_sparse(codes).astype(np.uint8),
                     _parse_sparse(dec)))
    return rows


@pytest.mark.parametrize("case", _golden(), ids=lambda c: c[0])
def test_hif4_golden_examples(oracle, case):
    _, x, meta, nib, dec = case
    codes, m, deq = oracle.hif4_quantize_rows(x[None])
    got_nib = np.empty(64, np.uint8)
    got_nib[0::2] = codes[0] & 15
    got_nib[1::2] = codes[0] >> 4
    assert int(m[0, 0]) == meta, hex(int(m[0, 0]))
    assert np.array_equal(got_nib, nib)
    assert np.array_equal(deq[0], dec)
    assert np.array_equal(oracle.hif4_decode_rows(codes, m)[0], dec)


# ---------------------------------------------------------------- brute force on small inputs
def _brute_encode(x):
    """Enumerative statement of the reading, in exact rational arithmetic."""
    xf = [Fraction(float(v)) for v in x]
    A = max(abs(v) for v in xf)
    if A == 0:
        return 0, [0] * 64
    e6m2 = [Fraction(4 + (c & 3), 4) * Fraction(2) ** ((c >> 2) - 48) for c in range(256)]
    ok = [c for c in range(256) if 7 * e6m2[c] >= A]
    code = min(ok, key=lambda c: e6m2[c]) if ok else 255
    S = e6m2[code]
    need = []
    for t in range(16):
        At = max(abs(v) for v in xf[4 * t:4 * t + 4])
        ks = [k for k in (0, 1, 2) if 7 * S * 2 ** k / 4 >= At]
        need.append(min(ks) if ks else 2)
    meta = code
    shift = [0] * 16
    for u in range(8):
        best = None
        for a in (1, 0):                      # a = 1 wins a tie in total shift
            for b0 in (0, 1):
                for b1 in (0, 1):
                    if a + b0 >= need[2 * u] and a + b1 >= need[2 * u + 1]:
                        cost = 2 * a + b0 + b1
                        if best is None or cost < best[0]:
                            best = (cost, a, b0, b1)
        _, a, b0, b1 = best
        meta |= (a << (8 + u)) | (b0 << (16 + 2 * u)) | (b1 << (17 + 2 * u))
        shift[2 * u], shift[2 * u + 1] = a + b0, a + b1
    nib = []
    for i, v in enumerate(xf):
        step = S * 2 ** shift[i // 4] / 4
        cands = sorted(range(8), key=lambda m: (abs(abs(v) - m * step), m & 1))   # nearest, even on ties
        m = cands[0]
        nib.append(m | (8 if (v < 0 and m > 0) else 0))
    return meta, nib


def _unpack(codes):
    nib = np.empty(codes.shape[:-1] + (codes.shape[-1] * 2,), np.uint8)
    nib[..., 0::2] = codes & 15
    nib[..., 1::2] = codes >> 4
    return nib


def test_hif4_matches_bruteforce(oracle):
    rng = np.random.default_rng(7)
    groups = []
    for trial in range(160):
        kind = trial % 8
        x = rng.standard_normal(64)
        if kind == 1:
            x[rng.integers(64)] *= 20
        elif kind == 2:
            x = np.abs(x) * 2.0 ** rng.integers(-20, 10)
        elif kind == 3:      # values on a coarse grid: many exact ties and threshold hits
            x = rng.integers(-28, 29, 64) * 0.125 * 2.0 ** rng.integers(-3, 4)
        elif kind == 4:
            x = np.exp(-np.abs(rng.standard_normal(64)) * 4)      # softmax-like row
            x[rng.integers(64)] = 1.0
        elif kind == 5:      # exactly 7*S, 1.75*S, 3.5*S for random S
            S = oracle.e6m2_value(int(rng.integers(150, 230)))
            x = rng.choice([7 * S, 1.75 * S, 3.5 * S, 0.5 * S / 4, 1.5 * S / 4, 2.5 * S, 0.0], 64)
        elif kind == 6:
            x = np.float16(x).astype(np.float64)
        elif kind == 7:
            x[:] = 0
            x[rng.integers(64)] = rng.standard_normal()
        groups.append(x)
    X = np.array(groups)
    codes, meta, _ = oracle.hif4_quantize_rows(X)
    nib = _unpack(codes)
    for g, x in enumerate(X):
        bmeta, bnib = _brute_encode(x)
        assert int(meta[g, 0]) == bmeta, (g, hex(int(meta[g, 0])), hex(bmeta))
        assert list(nib[g]) == bnib, g


# ---------------------------------------------------------------- invariants
def _steps(meta):
    """Per-element step from metadata, written independently of the C decoder."""
    meta = np.asarray(meta, np.uint64)
    e = ((meta >> np.uint64(2)) & np.uint64(63)).astype(np.int64)
    M = (meta & np.uint64(3)).astype(np.float64)
    S = (1 + M / 4) * 2.0 ** (e - 48)
    i = np.arange(64)
    a = (meta[..., None] >> (8 + i // 8).astype(np.uint64)) & np.uint64(1)
    b = (meta[..., None] >> (16 + i // 4).astype(np.uint64)) & np.uint64(1)
    return S[..., None] * 2.0 ** (a + b).astype(np.float64) / 4


def test_hif4_invariants(oracle):
    rng = np.random.default_rng(3)
    X = rng.standard_normal((400, 64)) * np.exp(rng.standard_normal((400, 1)) * 2)
    X[::5, 7] *= 30
    assert np.abs(X).max() < 7 * oracle.e6m2_value(255)       # inside the E6M2 range: no clamping
    codes, meta, deq = oracle.hif4_quantize_rows(X)
    step = _steps(meta[:, 0])
    nib = _unpack(codes)
    # decoded = sign * m * step, and no element is further than half a step away (no clipping)
    assert np.array_equal(deq, np.where(nib & 8, -1.0, 1.0) * (nib & 7) * step)
    assert np.all(np.abs(X - deq) <= step / 2 * (1 + 1e-15))
    # the scale is minimal: the group max exceeds what the next smaller E6M2 value could hold
    code = (meta[:, 0] & 0xFF).astype(int)
    S = np.array([oracle.e6m2_value(c) for c in code])
    Sprev = np.array([oracle.e6m2_value(max(c - 1, 0)) for c in code])
    A = np.abs(X).max(1)
    assert np.all(7 * S >= A) and np.all(7 * Sprev < A)
    # storage: 4 bits per element + 32 bits per 64 -> 4.5 bits per value
    assert (codes.nbytes + meta.nbytes) * 8 / X.size == 4.5
    # power-of-two homogeneity and sign symmetry
    c2, m2, d2 = oracle.hif4_quantize_rows(X * 2.0 ** -5)
    assert np.array_equal(c2, codes) and np.array_equal(d2, deq / 32)
    assert np.array_equal((m2[:, 0] & 0xFF).astype(int), code - 5 * 4)
    assert np.array_equal(m2 >> 8, meta >> 8)
    c3, m3, d3 = oracle.hif4_quantize_rows(-X)
    assert np.array_equal(d3, -deq) and np.array_equal(m3, meta)
    # permuting inside every 4-subgroup permutes codes only
    perm = np.arange(64).reshape(16, 4)[:, [2, 0, 3, 1]].reshape(-1)
    c4, m4, d4 = oracle.hif4_quantize_rows(X[:, perm])
    assert np.array_equal(m4, meta) and np.array_equal(d4, deq[:, perm])
    # representable inputs whose maximum is exactly 7*S come back unchanged
    grid = (rng.integers(-7, 8, (50, 64))).astype(np.float64) * 0.25
    grid[:, 0] = 1.75                                           # 7 * S / 4 with S = 1: finest step holds it
    _, mg, dg = oracle.hif4_quantize_rows(grid)
    assert np.array_equal(dg, grid)


def test_zero_group_and_single_outlier(oracle):
    z = np.zeros((1, 128))
    codes, meta, deq = oracle.hif4_quantize_rows(z)
    assert not codes.any() and not meta.any() and not deq.any()
    # the outlier pathology the paper describes: one large element flushes the rest
    x = np.ones((1, 64)); x[0, 5] = 100
    _, _, deq = oracle.hif4_quantize_rows(x)
    assert deq[0, 5] == 96 and np.count_nonzero(deq) == 1


def test_scale_range_clamps(oracle):
    """Outside the E6M2 range the scale code clamps (largest code: elements saturate at 7;
    smallest code: values far below the finest step flush to zero)."""
    big = np.zeros((1, 64)); big[0, 0] = 1e9; big[0, 1] = -3e5
    codes, meta, deq = oracle.hif4_quantize_rows(big)
    assert int(meta[0, 0]) & 0xFF == 255 and deq[0, 0] == 7 * oracle.e6m2_value(255)
    tiny = np.full((1, 64), 2.0 ** -60)
    codes, meta, deq = oracle.hif4_quantize_rows(tiny)
    assert int(meta[0, 0]) & 0xFF == 0 and not deq.any()
