"""ctypes front end of the HiFA4 CPU oracle (hifa4_oracle.c).

TEST INFRASTRUCTURE: only tests, the smoke check and the benchmark's
cpu_baseline / reference legs may import this module.  It compiles the C file
beside it with gcc on first use and exposes numpy-facing wrappers.  It imports
nothing from the CUDA package.

Parity unpinned: the HIF4 element/scale conversion is a reading of the format
facts the paper states (Background, "HIF4"); see the header of the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hifa4_oracle.c")
_LIB = os.path.join(_HERE, "libhifa4_oracle.so")
_lib = None

F16, BF16, F32, F64 = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
             _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class Params(C.Structure):
    _fields_ = [("N", C.c_int), ("d", C.c_int), ("causal", C.c_int), ("Bc", C.c_int),
                ("in_dtype", C.c_int),
                ("quant_q", C.c_int), ("quant_k", C.c_int), ("quant_v", C.c_int), ("quant_p", C.c_int),
                ("v_axis", C.c_int), ("normalizer", C.c_int), ("qmean", C.c_int),
                ("state", C.c_int), ("p_dtype", C.c_int), ("out_dtype", C.c_int),
                ("softmax_scale", C.c_double)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.hifa4_oracle_rn_f16.restype = C.c_double
        _lib.hifa4_oracle_rn_f16.argtypes = [C.c_double]
        _lib.hifa4_oracle_rn_bf16.restype = C.c_double
        _lib.hifa4_oracle_rn_bf16.argtypes = [C.c_double]
        _lib.hifa4_oracle_e6m2_value.restype = C.c_double
        _lib.hifa4_oracle_e6m2_value.argtypes = [C.c_int]
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def num_threads() -> int:
    return int(lib().hifa4_oracle_num_threads())


def rn_f16(x: float) -> float:
    return float(lib().hifa4_oracle_rn_f16(float(x)))


def rn_bf16(x: float) -> float:
    return float(lib().hifa4_oracle_rn_bf16(float(x)))


def e6m2_value(code: int) -> float:
    return float(lib().hifa4_oracle_e6m2_value(int(code)))


def hif4_quantize_rows(x: np.ndarray):
    """Quantize along the last axis (length % 64 == 0).

    Returns (codes uint8 [..., len/2], meta uint32 [..., len/64], deq float64)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    ln = x.shape[-1]
    rows = x.size // ln
    codes = np.empty(x.shape[:-1] + (ln // 2,), np.uint8)
    meta = np.empty(x.shape[:-1] + (ln // 64,), np.uint32)
    deq = np.empty_like(x)
    rc = lib().hifa4_oracle_hif4_quantize_rows(
        _p(x, C.c_double), C.c_long(rows), C.c_long(ln), _p(codes, C.c_uint8),
        _p(meta, C.c_uint32), _p(deq, C.c_double))
    if rc:
        raise ValueError("hif4_quantize_rows: length must be a multiple of 64")
    return codes, meta, deq


def hif4_decode_rows(codes: np.ndarray, meta: np.ndarray) -> np.ndarray:
    """Decode packed codes + metadata back to float64 values."""
    codes = np.ascontiguousarray(codes, np.uint8)
    meta = np.ascontiguousarray(meta, np.uint32)
    ln = codes.shape[-1] * 2
    nib = np.empty(codes.shape[:-1] + (ln,), np.uint8)
    nib[..., 0::2] = codes & 15
    nib[..., 1::2] = codes >> 4
    nibf = nib.reshape(-1, 64)
    metaf = meta.reshape(-1)
    out = np.empty(nibf.shape, np.float64)
    L = lib()
    for g in range(nibf.shape[0]):
        L.hifa4_oracle_hif4_decode_group(_p(nibf[g], C.c_uint8), C.c_uint32(int(metaf[g])),
                                         _p(out[g], C.c_double))
    return out.reshape(nib.shape)


def smooth_apply(x: np.ndarray, scale, dtype: int) -> np.ndarray:
    """round_dtype(fl32(x * scale)) per channel of the last axis; float64 result."""
    x = np.ascontiguousarray(x, np.float32)
    d = x.shape[-1]
    y = np.empty(x.shape, np.float64)
    sc = None if scale is None else np.ascontiguousarray(scale, np.float32)
    lib().hifa4_oracle_smooth_apply(_p(x, C.c_float), C.c_long(x.size // d), C.c_int(d),
                                    _p(sc, C.c_float), C.c_int(dtype), _p(y, C.c_double))
    return y


def smooth_quantize(x: np.ndarray, scale, dtype: int, axis_tokens: bool = False):
    """Smooth-QK scaling then HIF4 along channels (Q, K) or tokens (V).

    x [..., N, d].  For axis_tokens the result arrays are laid out [..., d, N/2]
    (codes) and [..., d, N/64] (meta), i.e. with the token axis last."""
    y = smooth_apply(x, scale, dtype)
    if axis_tokens:
        y = np.ascontiguousarray(np.swapaxes(y, -1, -2))
    return hif4_quantize_rows(y)


def qmean_rows(x: np.ndarray, scale, dtype: int):
    """Algorithm 1 lines 1-2 for Q: smooth, subtract the per-token mean (kept in FP16), round to the
    activation dtype.  x [..., N, d]; returns (q_z float64 [..., N, d], mu [..., N])."""
    x = np.ascontiguousarray(x, np.float32)
    d = x.shape[-1]
    rows = x.size // d
    y = np.empty(x.shape, np.float64)
    mu = np.empty(x.shape[:-1], np.float64)
    sc = None if scale is None else np.ascontiguousarray(scale, np.float32)
    lib().hifa4_oracle_qmean_rows(_p(x, C.c_float), C.c_long(rows), C.c_int(d), _p(sc, C.c_float),
                                  C.c_int(dtype), _p(y, C.c_double), _p(mu, C.c_double))
    return y, mu


def qmean_quantize(x: np.ndarray, scale, dtype: int):
    """Algorithm 1 lines 1-3 for Q with the Q-Mean auxiliary: qmean_rows, then HIF4 along channels.
    x [..., N, d]; returns (codes, meta, deq, mu [..., N])."""
    y, mu = qmean_rows(x, scale, dtype)
    return hif4_quantize_rows(y) + (mu,)


def ksum_rows(x: np.ndarray, scale, dtype: int) -> np.ndarray:
    """Sum over channels of the smoothed key, kept in FP16 (Algorithm 1 line 6).  x [..., N, d]."""
    x = np.ascontiguousarray(x, np.float32)
    d = x.shape[-1]
    ks = np.empty(x.shape[:-1], np.float64)
    sc = None if scale is None else np.ascontiguousarray(scale, np.float32)
    lib().hifa4_oracle_ksum_rows(_p(x, C.c_float), C.c_long(x.size // d), C.c_int(d), _p(sc, C.c_float),
                                 C.c_int(dtype), _p(ks, C.c_double))
    return ks


AGG_RMS, AGG_MEAN, AGG_P99 = 0, 0x100, 0x200


def smooth_calibrate(q_cal: np.ndarray, k_cal: np.ndarray, mode: int, alpha: float = 0.0,
                     q_to_kv=None, aggregator: int = AGG_RMS):
    """q_cal [S,Hq,Ncal,d], k_cal [S,Hkv,Ncal,d] -> dict(s, inv_s, kagg, qagg, stats).
    aggregator: how the per-sample channel maxima are combined over samples (RMS, mean, 99th percentile)."""
    mode = int(mode) | int(aggregator)
    q_cal = np.ascontiguousarray(q_cal, np.float32)
    k_cal = np.ascontiguousarray(k_cal, np.float32)
    S, Hq, Ncal, d = q_cal.shape
    Hkv = k_cal.shape[1]
    s = np.empty((Hkv, d), np.float32)
    inv_s = np.empty((Hkv, d), np.float32)
    kagg = np.empty((Hkv, d), np.float64)
    qagg = np.empty((Hkv, d), np.float64)
    stats = np.zeros(4, np.float64)
    mp = None if q_to_kv is None else np.ascontiguousarray(q_to_kv, np.int32)
    rc = lib().hifa4_oracle_smooth_calibrate(
        _p(q_cal, C.c_float), _p(k_cal, C.c_float), S, Hq, Hkv, Ncal, d, _p(mp, C.c_int),
        C.c_int(mode), C.c_double(alpha), _p(s, C.c_float), _p(inv_s, C.c_float),
        _p(kagg, C.c_double), _p(qagg, C.c_double), _p(stats, C.c_double))
    if rc:
        raise RuntimeError(f"oracle calibrate failed: {rc}")
    return dict(s=s, inv_s=inv_s, kagg=kagg, qagg=qagg,
                rho_K=stats[0], T_KQ=stats[1], branch=int(stats[2]), alpha=stats[3])


def attention_rows(q_rows, q_pos, k, v, s=None, inv_s=None, *, causal=False, Bc=128,
                   in_dtype=BF16, quant=(1, 1, 1, 1), v_axis=0, normalizer=0, qmean=0,
                   state=0, p_dtype=F16, out_dtype=F32, softmax_scale=0.0, dumps=False):
    """Algorithm 1 for query rows sharing one KV head.

    q_rows [R,d], q_pos [R], k,v [N,d] (float32 holding the 16-bit input values).
    Returns out [R,d] float64, or (out, dict of dumps) when dumps=True."""
    q_rows = np.ascontiguousarray(q_rows, np.float32)
    k = np.ascontiguousarray(k, np.float32)
    v = np.ascontiguousarray(v, np.float32)
    R, d = q_rows.shape
    N = k.shape[0]
    q_pos = np.ascontiguousarray(q_pos, np.int32)
    prm = Params(N, d, int(causal), Bc, in_dtype, quant[0], quant[1], quant[2], quant[3],
                 v_axis, normalizer, qmean, state, p_dtype, out_dtype, float(softmax_scale))
    out = np.empty((R, d), np.float64)
    sc = None if s is None else np.ascontiguousarray(s, np.float32)
    isc = None if inv_s is None else np.ascontiguousarray(inv_s, np.float32)
    nt = (N + Bc - 1) // Bc
    if dumps:
        pc = np.zeros((R, N), np.uint8)
        ps = np.zeros((R, N // 4), np.float32)
        pr = np.zeros((R, N), np.float64)
        ph = np.zeros((R, N), np.float64)
        mt = np.zeros((R, nt), np.float64)
        lo = np.zeros(R, np.float64)
    else:
        pc = ps = pr = ph = mt = lo = None
    rc = lib().hifa4_oracle_attention_rows(
        C.byref(prm), _p(q_rows, C.c_float), _p(q_pos, C.c_int), C.c_int(R), _p(k, C.c_float),
        _p(v, C.c_float), _p(sc, C.c_float), _p(isc, C.c_float), _p(out, C.c_double),
        _p(pc, C.c_uint8), _p(ps, C.c_float), _p(pr, C.c_double), _p(ph, C.c_double),
        _p(mt, C.c_double), _p(lo, C.c_double))
    if rc:
        raise RuntimeError(f"oracle attention failed: {rc}")
    if dumps:
        return out, dict(p_codes=pc, p_step=ps, p_raw=pr, p_hat=ph, m_trace=mt, l=lo)
    return out


def attention(q, k, v, s=None, inv_s=None, q_to_kv=None, rows=None, **kw):
    """Whole-tensor driver.  q [B,Hq,N,d], k,v [B,Hkv,N,d]; s, inv_s [Hkv,d].

    rows: optional list of (b, h, i) to evaluate (others are not computed).
    Returns out [B,Hq,N,d] float64 (NaN where not computed) and, with
    dumps=True, a dict keyed by (b, h) of (row indices, per-row dumps)."""
    B, Hq, N, d = q.shape
    Hkv = k.shape[1]
    out = np.full((B, Hq, N, d), np.nan, np.float64)
    dumps = {}
    want = {}
    if rows is None:
        for b in range(B):
            for h in range(Hq):
                want[(b, h)] = np.arange(N, dtype=np.int32)
    else:
        for (b, h, i) in rows:
            want.setdefault((b, h), []).append(i)
    for (b, h), idx in want.items():
        idx = np.asarray(idx, np.int32)
        g = int(q_to_kv[h]) if q_to_kv is not None else h // (Hq // Hkv)
        res = attention_rows(q[b, h, idx], idx, k[b, g], v[b, g],
                             None if s is None else s[g], None if inv_s is None else inv_s[g], **kw)
        if kw.get("dumps"):
            out[b, h, idx] = res[0]
            dumps[(b, h)] = (idx, res[1])
        else:
            out[b, h, idx] = res
    return (out, dumps) if kw.get("dumps") else out
