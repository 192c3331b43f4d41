"""Thin ctypes binding of libhifa4 (the C ABI declared in include/hifa4.h).

Argument marshalling only: every step of the path runs in the CUDA kernels of the library.
torch supplies device memory and the current stream.  There is no CPU fallback: if the shared
library is missing or cannot be loaded, every call raises."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

from . import build as _build

F16, BF16, F32 = 0, 1, 2
Q, K, V = 0, 1, 2
CODES, META, MMA, AUX = 0, 1, 2, 3
MODE_BYPASS, MODE_STRONG, MODE_MILD, MODE_AUTO, MODE_CUSTOM = 0, 1, 2, 3, 4
AGG_RMS, AGG_MEAN, AGG_P99 = 0, 0x100, 0x200            # OR-ed into the calibration mode
MAX_DEBUG_BLOCKS = 16

_DT = {torch.float16: F16, torch.bfloat16: BF16, torch.float32: F32}
_TORCH_DT = {F16: torch.float16, BF16: torch.bfloat16, F32: torch.float32}


class Hifa4Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class _Shape(C.Structure):
    _fields_ = [("B", C.c_int), ("Hq", C.c_int), ("Hkv", C.c_int), ("N", C.c_int), ("d", C.c_int),
                ("q_to_kv", C.POINTER(C.c_int)), ("in_dtype", C.c_int)]


class _QKV(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("q_codes", "q_meta", "q_mma", "k_codes", "k_meta", "k_mma",
                                          "v_codes", "v_meta", "v_mma", "q_mu", "k_sum")]


class _AttnParams(C.Structure):
    _fields_ = [("causal", C.c_int), ("Br", C.c_int), ("Bc", C.c_int), ("normalizer", C.c_int),
                ("qmean", C.c_int), ("p_dtype", C.c_int), ("out_dtype", C.c_int),
                ("softmax_scale", C.c_float)]


class _Debug(C.Structure):
    _fields_ = [("n_blocks", C.c_int), ("blocks", C.POINTER(C.c_int)), ("p_codes", C.c_void_p),
                ("p_step", C.c_void_p), ("l_out", C.c_void_p), ("m_out", C.c_void_p)]


class _CalibStats(C.Structure):
    _fields_ = [("rho_K", C.c_float), ("T_KQ", C.c_float), ("branch", C.c_int), ("alpha", C.c_float)]


class _MassStats(C.Structure):
    _fields_ = [("hist", C.c_void_p), ("n_bins", C.c_int), ("lo", C.c_double), ("hi", C.c_double)]


_lib = None


def lib_path() -> str:
    return _build.LIB


def lib():
    """Load libhifa4.so (built in-tree by paper_2607_04302_b200.build).  Raises if it is absent."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise FileNotFoundError(
                f"{path} not found: build it with `python -m paper_2607_04302_b200.build` "
                "(the HiFA4 path has no CPU fallback)")
        L = C.CDLL(path)
        L.hifa4_status_string.restype = C.c_char_p
        L.hifa4_status_string.argtypes = [C.c_int]
        L.hifa4_get_counters.restype = None
        L.hifa4_quant_bytes.restype = C.c_size_t
        L.hifa4_quant_bytes.argtypes = [C.POINTER(_Shape), C.c_int, C.c_int]
        L.hifa4_attention_workspace_bytes.restype = C.c_size_t
        L.hifa4_attention_workspace_bytes.argtypes = [C.POINTER(_Shape), C.POINTER(_AttnParams)]
        L.hifa4_attention_raw_workspace_bytes.restype = C.c_size_t
        L.hifa4_attention_raw_workspace_bytes.argtypes = [C.POINTER(_Shape), C.POINTER(_AttnParams)]
        L.hifa4_smooth_calibrate.restype = C.c_int
        L.hifa4_smooth_calibrate.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                             C.c_int, C.POINTER(C.c_int), C.c_int, C.c_int, C.c_float,
                                             C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(_CalibStats),
                                             C.c_void_p]
        L.hifa4_smooth_calibrate_auto.restype = C.c_int
        L.hifa4_smooth_calibrate_auto.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                                  C.c_int, C.POINTER(C.c_int), C.c_int, C.c_void_p, C.c_void_p,
                                                  C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.hifa4_smooth_calibrate_static.restype = C.c_int
        L.hifa4_smooth_calibrate_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                                    C.c_int, C.POINTER(C.c_int), C.c_int, C.c_int, C.c_float,
                                                    C.c_void_p, C.c_void_p, C.POINTER(_CalibStats), C.c_void_p]
        L.hifa4_quantize_qkv.restype = C.c_int
        L.hifa4_quantize_qkv.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.POINTER(_QKV), C.c_void_p, C.c_void_p]
        L.hifa4_attention_fwd.restype = C.c_int
        L.hifa4_attention_fwd.argtypes = [C.POINTER(_Shape), C.POINTER(_QKV), C.POINTER(_AttnParams),
                                          C.c_void_p, C.c_void_p, C.POINTER(_Debug), C.c_void_p, C.c_void_p]
        L.hifa4_attention_fwd_qraw.restype = C.c_int
        L.hifa4_attention_fwd_qraw.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_void_p, C.POINTER(_QKV),
                                               C.POINTER(_AttnParams), C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_void_p]
        L.hifa4_f8qk_workspace_bytes.restype = C.c_size_t
        L.hifa4_f8qk_workspace_bytes.argtypes = [C.POINTER(_Shape)]
        L.hifa4_attention_fwd_f8qk.restype = C.c_int
        L.hifa4_attention_fwd_f8qk.argtypes = [C.POINTER(_Shape), C.POINTER(_QKV), C.POINTER(_AttnParams), C.c_void_p,
                                               C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.hifa4_selftest_wait_timeout.restype = C.c_int
        L.hifa4_selftest_wait_timeout.argtypes = [C.POINTER(_Shape), C.POINTER(_QKV), C.POINTER(_AttnParams),
                                                  C.c_void_p, C.c_void_p, C.c_void_p]
        L.hifa4_attention_fwd_stats.restype = C.c_int
        L.hifa4_attention_fwd_stats.argtypes = [C.POINTER(_Shape), C.POINTER(_QKV), C.POINTER(_AttnParams),
                                                C.c_void_p, C.c_void_p, C.POINTER(_MassStats), C.c_void_p,
                                                C.c_void_p]
        L.hifa4_attention_fwd_raw.restype = C.c_int
        L.hifa4_attention_fwd_raw.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_void_p, C.c_void_p,
                                              C.c_void_p, C.c_void_p, C.POINTER(_AttnParams), C.c_void_p,
                                              C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


STATIC_CALIB_MAX_FLOATS = 1 << 20

EXPORTS = ("hifa4_status_string", "hifa4_get_counters", "hifa4_smooth_calibrate",
           "hifa4_smooth_calibrate_static", "hifa4_smooth_calibrate_auto", "hifa4_quant_bytes",
           "hifa4_quantize_qkv", "hifa4_attention_workspace_bytes", "hifa4_attention_fwd",
           "hifa4_attention_fwd_stats", "hifa4_attention_raw_workspace_bytes", "hifa4_attention_fwd_raw",
           "hifa4_attention_fwd_qraw", "hifa4_f8qk_workspace_bytes", "hifa4_attention_fwd_f8qk",
           "hifa4_selftest_wait_timeout")


def status_string(status: int) -> str:
    return lib().hifa4_status_string(int(status)).decode()


def get_counters():
    arr = (C.c_ulonglong * 4)()
    lib().hifa4_get_counters(arr)
    return dict(calibrate=arr[0], quantize=arr[1], attention=arr[2], launches=arr[3])


def _check(rc: int, where: str):
    if rc != 0:
        raise Hifa4Error(rc, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _map_arr(q_to_kv):
    if q_to_kv is None:
        return None, None
    arr = (C.c_int * len(q_to_kv))(*[int(x) for x in q_to_kv])
    return arr, C.cast(arr, C.POINTER(C.c_int))


def _shape(B, Hq, Hkv, N, d, in_dtype, q_to_kv=None):
    keep, p = _map_arr(q_to_kv)
    s = _Shape(B, Hq, Hkv, N, d, p, in_dtype)
    s._keep = keep
    return s


def _params(causal, Bc, out_dtype, Br=128, normalizer=0, qmean=0, p_dtype=F16, softmax_scale=0.0):
    return _AttnParams(int(causal), Br, Bc, normalizer, qmean, p_dtype, out_dtype, float(softmax_scale))


@dataclass
class QuantizedQKV:
    """Device buffers of one hifa4_qkv (see include/hifa4.h for the layouts)."""
    B: int
    Hq: int
    Hkv: int
    N: int
    d: int
    in_dtype: int
    q_to_kv: object
    q_codes: torch.Tensor
    q_meta: torch.Tensor
    q_mma: torch.Tensor
    k_codes: torch.Tensor
    k_meta: torch.Tensor
    k_mma: torch.Tensor
    v_codes: torch.Tensor
    v_meta: torch.Tensor
    v_mma: torch.Tensor
    q_mu: torch.Tensor | None = None        # Q-Mean auxiliary: per-token mean of the smoothed query
    k_sum: torch.Tensor | None = None       # Q-Mean auxiliary: channel sum of the smoothed key

    def struct(self) -> _QKV:
        ptrs = [getattr(self, n).data_ptr() for n in ("q_codes", "q_meta", "q_mma", "k_codes",
                                                      "k_meta", "k_mma", "v_codes", "v_meta", "v_mma")]
        ptrs += [None if t is None else t.data_ptr() for t in (self.q_mu, self.k_sum)]
        return _QKV(*ptrs)


def quant_bytes(B, Hq, Hkv, N, d, in_dtype, which, part) -> int:
    s = _shape(B, Hq, Hkv, N, d, in_dtype)
    return int(lib().hifa4_quant_bytes(C.byref(s), which, part))


def alloc_qkv(B, Hq, Hkv, N, d, in_dtype, device, q_to_kv=None, qmean=False) -> QuantizedQKV:
    """Allocate the buffers with the sizes the library reports (qmean: also the two Q-Mean vectors)."""
    bufs = {}
    for w, name, H in ((Q, "q", Hq), (K, "k", Hkv), (V, "v", Hkv)):
        nb = [quant_bytes(B, Hq, Hkv, N, d, in_dtype, w, p) for p in (CODES, META, MMA)]
        if 0 in nb:
            raise Hifa4Error(2, "hifa4_quant_bytes")
        tok_axis = (w == V)
        lead = (B, H, d) if tok_axis else (B, H, N)
        ln = N if tok_axis else d
        bufs[name + "_codes"] = torch.empty(lead + (ln // 2,), dtype=torch.uint8, device=device)
        bufs[name + "_meta"] = torch.empty(lead + (ln // 64,), dtype=torch.int32, device=device)
        bufs[name + "_mma"] = torch.empty(lead + (ln,), dtype=torch.bfloat16, device=device)
        assert bufs[name + "_codes"].numel() == nb[0] and bufs[name + "_meta"].numel() * 4 == nb[1]
        assert bufs[name + "_mma"].numel() * 2 == nb[2]
    if qmean:
        assert quant_bytes(B, Hq, Hkv, N, d, in_dtype, Q, AUX) == B * Hq * N * 4
        bufs["q_mu"] = torch.empty((B, Hq, N), dtype=torch.float32, device=device)
        bufs["k_sum"] = torch.empty((B, Hkv, N), dtype=torch.float32, device=device)
    return QuantizedQKV(B, Hq, Hkv, N, d, in_dtype, q_to_kv, **bufs)


def smooth_calibrate(q_cal, k_cal, mode, alpha=0.0, q_to_kv=None, aggregator=AGG_RMS):
    """q_cal [S,Hq,Ncal,d], k_cal [S,Hkv,Ncal,d] device tensors -> (s, inv_s) [Hkv,d] float32.
    aggregator: AGG_RMS (the paper's choice), AGG_MEAN or AGG_P99 over the calibration samples."""
    assert q_cal.is_cuda and k_cal.is_cuda and q_cal.is_contiguous() and k_cal.is_contiguous()
    S, Hq, Ncal, d = q_cal.shape
    Hkv = k_cal.shape[1]
    dev = q_cal.device
    s = torch.empty((Hkv, d), dtype=torch.float32, device=dev)
    inv_s = torch.empty_like(s)
    ws = torch.empty((2, S, Hkv, d), dtype=torch.float32, device=dev)
    keep, mp = _map_arr(q_to_kv)
    stats = _CalibStats()
    rc = lib().hifa4_smooth_calibrate(_ptr(q_cal), _ptr(k_cal), S, Hq, Hkv, Ncal, d, mp, _DT[q_cal.dtype],
                                      int(mode) | int(aggregator), float(alpha), _ptr(s), _ptr(inv_s), _ptr(ws),
                                      C.byref(stats), _stream())
    _check(rc, "hifa4_smooth_calibrate")
    return s, inv_s


GATE_WS_BYTES = 32768 * 4 + 64


def smooth_calibrate_auto(q_cal, k_cal, q_to_kv=None):
    """Calibration with the applicability gate deciding the branch on the device.
    Returns (s, inv_s, stats) with stats a DEVICE float32 tensor [rho_K, T_K/Q, branch, alpha]."""
    assert q_cal.is_cuda and k_cal.is_cuda and q_cal.is_contiguous() and k_cal.is_contiguous()
    S, Hq, Ncal, d = q_cal.shape
    Hkv = k_cal.shape[1]
    dev = q_cal.device
    s = torch.empty((Hkv, d), dtype=torch.float32, device=dev)
    inv_s = torch.empty_like(s)
    ws = torch.empty((2, S, Hkv, d), dtype=torch.float32, device=dev)
    gate_ws = torch.empty(GATE_WS_BYTES // 8, dtype=torch.int64, device=dev)
    stats = torch.zeros(4, dtype=torch.float32, device=dev)
    keep, mp = _map_arr(q_to_kv)
    rc = lib().hifa4_smooth_calibrate_auto(_ptr(q_cal), _ptr(k_cal), S, Hq, Hkv, Ncal, d, mp, _DT[q_cal.dtype],
                                           _ptr(s), _ptr(inv_s), _ptr(ws), _ptr(gate_ws), _ptr(stats), _stream())
    _check(rc, "hifa4_smooth_calibrate_auto")
    return s, inv_s, stats


def smooth_calibrate_static(q_cal, k_cal, mode, alpha=0.0, q_to_kv=None, s=None, inv_s=None):
    """smooth_calibrate through the entry point that allocates nothing on the device: the scratch
    is the library's fixed array (2*S*Hkv*d <= STATIC_CALIB_MAX_FLOATS, else Hifa4Error with status
    3).  The caller may pass preallocated outputs s, inv_s [Hkv,d] float32; they are created here
    only for convenience when omitted (the C entry point itself never allocates)."""
    assert q_cal.is_cuda and k_cal.is_cuda and q_cal.is_contiguous() and k_cal.is_contiguous()
    S, Hq, Ncal, d = q_cal.shape
    Hkv = k_cal.shape[1]
    if s is None:
        s = torch.empty((Hkv, d), dtype=torch.float32, device=q_cal.device)
    if inv_s is None:
        inv_s = torch.empty_like(s)
    keep, mp = _map_arr(q_to_kv)
    stats = _CalibStats()
    rc = lib().hifa4_smooth_calibrate_static(_ptr(q_cal), _ptr(k_cal), S, Hq, Hkv, Ncal, d, mp,
                                             _DT[q_cal.dtype], int(mode), float(alpha), _ptr(s), _ptr(inv_s),
                                             C.byref(stats), _stream())
    _check(rc, "hifa4_smooth_calibrate_static")
    return s, inv_s


def quantize_qkv(q, k, v, s=None, inv_s=None, q_to_kv=None, out: QuantizedQKV | None = None,
                 d_status=None, qmean=False, Hq=None) -> QuantizedQKV:
    """Smooth-QK + HIF4 quantization of device tensors q [B,Hq,N,d], k, v [B,Hkv,N,d].
    qmean: also apply the Q-Mean auxiliary (the Q buffers then hold the mean-free Q_z).
    q = None: K and V only (for attention_fwd_qraw); Hq then names the number of query heads."""
    assert k.is_cuda and k.is_contiguous() and v.is_contiguous() and (q is None or q.is_contiguous())
    if q is None:
        assert Hq is not None and not qmean
        B, _, N, d = k.shape
    else:
        B, Hq, N, d = q.shape
    Hkv = k.shape[1]
    dt = _DT[k.dtype]
    if out is None:
        out = alloc_qkv(B, Hq, Hkv, N, d, dt, k.device, q_to_kv, qmean=qmean)
    sh = _shape(B, Hq, Hkv, N, d, dt, q_to_kv)
    st = out.struct()
    rc = lib().hifa4_quantize_qkv(C.byref(sh), _ptr(q), _ptr(k), _ptr(v), _ptr(s), _ptr(inv_s),
                                  C.byref(st), _ptr(d_status), _stream())
    _check(rc, "hifa4_quantize_qkv")
    return out


def attention_fwd(qkv: QuantizedQKV, causal: bool, Bc: int = 64, out_dtype=F32, out=None,
                  debug_blocks=None, d_status=None, softmax_scale=0.0, Br=128, qmean=False, normalizer=0,
                  p_dtype=F16):
    """Fused attention forward on quantized operands.  Returns out [B,Hq,N,d], or
    (out, dict(p_codes, p_step, l, m)) when debug_blocks (a list of (b, h, query block)) is given."""
    dev = qkv.q_mma.device
    sh = _shape(qkv.B, qkv.Hq, qkv.Hkv, qkv.N, qkv.d, qkv.in_dtype, qkv.q_to_kv)
    prm = _params(causal, Bc, out_dtype, Br=Br, softmax_scale=softmax_scale, qmean=int(qmean),
                  normalizer=int(normalizer), p_dtype=p_dtype)
    if out is None:
        out = torch.empty((qkv.B, qkv.Hq, qkv.N, qkv.d), dtype=_TORCH_DT[out_dtype], device=dev)
    st = qkv.struct()
    dbg_p, dump = None, None
    if debug_blocks:
        nb = len(debug_blocks)
        flat = (C.c_int * (3 * nb))(*[int(x) for t in debug_blocks for x in t])
        dump = dict(p_codes=torch.zeros((nb, 128, qkv.N), dtype=torch.uint8, device=dev),
                    p_step=torch.zeros((nb, 128, qkv.N // 4), dtype=torch.float32, device=dev),
                    l=torch.zeros((nb, 128), dtype=torch.float32, device=dev),
                    m=torch.zeros((nb, 128), dtype=torch.float32, device=dev))
        dbg = _Debug(nb, C.cast(flat, C.POINTER(C.c_int)), dump["p_codes"].data_ptr(),
                     dump["p_step"].data_ptr(), dump["l"].data_ptr(), dump["m"].data_ptr())
        dbg_p = C.byref(dbg)
    ws_bytes = int(lib().hifa4_attention_workspace_bytes(C.byref(sh), C.byref(prm)))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev) if ws_bytes else None
    rc = lib().hifa4_attention_fwd(C.byref(sh), C.byref(st), C.byref(prm), _ptr(out), _ptr(ws), dbg_p,
                                   _ptr(d_status), _stream())
    _check(rc, "hifa4_attention_fwd")
    return (out, dump) if debug_blocks else out


def attention_fwd_qraw(q, s, kv: QuantizedQKV, causal: bool, out_dtype=F32, out=None, d_status=None,
                       softmax_scale=0.0, p_dtype=F16):
    """attention_fwd whose kernel smooths and quantizes the raw q [B,Hq,N,d] itself (s: [Hkv,d] or None); kv holds
    the K and V images from quantize_qkv(None, k, v, ...).  Bc = 64, d = 64 or 128, no Q-Mean."""
    assert q.is_cuda and q.is_contiguous() and _DT[q.dtype] == kv.in_dtype
    sh = _shape(kv.B, kv.Hq, kv.Hkv, kv.N, kv.d, kv.in_dtype, kv.q_to_kv)
    assert tuple(q.shape) == (kv.B, kv.Hq, kv.N, kv.d)
    prm = _params(causal, 64, out_dtype, softmax_scale=softmax_scale, p_dtype=p_dtype)
    if out is None:
        out = torch.empty((kv.B, kv.Hq, kv.N, kv.d), dtype=_TORCH_DT[out_dtype], device=q.device)
    st = kv.struct()
    rc = lib().hifa4_attention_fwd_qraw(C.byref(sh), _ptr(q), _ptr(s), C.byref(st), C.byref(prm), _ptr(out), None,
                                        _ptr(d_status), _stream())
    _check(rc, "hifa4_attention_fwd_qraw")
    return out


def attention_fwd_f8qk(qkv: QuantizedQKV, causal: bool, out_dtype=F32, out=None, workspace=None, d_status=None,
                       softmax_scale=0.0):
    """attention_fwd with Q K^T issued as kind::f8f6f4 on E4M3 images (experiment; d = 128, Bc = 64)."""
    dev = qkv.k_mma.device
    sh = _shape(qkv.B, qkv.Hq, qkv.Hkv, qkv.N, qkv.d, qkv.in_dtype, qkv.q_to_kv)
    prm = _params(causal, 64, out_dtype, softmax_scale=softmax_scale)
    need = int(lib().hifa4_f8qk_workspace_bytes(C.byref(sh)))
    if need == 0:
        raise Hifa4Error(2, "hifa4_f8qk_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    if out is None:
        out = torch.empty((qkv.B, qkv.Hq, qkv.N, qkv.d), dtype=_TORCH_DT[out_dtype], device=dev)
    st = qkv.struct()
    rc = lib().hifa4_attention_fwd_f8qk(C.byref(sh), C.byref(st), C.byref(prm), _ptr(out), _ptr(workspace),
                                        C.c_size_t(workspace.numel()), _ptr(d_status), _stream())
    _check(rc, "hifa4_attention_fwd_f8qk")
    return out


def selftest_wait_timeout(qkv: QuantizedQKV, causal: bool, d_status, out=None):
    """Launches the self-test instantiation whose wait for P V runs out (see include/hifa4.h).  d_status: device
    int32 tensor (zero on entry); afterwards it holds HIFA4_ERR_TIMEOUT + 16 * 7.  Returns the (unwritten) out."""
    sh = _shape(qkv.B, qkv.Hq, qkv.Hkv, qkv.N, qkv.d, qkv.in_dtype, qkv.q_to_kv)
    prm = _params(causal, 64, F32)
    if out is None:
        out = torch.empty((qkv.B, qkv.Hq, qkv.N, qkv.d), dtype=torch.float32, device=qkv.q_mma.device)
    st = qkv.struct()
    rc = lib().hifa4_selftest_wait_timeout(C.byref(sh), C.byref(st), C.byref(prm), _ptr(out), _ptr(d_status), _stream())
    _check(rc, "hifa4_selftest_wait_timeout")
    return out


def attention_fwd_stats(qkv: QuantizedQKV, causal: bool, n_bins: int, lo: float, hi: float, Bc: int = 64,
                        out_dtype=F32, hist=None, d_status=None, softmax_scale=0.0, qmean=False, normalizer=0):
    """Attention forward that also adds to the histogram of the per-(row, key tile) mass error of P-hat.
    Returns (out, hist) with hist a device int64 tensor of n_bins + 2 counters (last two: below lo, at or above hi)."""
    dev = qkv.q_mma.device
    sh = _shape(qkv.B, qkv.Hq, qkv.Hkv, qkv.N, qkv.d, qkv.in_dtype, qkv.q_to_kv)
    prm = _params(causal, Bc, out_dtype, softmax_scale=softmax_scale, qmean=int(qmean), normalizer=int(normalizer))
    out = torch.empty((qkv.B, qkv.Hq, qkv.N, qkv.d), dtype=_TORCH_DT[out_dtype], device=dev)
    if hist is None:
        hist = torch.zeros(n_bins + 2, dtype=torch.int64, device=dev)
    st = qkv.struct()
    stats = _MassStats(hist.data_ptr(), int(n_bins), float(lo), float(hi))
    rc = lib().hifa4_attention_fwd_stats(C.byref(sh), C.byref(st), C.byref(prm), _ptr(out), None,
                                         C.byref(stats), _ptr(d_status), _stream())
    _check(rc, "hifa4_attention_fwd_stats")
    return out, hist


def attention_raw_workspace_bytes(B, Hq, Hkv, N, d, in_dtype, causal, Bc, out_dtype=F32, qmean=False) -> int:
    sh = _shape(B, Hq, Hkv, N, d, in_dtype)
    prm = _params(causal, Bc, out_dtype, qmean=int(qmean))
    return int(lib().hifa4_attention_raw_workspace_bytes(C.byref(sh), C.byref(prm)))


def attention_fwd_raw(q, k, v, s, inv_s, causal: bool, Bc: int = 64, out_dtype=F32, q_to_kv=None,
                      out=None, workspace=None, d_status=None, softmax_scale=0.0, qmean=False):
    """Algorithm 1 end to end on raw device tensors (quantize into the workspace, then attend)."""
    B, Hq, N, d = q.shape
    Hkv = k.shape[1]
    dt = _DT[q.dtype]
    sh = _shape(B, Hq, Hkv, N, d, dt, q_to_kv)
    prm = _params(causal, Bc, out_dtype, softmax_scale=softmax_scale, qmean=int(qmean))
    need = int(lib().hifa4_attention_raw_workspace_bytes(C.byref(sh), C.byref(prm)))
    if need == 0:
        raise Hifa4Error(2, "hifa4_attention_raw_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty((B, Hq, N, d), dtype=_TORCH_DT[out_dtype], device=q.device)
    rc = lib().hifa4_attention_fwd_raw(C.byref(sh), _ptr(q), _ptr(k), _ptr(v), _ptr(s), _ptr(inv_s),
                                       C.byref(prm), _ptr(out), _ptr(workspace),
                                       C.c_size_t(workspace.numel()), _ptr(d_status), _stream())
    _check(rc, "hifa4_attention_fwd_raw")
    return out
