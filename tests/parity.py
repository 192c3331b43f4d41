"""Shared parity harness: runs the CUDA path through the C-ABI binding and the CPU oracle on the
same seeded inputs and compares them.  Used by the -m gpu tests."""
from __future__ import annotations

import numpy as np
import torch

from oracle import hifa4_oracle as orc
from paper_2607_04302_b200 import binding as hb
from paper_2607_04302_b200 import synth

# the benchmark spec tolerances
P_MISMATCH_MAX = 1e-4          # fraction of P-hat elements whose code or step differs
OUT_MAX_ABS = 1e-2             # x output RMS, on rows whose P-hat matches the oracle exactly
OUT_MEAN_ABS = 1e-3            # x output RMS, over all compared rows


def np32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def unpack(codes: np.ndarray) -> np.ndarray:
    nib = np.empty(codes.shape[:-1] + (codes.shape[-1] * 2,), np.uint8)
    nib[..., 0::2] = codes & 15
    nib[..., 1::2] = codes >> 4
    return nib


def calibrate(cfg, device):
    """Library calibration on the config's calibration set -> (s, inv_s) device tensors or (None, None)."""
    if cfg.smooth_mode == 0:
        return None, None
    qc, kc = synth.make_calibration(cfg)
    return hb.smooth_calibrate(qc.to(device), kc.to(device), cfg.smooth_mode)


def check_quantized(cfg, q, k, v, s, inv_s, qkv, qmean=False):
    """Bit-exact comparison of codes, metadata and the BF16 operand image with the oracle (and of
    the two Q-Mean vectors when qmean is set)."""
    dt = orc.F16 if cfg.dtype == "fp16" else orc.BF16
    s_np = None if s is None else np32(s)
    is_np = None if inv_s is None else np32(inv_s)
    Hq, Hkv = cfg.Hq, cfg.Hkv
    grp = Hq // Hkv
    for name, x, sc, tok in (("q", q, None if s_np is None else np.repeat(s_np, grp, 0), False),
                             ("k", k, is_np, False), ("v", v, None, True)):
        xn = np32(x)
        codes_l, meta_l, deq_l = [], [], []
        aux_l = []
        for h in range(xn.shape[1]):
            if qmean and name == "q":
                c, m, dq, mu = orc.qmean_quantize(xn[:, h], None if sc is None else sc[h], dt)
                aux_l.append(mu)
            else:
                c, m, dq = orc.smooth_quantize(xn[:, h], None if sc is None else sc[h], dt, axis_tokens=tok)
                if qmean and name == "k":
                    aux_l.append(orc.ksum_rows(xn[:, h], None if sc is None else sc[h], dt))
            codes_l.append(c); meta_l.append(m); deq_l.append(dq)
        if aux_l:
            g_aux = getattr(qkv, "q_mu" if name == "q" else "k_sum").cpu().numpy().astype(np.float64)
            assert np.array_equal(g_aux, np.stack(aux_l, 1)), f"{name} Q-Mean vector differs"
        codes, meta, deq = (np.stack(a, 1) for a in (codes_l, meta_l, deq_l))
        g_codes = getattr(qkv, name + "_codes").cpu().numpy()
        g_meta = getattr(qkv, name + "_meta").cpu().numpy().view(np.uint32)
        g_img = np32(getattr(qkv, name + "_mma")).astype(np.float64)
        assert np.array_equal(g_meta, meta), f"{name} metadata differs in {np.count_nonzero(g_meta != meta)} groups"
        assert np.array_equal(g_codes, codes), f"{name} codes differ in {np.count_nonzero(g_codes != codes)} bytes"
        assert np.array_equal(g_img, deq), f"{name} operand image differs"


def run_case(cfg, device="cuda:0", blocks=None, out_dtype=hb.F32, check_quant=True, rows_per_block=None,
             qkv_host=None, qmean=False, normalizer=0, p_dtype=hb.F16, qkv_dev=None):
    """Full path on the GPU + oracle on the requested 128-row query blocks.

    blocks: list of (b, h, query_block); default: every block (small cases only).
    qkv_dev: inputs already on the device (sizes too large to draw on the host); only the sampled
    query rows and their K/V head are then copied to the host for the oracle (no check_quant).
    Every attention launch is made twice: once with the P-hat dump (the instantiation the oracle
    comparison reads) and once without it (the instantiation callers and the benchmark run); the two
    outputs must be bit-identical, which puts the plain instantiation under the same comparison.
    Returns a dict of measured discrepancies (the bars are asserted by the callers)."""
    if qkv_dev is not None:
        assert not check_quant, "check_quant needs host inputs"
        q, k, v = qkv_dev
    else:
        q, k, v = qkv_host if qkv_host is not None else synth.make_qkv(cfg)
    s, inv_s = calibrate(cfg, device)
    qd, kd, vd = q.to(device), k.to(device), v.to(device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    qkv = hb.quantize_qkv(qd, kd, vd, s, inv_s, d_status=status, qmean=qmean)
    if check_quant:
        check_quantized(cfg, q, k, v, s, inv_s, qkv, qmean=qmean)
    n_qb = (cfg.N + 127) // 128
    if blocks is None:
        blocks = [(b, h, t) for b in range(cfg.B) for h in range(cfg.Hq) for t in range(n_qb)]
    res = dict(p_total=0, p_mismatch=0, rows=0, rows_clean=0, max_abs_all=0.0, max_abs_clean=0.0,
               sum_abs=0.0, n_out=0, sq_sum=0.0, flips=[])
    out_full = None
    for i0 in range(0, len(blocks), hb.MAX_DEBUG_BLOCKS):
        chunk = blocks[i0:i0 + hb.MAX_DEBUG_BLOCKS]
        out, dump = hb.attention_fwd(qkv, cfg.causal, Bc=cfg.Bc, out_dtype=out_dtype, debug_blocks=chunk,
                                     d_status=status, qmean=qmean, normalizer=normalizer, p_dtype=p_dtype)
        if i0 == 0:
            plain = hb.attention_fwd(qkv, cfg.causal, Bc=cfg.Bc, out_dtype=out_dtype, d_status=status, qmean=qmean,
                                     normalizer=normalizer, p_dtype=p_dtype)
            assert torch.equal(plain, out), "output without the P-hat dump differs from the dumped launch"
            del plain
        torch.cuda.synchronize()
        assert int(status.item()) == 0, f"device status {int(status.item())}"
        out_full = out
        pc, ps = dump["p_codes"].cpu().numpy(), dump["p_step"].cpu().numpy()
        dt = orc.F16 if cfg.dtype == "fp16" else orc.BF16
        s_np = None if s is None else np32(s)
        is_np = None if inv_s is None else np32(inv_s)
        kv_cache = {}
        for bi, (b, h, t) in enumerate(chunk):
            g = h // (cfg.Hq // cfg.Hkv)
            r0, r1 = t * 128, min(t * 128 + 128, cfg.N)
            idx = np.arange(r0, r1, dtype=np.int32)
            if rows_per_block is not None and rows_per_block < len(idx):
                idx = idx[np.linspace(0, len(idx) - 1, rows_per_block).astype(int)]
            if (b, g) not in kv_cache:
                kv_cache.clear()                               # one K/V head on the host at a time
                kv_cache[(b, g)] = (np32(k[b, g]), np32(v[b, g]))
            kn_bg, vn_bg = kv_cache[(b, g)]
            q_rows = np32(q[b, h][torch.as_tensor(idx, dtype=torch.long, device=q.device)])
            o_ref, d = orc.attention_rows(q_rows, idx, kn_bg, vn_bg,
                                          None if s_np is None else s_np[g], None if is_np is None else is_np[g],
                                          causal=cfg.causal, Bc=cfg.Bc, in_dtype=dt, out_dtype=out_dtype,
                                          qmean=int(qmean), normalizer=normalizer, p_dtype=p_dtype, dumps=True)
            loc = idx - r0
            code_ne = pc[bi, loc] != d["p_codes"]
            step_ne = np.repeat(ps[bi, loc] != d["p_step"], 4, axis=1)
            bad = code_ne | step_ne
            res["p_total"] += bad.size
            res["p_mismatch"] += int(bad.sum())
            err = np.abs(np32(out[b, h][torch.as_tensor(idx, dtype=torch.long, device=out.device)]).astype(np.float64) - o_ref)
            clean = ~bad.any(1)
            res["rows"] += len(idx)
            res["rows_clean"] += int(clean.sum())
            res["max_abs_all"] = max(res["max_abs_all"], float(err.max()))
            if clean.any():
                res["max_abs_clean"] = max(res["max_abs_clean"], float(err[clean].max()))
            res["sum_abs"] += float(err.sum())
            res["n_out"] += err.size
            res["sq_sum"] += float((o_ref ** 2).sum())
            for r in np.nonzero(~clean)[0][:4]:
                j = int(np.nonzero(bad[r])[0][0])
                res["flips"].append((b, h, int(idx[r]), j, int(pc[bi, loc[r], j]), int(d["p_codes"][r, j]),
                                     float(d["p_raw"][r, j]), float(d["p_step"][r, j // 4])))
            # the final normalizer (the rescaled row sum of P-hat, or of P when mismatched) against the oracle's
            l_gpu = dump["l"][bi, loc].cpu().numpy().astype(np.float64)
            assert np.allclose(l_gpu[clean], d["l"][clean], rtol=2e-3), "normalizer differs"
    rms = np.sqrt(res["sq_sum"] / max(res["n_out"], 1))
    res["rms"] = rms
    res["p_mismatch_frac"] = res["p_mismatch"] / max(res["p_total"], 1)
    res["max_abs_all_rel"] = res["max_abs_all"] / rms
    res["max_abs_clean_rel"] = res["max_abs_clean"] / rms
    res["mean_abs_rel"] = res["sum_abs"] / max(res["n_out"], 1) / rms
    res["out"] = out_full
    return res


def assert_within_bars(res, what=""):
    msg = (f"{what}: P-hat mismatch {res['p_mismatch_frac']:.2e}, max-abs(clean rows) "
           f"{res['max_abs_clean_rel']:.2e} x RMS, max-abs(all) {res['max_abs_all_rel']:.2e} x RMS, "
           f"mean-abs {res['mean_abs_rel']:.2e} x RMS, flips {res['flips'][:3]}")
    assert res["p_mismatch_frac"] <= P_MISMATCH_MAX, msg
    assert res["max_abs_clean_rel"] <= OUT_MAX_ABS, msg
    assert res["mean_abs_rel"] <= OUT_MEAN_ABS, msg
    return msg
