#!/usr/bin/env python
"""Benchmark of the HiFA4 hot path on B200: one step = Smooth-QK + HIF4 quantization of Q/K/V
followed by the fused 4-bit-operand attention forward (Algorithm 1) over one batch of synthetic
prefill activations.  Prints ONE JSON line: metric, value (whole-job TFLOP/s over the timed steps),
roofline (attention launch against the measured BF16 tensor peak), quantize split, end-to-end figure
with host buffers, clocks sampled during the timed region, CPU-oracle baseline and context numbers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2] [--impl ours|reference]

N > 1 is launched by torch.distributed.run, one rank per GPU; every rank processes its own copy
of the workload (independent batches: the path has no exchange step), so scaling is weak.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_04302_b200 import synth  # noqa: E402

METRIC = "4-bit attention prefill TFLOPS on 1 B200; % of dense 4-bit tensor peak"
UNIT = "TFLOP/s"
NOMINAL = {"fp4": 9000.0, "fp8": 4500.0, "bf16": 2250.0}      # dense TFLOP/s, context only
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch, from the ncu capture
# summarised in profiles/attention_fwd_ws_C2.md (bytes per launch; None where not captured)
NCU_INSTR_PER_WARP_SCORE = {"attention_fwd_ws64_kernel<128>": 17.9}   # profiles/attention_fwd_ws64_C2.md
NCU_TRAFFIC_BYTES = {("C2-qwen3-8b-4k", 64): 68.70e6, ("C2-qwen3-8b-4k", 128): 67.14e6}


def attn_flops(cfg) -> float:
    f = 4.0 * cfg.B * cfg.Hq * cfg.N * cfg.N * cfg.d
    return f / 2 if cfg.causal else f


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the GPU is under load.

    nvidia-smi needs ~100 ms per sample, so a short timed region yields few samples; the sampler is
    started before warm-up and the benchmark keeps the GPU busy (same step function) until at least
    a few samples fall inside the marked window."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thr = index, [], None, None
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            return
        self.thr = threading.Thread(target=self._read, daemon=True)
        self.thr.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(",")]))

    def mark_begin(self):
        self.t0 = time.perf_counter()

    def mark_end(self):
        self.t1 = time.perf_counter()

    def samples_in_window(self):
        if self.t0 is None:
            return 0
        t1 = self.t1 if self.t1 is not None else time.perf_counter()
        return sum(1 for t, _ in self.rows if self.t0 <= t <= t1)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], None, set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for t, r in self.rows:
            if self.t0 is None or not (self.t0 <= t <= (self.t1 or t)):
                continue
            try:
                sm.append(float(r[0])); mx = float(r[1]); power.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm),
                "power_w_max": max(power) if power else None,
                "window": "timed steps plus identical untimed steps run until 8 samples were taken"}


def max_over_ranks(dist, ms: float, device) -> float:
    """Device time of the slowest rank (the job is as slow as its slowest rank)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(cfg, world: int, steps: int, total_ms: float) -> float:
    """Aggregate over all ranks: every rank processes its own copy of the workload (weak scaling)."""
    return world * attn_flops(cfg) * steps / (total_ms * 1e-3) / 1e12


def oracle_time(cfg, q, k, v, s, inv_s, heads):
    """Time the CPU oracle, as it stands, on whole heads of the workload (batch 0)."""
    from oracle import hifa4_oracle as orc
    import numpy as np
    dt = orc.F16 if cfg.dtype == "fp16" else orc.BF16
    idx = np.arange(cfg.N, dtype=np.int32)
    grp = cfg.Hq // cfg.Hkv
    t0 = time.perf_counter()
    for h in heads:
        g = h // grp
        orc.attention_rows(q[0, h], idx, k[0, g], v[0, g], None if s is None else s[g],
                           None if inv_s is None else inv_s[g], causal=cfg.causal, Bc=cfg.Bc, in_dtype=dt)
    return time.perf_counter() - t0, orc.num_threads()


def head_flops(cfg) -> float:
    f = 4.0 * cfg.N * cfg.N * cfg.d
    return f / 2 if cfg.causal else f


def host_inputs(cfg):
    q, k, v = synth.make_qkv(cfg)
    return q, k, v


def oracle_scales(cfg):
    """Smooth-QK factors from the oracle's own calibration (used by the CPU legs only)."""
    if cfg.smooth_mode == 0:
        return None, None
    from oracle import hifa4_oracle as orc
    small = synth.config(cfg.name.split("-")[0], cal_samples=min(cfg.cal_samples, 4), cal_tokens=min(cfg.cal_tokens, 256))
    qc, kc = synth.make_calibration(small)
    cal = orc.smooth_calibrate(qc.float().numpy(), kc.float().numpy(), cfg.smooth_mode)
    return cal["s"], cal["inv_s"]


def run_reference(args, cfg, rank):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step."""
    if rank != 0:
        return
    from oracle import hifa4_oracle as orc
    orc.build()
    q, k, v = (t.float().numpy() for t in host_inputs(cfg))
    s, inv_s = oracle_scales(cfg)
    t1, cores = oracle_time(cfg, q, k, v, s, inv_s, [0])
    # the whole run (warm-up included) gets about two minutes of CPU work, at most 8 s per step
    per_step = min(8.0, 120.0 / max(args.steps + args.warmup, 1))
    n_heads = max(1, min(cfg.Hq, int(per_step / max(t1, 1e-3))))
    heads = [int(i * cfg.Hq / n_heads) for i in range(n_heads)]
    for _ in range(args.warmup):
        oracle_time(cfg, q, k, v, s, inv_s, heads[:1])
    tot = 0.0
    for _ in range(args.steps):
        t, cores = oracle_time(cfg, q, k, v, s, inv_s, heads)
        tot += t
    val = n_heads * head_flops(cfg) * args.steps / tot / 1e12
    sample = f"{n_heads} of {cfg.B * cfg.Hq} (batch, head) slices of {cfg.name}, all {cfg.N} rows each, per step"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": cfg.name, "causal": cfg.causal, "Bc": cfg.Bc},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="C2", help="C2 (headline), C3, C4, C5 or C5@<N>")
    ap.add_argument("--noncausal", action="store_true")
    ap.add_argument("--Bc", type=int, default=0, help="key-tile width (default: the configuration's, 64)")
    ap.add_argument("--p-f32", action="store_true",
                    help="variant: quantize the FP32 exponential (not the method's FP16 P; for comparison only)")
    ap.add_argument("--qmean", action="store_true", help="with the Q-Mean auxiliary (Algorithm 1 lines 2 and 6)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the torch SDPA / N=8192 context numbers")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    name, _, n_over = args.workload.partition("@")
    over = {}
    if n_over:
        over["N"] = int(n_over)
    if args.noncausal:
        over["causal"] = False
    if args.Bc:
        over["Bc"] = args.Bc
    cfg = synth.config(name, **over)

    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return

    from paper_2607_04302_b200 import binding as hb
    hb.lib()                                  # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    # ---- inputs (resident in HBM) and offline calibration
    big = cfg.B * cfg.Hq * cfg.N * cfg.d > (1 << 28)
    if big:
        q, k, v = synth.make_qkv_device(cfg, dev)
        qh = kh = vh = None
    else:
        qh, kh, vh = host_inputs(cfg)
        q, k, v = qh.to(dev), kh.to(dev), vh.to(dev)
    s = inv_s = None
    if cfg.smooth_mode:
        qc, kc = synth.make_calibration(cfg, samples=min(cfg.cal_samples, 8), tokens=min(cfg.cal_tokens, 512))
        s, inv_s = hb.smooth_calibrate(qc.to(dev), kc.to(dev), cfg.smooth_mode)
    dt = hb._DT[q.dtype]
    qkv = hb.alloc_qkv(cfg.B, cfg.Hq, cfg.Hkv, cfg.N, cfg.d, dt, dev, qmean=args.qmean)
    out = torch.empty((cfg.B, cfg.Hq, cfg.N, cfg.d), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)       # > 126 MB of L2
    flush_rd = torch.zeros(64 << 20, dtype=torch.float32, device=dev)   # 256 MiB that are only read

    def flush_l2():
        # Write a buffer larger than L2, then read another one: the write evicts every line of the
        # previous step, the read pass pushes the dirty lines of the write out to HBM, so that their
        # write-back does not run inside the next step's timed region.
        flush.zero_()
        flush_rd.sum()

    def step(split=False):
        """One pass of the hot path.  split: record an event between the two launches (used only by the
        pass that attributes time to each kernel: the event keeps the attention grid, which is launched
        with programmatic stream serialization, from starting while the quantize grid drains)."""
        hb.quantize_qkv(q, k, v, s, inv_s, out=qkv, d_status=status, qmean=args.qmean)
        mid = None
        if split:
            mid = torch.cuda.Event(enable_timing=True)
            mid.record()
        hb.attention_fwd(qkv, cfg.causal, Bc=cfg.Bc, out_dtype=hb.F32, out=out, d_status=status,
                         p_dtype=hb.F32 if args.p_f32 else hb.F16, qmean=args.qmean)
        return mid

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    # spin-up (untimed, before the W warm-up steps): a fresh process on a fresh box starts with idle
    # clocks and unloaded modules; a quarter of a second of the same steps brings both up
    t_spin = time.perf_counter() + 0.25
    while time.perf_counter() < t_spin:
        for _ in range(10):
            flush_l2()
            step()
        torch.cuda.synchronize()
    for _ in range(args.warmup):
        flush_l2()
        step()
    barrier()
    assert int(status.item()) == 0, f"device status {int(status.item())}"

    c0 = hb.get_counters()["launches"]
    ev = []
    barrier()
    sampler.mark_begin()
    for _ in range(args.steps):
        flush_l2()                                                      # L2 flush, outside the events
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record()
        step()
        b.record()
        ev.append((a, b))
    barrier()
    launches = hb.get_counters()["launches"] - c0
    # second pass over the same steps with one more event per step, for the per-kernel durations
    ev_split = []
    for _ in range(args.steps):
        flush_l2()
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record()
        mid = step(split=True)
        b.record()
        ev_split.append((a, mid, b))
    barrier()
    # keep the same load on the GPU (untimed) until nvidia-smi has taken a few samples of it
    t_lim = time.perf_counter() + 3.0
    while sampler.proc is not None and sampler.samples_in_window() < 8 and time.perf_counter() < t_lim:
        for _ in range(20):
            flush_l2()
            step()
        torch.cuda.synchronize()
    sampler.mark_end()
    clocks = sampler.stop()
    step_ms = [a.elapsed_time(b) for a, b in ev]
    attn_ms = [m.elapsed_time(b) for _, m, b in ev_split]
    quant_ms = [a.elapsed_time(m) for a, m, _ in ev_split]
    split_step_ms = sum(a.elapsed_time(b) for a, _, b in ev_split) / len(ev_split)
    total_ms = sum(step_ms)
    total_ms = max_over_ranks(dist, total_ms, dev)
    assert int(status.item()) == 0, f"device status {int(status.item())}"

    # ---- end to end through the raw C-ABI entry point with host buffers (pinned), copies timed
    e2e = None
    if not big and not args.qmean:
        pq, pk, pv = qh.pin_memory(), kh.pin_memory(), vh.pin_memory()
        po = torch.empty(out.shape, dtype=torch.float32).pin_memory()
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        # One problem per (batch, KV head group): its Q/K/V slices are contiguous, so each goes through
        # hifa4_attention_fwd_raw on its own, and three streams keep the host-to-device copy of one
        # slice, the kernels of another and the device-to-host copy of a third in flight together.
        G = cfg.Hq // cfg.Hkv
        streams = [torch.cuda.Stream(device=dev) for _ in range(3)]
        ws_bytes = hb.attention_raw_workspace_bytes(1, G, 1, cfg.N, cfg.d, dt, cfg.causal, cfg.Bc)
        ws_s = [torch.empty(ws_bytes, dtype=torch.uint8, device=dev) for _ in streams]
        slices = [(bb, g) for bb in range(cfg.B) for g in range(cfg.Hkv)]

        def e2e_step():
            for i, (bb, g) in enumerate(slices):
                st_i = streams[i % len(streams)]
                hs = slice(g * G, (g + 1) * G)
                with torch.cuda.stream(st_i):
                    dq[bb:bb + 1, hs].copy_(pq[bb:bb + 1, hs], non_blocking=True)
                    dk[bb:bb + 1, g:g + 1].copy_(pk[bb:bb + 1, g:g + 1], non_blocking=True)
                    dv[bb:bb + 1, g:g + 1].copy_(pv[bb:bb + 1, g:g + 1], non_blocking=True)
                    hb.attention_fwd_raw(dq[bb:bb + 1, hs], dk[bb:bb + 1, g:g + 1], dv[bb:bb + 1, g:g + 1],
                                         None if s is None else s[g:g + 1], None if inv_s is None else inv_s[g:g + 1],
                                         cfg.causal, Bc=cfg.Bc, out=out[bb:bb + 1, hs], workspace=ws_s[i % len(streams)],
                                         d_status=status)
                    po[bb:bb + 1, hs].copy_(out[bb:bb + 1, hs], non_blocking=True)

        def fork():
            e = torch.cuda.Event()
            e.record()
            for st_i in streams:
                st_i.wait_event(e)

        def join():
            for st_i in streams:
                e = torch.cuda.Event()
                e.record(st_i)
                torch.cuda.current_stream().wait_event(e)

        fork()
        for _ in range(3):
            e2e_step()
        join()
        barrier()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        n_e2e = max(3, min(args.steps, 10))
        a.record()
        fork()
        for _ in range(n_e2e):
            e2e_step()
        join()
        b.record()
        barrier()
        assert int(status.item()) == 0, f"device status {int(status.item())}"
        assert torch.equal(po.to(dev), out), "end-to-end output differs from the device result"
        e_ms = a.elapsed_time(b)
        e_ms = max_over_ranks(dist, e_ms, dev)
        h2d = (pq.numel() + pk.numel() + pv.numel()) * pq.element_size()
        e2e = {"value": whole_job_tflops(cfg, world, n_e2e, e_ms), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": po.numel() * 4, "ms_per_step": e_ms / n_e2e,
               "how": f"hifa4_attention_fwd_raw per (batch, KV head group) slice, {len(slices)} slices over "
                      f"{len(streams)} streams, pinned host buffers"}

    # ---- context (not the product): torch SDPA in BF16 on the same inputs, and, for the headline
    # workload, its N = 8192 sibling (the target sentence names an 8K prefill, the configuration 4K)
    context = {}
    if rank == 0 and not args.no_context:
        import torch.nn.functional as F
        try:
            qb, kb, vb = (t.to(torch.bfloat16) for t in (q, k, v))
            for _ in range(3):
                F.scaled_dot_product_attention(qb, kb, vb, is_causal=cfg.causal, enable_gqa=True)
            torch.cuda.synchronize()
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(10):
                F.scaled_dot_product_attention(qb, kb, vb, is_causal=cfg.causal, enable_gqa=True)
            b.record()
            torch.cuda.synchronize()
            context["torch_sdpa_bf16_tflops"] = attn_flops(cfg) * 10 / (a.elapsed_time(b) * 1e-3) / 1e12
        except Exception as e:                                         # context only: never fail the bench on it
            context["torch_sdpa_bf16_tflops"] = None
            context["torch_sdpa_error"] = str(e)[:120]
        if cfg.name == synth.CONFIGS["C2"].name and cfg.N == 4096:
            c8 = synth.config("C2", N=8192, Bc=cfg.Bc, causal=cfg.causal)
            q8, k8, v8 = synth.make_qkv_device(c8, dev)
            qkv8 = hb.alloc_qkv(c8.B, c8.Hq, c8.Hkv, c8.N, c8.d, dt, dev)
            out8 = torch.empty((c8.B, c8.Hq, c8.N, c8.d), dtype=torch.float32, device=dev)

            def step8():
                hb.quantize_qkv(q8, k8, v8, s, inv_s, out=qkv8, d_status=status)
                hb.attention_fwd(qkv8, c8.causal, Bc=c8.Bc, out_dtype=hb.F32, out=out8, d_status=status)

            for _ in range(3):
                flush_l2(); step8()
            torch.cuda.synchronize()
            ms8 = 0.0
            for _ in range(20):
                flush_l2()
                a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
                a.record(); step8(); b.record()
                torch.cuda.synchronize()
                ms8 += a.elapsed_time(b)
            context["C2_at_N8192_step_tflops"] = attn_flops(c8) * 20 / (ms8 * 1e-3) / 1e12
            del q8, k8, v8, qkv8, out8
        assert int(status.item()) == 0

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    fl = attn_flops(cfg)
    value = whole_job_tflops(cfg, world, args.steps, total_ms)
    attn_avg_ms = sum(attn_ms) / len(attn_ms)
    achieved = fl / (attn_avg_ms * 1e-3) / 1e12
    if cfg.Bc == 64 and cfg.d in (128, 256):
        kern = f"attention_fwd_ws64_kernel<{cfg.d}>"
    elif cfg.Bc == 128 and cfg.d == 128:
        kern = "attention_fwd_ws_kernel<4>"
    else:
        kern = f"attention_fwd_kernel<{cfg.d},{cfg.Bc}>"
    roofline = {"bound": "tensor", "kernel": kern, "achieved": achieved, "peak": peaks["bf16"],
                "unit": "TFLOP/s", "frac": achieved / peaks["bf16"],
                "traffic": NCU_TRAFFIC_BYTES.get((cfg.name, cfg.Bc) if cfg.causal and not args.p_f32 else None),
                "peak_source": f"{peaks['source']} cuBLAS bf16 burst (the MMA kind issued is kind::f16 on BF16 images)",
                "avg_launch_ms": attn_avg_ms,
                "timed_in": "a second pass of the same steps with one event between the two launches "
                            f"({split_step_ms:.4f} ms per step there)",
                "frac_of_nominal": {k_: achieved / v_ for k_, v_ in NOMINAL.items()}}
    # The binding resource of the attention kernel is the issue rate of its softmax/quantizer warps, not
    # the tensor pipe: scores per second against (SMs x 4 schedulers x clock) warp-instructions per second
    # divided by the warp-instructions the kernel executes per 32 scores (ncu opcode counters, profiles/).
    n_scores = cfg.B * cfg.Hq * sum(min(cfg.N, ((qb * 128 + 127) // cfg.Bc + 1) * cfg.Bc) if cfg.causal else cfg.N
                                    for qb in range((cfg.N + 127) // 128)) * 128
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    sm_hz = (clocks.get("sm_mhz") or 1965.0) * 1e6
    instr_per_warp_score = NCU_INSTR_PER_WARP_SCORE.get(kern)
    roofline_alu = None
    if instr_per_warp_score:
        peak_scores = sm_count * 4 * sm_hz * 32 / instr_per_warp_score
        ach_scores = n_scores / (attn_avg_ms * 1e-3)
        roofline_alu = {"bound": "alu", "kernel": kern, "achieved": ach_scores / 1e9, "peak": peak_scores / 1e9,
                        "unit": "Gscore/s", "frac": ach_scores / peak_scores,
                        "instr_per_warp_score": instr_per_warp_score,
                        "peak_source": f"{sm_count} SMs x 4 schedulers x {sm_hz / 1e6:.0f} MHz (sampled) x 32 lanes / "
                                       "executed warp instructions per warp-score (ncu)"}
    q_bytes = sum(t.numel() for t in (q, k, v)) * (2 + 0.5625)
    quant = {"avg_ms": sum(quant_ms) / len(quant_ms), "algorithmic_gbs": q_bytes / (sum(quant_ms) / len(quant_ms) * 1e-3) / 1e9,
             "hbm_peak_gbs": peaks["hbm"]}

    cpu = None
    if not args.no_cpu_baseline and not big:
        from oracle import hifa4_oracle as orc
        orc.build()
        qn, kn, vn = (t.float().numpy() for t in (qh, kh, vh))
        sn = None if s is None else s.cpu().numpy()
        isn = None if inv_s is None else inv_s.cpu().numpy()
        t1, cores = oracle_time(cfg, qn, kn, vn, sn, isn, [0])
        n_heads = max(1, min(cfg.Hq - 1, int(12.0 / max(t1, 1e-3))))
        heads = [1 + int(i * (cfg.Hq - 1) / n_heads) for i in range(n_heads)]
        t, cores = oracle_time(cfg, qn, kn, vn, sn, isn, heads)
        cpu = {"value": n_heads * head_flops(cfg) / t / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"{n_heads} of {cfg.B * cfg.Hq} (batch, head) slices of {cfg.name}, all {cfg.N} rows each, "
                         f"{t:.1f} s"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "N": cfg.N, "d": cfg.d,
                       "causal": cfg.causal, "Br": 128, "Bc": cfg.Bc, "in_dtype": cfg.dtype, "out_dtype": "f32",
                       "p_dtype": "f32 (variant)" if args.p_f32 else "f16", "qmean": bool(args.qmean),
                       "smooth_mode": cfg.smooth_mode, "step": "hifa4_quantize_qkv + hifa4_attention_fwd",
                       "l2": "flushed between steps (256 MiB write, then a 256 MiB read that drains the dirty lines), outside the per-step events",
                       "parallelism": f"replicated batches x{world}"},
            "frac_of_nominal_peak": {k_: value / world / v_ for k_, v_ in NOMINAL.items()},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
            "roofline_alu": roofline_alu, "quantize": quant, "cpu_baseline": cpu, "context": context}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
