"""GPU parity of the fused attention forward against the CPU oracle (Algorithm 1), through the
C ABI: P-hat codes/steps, normalizer and output, on small cases element by element and on sampled
query blocks of the full-size configurations."""
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


def test_tiny_config(hb, par):
    """Configuration 1: B=1, H=1, N=128, d=128, fp16, x20 K channels, 64x64 tiles, non-causal."""
    cfg = synth.config("C1")
    res = par.run_case(cfg, DEV)
    print(par.assert_within_bars(res, "C1"))
    assert res["rows"] == 128


SMALL = {
    "d128-bc128-causal-gqa": synth.config("C2", N=512, Hq=4, Hkv=2, Bc=128, cal_samples=4, cal_tokens=128),
    "d128-bc64-causal-gqa": synth.config("C2", N=512, Hq=4, Hkv=2, cal_samples=4, cal_tokens=128),
    "d128-bc64-causal": synth.config("C2", N=384, Hq=2, Hkv=1, Bc=64, cal_samples=4, cal_tokens=128),
    "d128-bc128-noncausal": synth.config("C2", N=256, Hq=2, Hkv=2, Bc=128, causal=False, cal_samples=4, cal_tokens=128),
    "d128-ragged-n": synth.config("C2", N=320, Hq=2, Hkv=1, Bc=128, cal_samples=4, cal_tokens=128),
    "d128-bc64-ragged-n": synth.config("C2", N=320, Hq=2, Hkv=1, cal_samples=4, cal_tokens=128),
    "d128-ragged-noncausal": synth.config("C3", N=192, Hq=1, Hkv=1, Bc=128, causal=False),
    "d128-bc64-noncausal": synth.config("C3", N=192, Hq=1, Hkv=1, causal=False),
    "d64-bc128": synth.config("C3", N=256, Hq=2, Hkv=1, d=64, Bc=128),
    "d64-bc64-fp16": synth.config("C3", N=256, Hq=2, Hkv=1, d=64, Bc=64, dtype="fp16"),
    "d64-bc64-causal-gqa-ragged": synth.config("C2", N=448, Hq=4, Hkv=2, d=64, cal_samples=3, cal_tokens=64),
    "d256-bc64-mild": synth.config("C4", N=256, Hq=2, Hkv=1, Bc=64, cal_samples=3, cal_tokens=64),
    "batch2": synth.config("C5", B=2, N=256, Hq=4, Hkv=2, Bc=128, cal_samples=2, cal_tokens=64),
    "batch2-bc64": synth.config("C5", B=2, N=256, Hq=4, Hkv=2, cal_samples=2, cal_tokens=64),
    "n64": synth.config("C3", N=64, Hq=1, Hkv=1, Bc=128),
    "n64-bc64": synth.config("C3", N=64, Hq=1, Hkv=1),
}


@pytest.mark.parametrize("name", list(SMALL))
def test_small_cases_elementwise(hb, par, name):
    cfg = SMALL[name]
    res = par.run_case(cfg, DEV)
    print(par.assert_within_bars(res, name))
    assert res["rows"] == cfg.B * cfg.Hq * cfg.N


def test_output_dtypes_and_determinism(hb, par):
    cfg = SMALL["d128-bc128-causal-gqa"]
    q, k, v = synth.make_qkv(cfg)
    s, inv_s = par.calibrate(cfg, DEV)
    qkv = hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s)
    o32 = hb.attention_fwd(qkv, True, Bc=128, out_dtype=hb.F32)
    o32b = hb.attention_fwd(qkv, True, Bc=128, out_dtype=hb.F32)
    assert torch.equal(o32, o32b)                              # no atomics: bit-identical reruns
    o16 = hb.attention_fwd(qkv, True, Bc=128, out_dtype=hb.F16)
    ob16 = hb.attention_fwd(qkv, True, Bc=128, out_dtype=hb.BF16)
    assert torch.equal(o16, o32.to(torch.float16)) and torch.equal(ob16, o32.to(torch.bfloat16))
    # Bc is part of the result; Br is not exposed beyond 128
    o64 = hb.attention_fwd(qkv, True, Bc=64, out_dtype=hb.F32)
    assert not torch.equal(o64, o32)
    assert torch.isfinite(o32).all()


def test_raw_entry_point_equals_two_step_path(hb, par):
    cfg = SMALL["d128-bc128-causal-gqa"]
    q, k, v = (t.to(DEV) for t in synth.make_qkv(cfg))
    s, inv_s = par.calibrate(cfg, DEV)
    a = hb.attention_fwd(hb.quantize_qkv(q, k, v, s, inv_s), True, Bc=128)
    b = hb.attention_fwd_raw(q, k, v, s, inv_s, True, Bc=128)
    assert torch.equal(a, b)
    with pytest.raises(hb.Hifa4Error):                          # undersized workspace is refused
        hb.attention_fwd_raw(q, k, v, s, inv_s, True, Bc=128,
                             workspace=torch.empty(1024, dtype=torch.uint8, device=DEV))


def test_unsupported_flags_are_refused(hb, par):
    cfg = SMALL["n64"]
    q, k, v = (t.to(DEV) for t in synth.make_qkv(cfg))
    qkv = hb.quantize_qkv(q, k, v)
    with pytest.raises(hb.Hifa4Error):
        hb.attention_fwd(qkv, True, Bc=96)
    with pytest.raises(hb.Hifa4Error):
        hb.attention_fwd(qkv, True, Bc=128, Br=64)


def _sampled_blocks(cfg, heads):
    n_qb = cfg.N // 128
    return [(b, h, t) for b in (0, cfg.B - 1) for h in heads for t in sorted({0, n_qb // 2, n_qb - 1})]


@pytest.mark.parametrize("name,Bc", [("C2", 64), ("C3", 64), ("C4", 64), ("C2", 128), ("C3", 128)])
def test_full_size_sampled_blocks(hb, par, name, Bc):
    """Full-size configurations in the launch configuration the benchmark times (Bc = 64) and with
    the 128-key tiles of the persistent kernel; the oracle evaluates sampled rows of the first, a
    middle and the last query block of two heads."""
    cfg = synth.config(name, cal_samples=4, cal_tokens=256, Bc=Bc)
    blocks = sorted(set(_sampled_blocks(cfg, (0, cfg.Hq - 1))))
    res = par.run_case(cfg, DEV, blocks=blocks, check_quant=(name in ("C2", "C4") and Bc == 64), rows_per_block=24)
    print(par.assert_within_bars(res, f"{name} Bc={Bc}"))
    out = res["out"]
    assert torch.isfinite(out).all()


@pytest.mark.parametrize("causal", [True, False])
def test_sweep_point_sampled(hb, par, causal):
    """Configuration 5 at N = 2048 (B = 4), causal and non-causal."""
    cfg = synth.config("C5", N=2048, causal=causal, cal_samples=2, cal_tokens=256)
    blocks = [(0, 0, 0), (3, 31, 15), (1, 17, 7)]
    res = par.run_case(cfg, DEV, blocks=blocks, check_quant=False, rows_per_block=16)
    print(par.assert_within_bars(res, f"C5 N=2048 causal={causal}"))


@pytest.mark.parametrize("Bc", [64, 128])
def test_sweep_point_8k_sampled(hb, par, Bc):
    """Configuration 5 at N = 8192 (B = 4, causal): 8192 CTAs of the 64-key kernel, 8192 work items of
    the persistent 128-key kernel."""
    cfg = synth.config("C5", N=8192, Bc=Bc, cal_samples=2, cal_tokens=256)
    blocks = [(0, 0, 0), (3, 31, 63), (2, 9, 31), (1, 30, 1)]
    res = par.run_case(cfg, DEV, blocks=blocks, check_quant=False, rows_per_block=12)
    print(par.assert_within_bars(res, "C5 N=8192 causal"))


@pytest.mark.parametrize("N,causal", [(8192, False), (16384, True), (16384, False), (32768, True), (32768, False)])
def test_sweep_top_sampled(hb, par, N, causal):
    """Configuration 5 at the top of its sweep with the real B = 4, Hq = 32, Hkv = 8, causal and non-causal.
    The inputs are drawn on the device (the recipe of the configuration, device generator); only the
    sampled query rows and the K/V head they attend to are copied to the host for the oracle."""
    cfg = synth.config("C5", N=N, causal=causal, cal_samples=2, cal_tokens=256)
    qkv_dev = synth.make_qkv_device(cfg, DEV)
    n_qb = N // 128
    blocks = [(0, 0, 0), (1, 13, n_qb // 2 + 1), (3, 31, n_qb - 1), (2, 22, 1)]
    res = par.run_case(cfg, DEV, blocks=blocks, check_quant=False, rows_per_block=4, qkv_dev=qkv_dev)
    print(par.assert_within_bars(res, f"C5 N={N} causal={causal}"))
    assert res["rows"] == 16 and torch.isfinite(res["out"]).all()


def test_long_sequence_head_major_order_sampled(hb, par):
    """B = 4, Hkv = 8, N = 16384: the K/V images (268 MB) exceed L2, so the 64-key kernel launches its CTAs
    head by head instead of query block by query block; sampled rows against the oracle."""
    cfg = synth.config("C5", N=16384, Hq=8, Hkv=8, cal_samples=2, cal_tokens=256)
    blocks = [(0, 0, 0), (3, 7, 127), (1, 3, 64), (2, 5, 1)]
    res = par.run_case(cfg, DEV, blocks=blocks, check_quant=False, rows_per_block=6)
    print(par.assert_within_bars(res, "C5-like N=16384 head-major"))


@pytest.mark.parametrize("causal,Bc", [(True, 64), (False, 64), (True, 128)])
def test_largest_sequence_properties(hb, causal, Bc):
    """N = 32768 (the top of the sequence sweep), too large for the oracle: properties that hold at any
    size.  With V constant per channel the output must be that constant's HIF4 value times
    rowsum(P-hat) / FP16(rowsum(P-hat)): numerator and normalizer come from the same P-hat
    (P-Reordering through the ones column), whatever the scores are.  Reruns are bit-identical."""
    B, Hq, Hkv, N, d = 1, 4, 2, 32768, 128
    gen = torch.Generator(device=DEV).manual_seed(7)
    q = torch.randn((B, Hq, N, d), generator=gen, device=DEV).to(torch.bfloat16)
    k = torch.randn((B, Hkv, N, d), generator=gen, device=DEV).to(torch.bfloat16)
    consts = torch.linspace(-3.0, 3.0, d, device=DEV).to(torch.bfloat16)
    v = consts.expand(B, Hkv, N, d).contiguous()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    qkv = hb.quantize_qkv(q, k, v, d_status=status)
    out = hb.attention_fwd(qkv, causal, Bc=Bc, d_status=status)
    out2 = hb.attention_fwd(qkv, causal, Bc=Bc, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out, out2) and torch.isfinite(out).all()
    vhat = qkv.v_mma[0, 0, :, 0].float()                       # V-hat of each channel (constant along tokens)
    assert torch.equal(qkv.v_mma[0, 0], vhat[:, None].expand(d, N).to(torch.bfloat16))
    rel = (out / vhat[None, None, None, :].clamp_min(-1e30) - 1.0)
    rel = rel[..., vhat != 0]
    assert rel.abs().max().item() <= 2.0 ** -10                # only the FP16 rounding of the normalizer is left


QMEAN = {
    "qmean-d128-causal-gqa": synth.config("C2", N=512, Hq=4, Hkv=2, Bc=128, cal_samples=4, cal_tokens=128),
    "qmean-d128-bc64-causal-gqa": synth.config("C2", N=512, Hq=4, Hkv=2, cal_samples=4, cal_tokens=128),
    "qmean-d128-ragged-noncausal": synth.config("C2", N=320, Hq=2, Hkv=1, Bc=128, causal=False, cal_samples=4, cal_tokens=128),
    "qmean-tiny-64x64-fp16": synth.config("C1"),
    "qmean-d256-bc64": synth.config("C4", N=256, Hq=2, Hkv=1, Bc=64, cal_samples=3, cal_tokens=64),
}


@pytest.mark.parametrize("name", list(QMEAN))
def test_qmean_auxiliary(hb, par, name):
    """Algorithm 1 with lines 2 and 6 (Q-Mean): Q_z codes, mu, k_sum bit-exact; P-hat and output in the bars.
    The inputs get a per-token offset on Q so that the mean is not negligible."""
    cfg = QMEAN[name]
    q, k, v = synth.make_qkv(cfg)
    q = (q.float() + 0.75).to(q.dtype)
    res = par.run_case(cfg, DEV, qkv_host=(q, k, v), qmean=True)
    print(par.assert_within_bars(res, name))
    # the correction matters on these inputs: without it the output differs
    s, inv_s = par.calibrate(cfg, DEV)
    a = hb.attention_fwd(hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s, qmean=True), cfg.causal, Bc=cfg.Bc, qmean=True)
    b = hb.attention_fwd(hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s), cfg.causal, Bc=cfg.Bc)
    assert not torch.equal(a, b)
    c = hb.attention_fwd_raw(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s, cfg.causal, Bc=cfg.Bc, qmean=True)
    assert torch.equal(a, c)


def test_qmean_full_size_sampled(hb, par):
    """Configuration 5 with every HiFA4 component on (Smooth-QK, Q-Mean, P-Reordering), N = 4096, B = 4."""
    cfg = synth.config("C5", N=4096, cal_samples=2, cal_tokens=256)
    q, k, v = synth.make_qkv(cfg)
    q = (q.float() + 0.5).to(q.dtype)
    blocks = [(0, 0, 0), (3, 31, 31), (1, 12, 17)]
    res = par.run_case(cfg, DEV, blocks=blocks, check_quant=False, rows_per_block=16, qkv_host=(q, k, v), qmean=True)
    print(par.assert_within_bars(res, "C5 N=4096 qmean"))


def test_uneven_head_map_equals_reordered_heads(hb, par):
    """An explicit query-head -> KV-head map with groups of different sizes and interleaved members gives,
    head by head, what the default grouping gives on the correspondingly gathered K/V heads."""
    cfg = synth.config("C3", N=320, Hq=4, Hkv=2)
    q, k, v = (t.to(DEV) for t in synth.make_qkv(cfg))
    head_map = [1, 0, 1, 1]                                     # three heads on KV head 1, one on KV head 0
    mapped = hb.attention_fwd(hb.quantize_qkv(q, k, v, q_to_kv=head_map), True, Bc=64)
    idx = torch.tensor(head_map, device=DEV)
    mha = hb.attention_fwd(hb.quantize_qkv(q, k[:, idx].contiguous(), v[:, idx].contiguous()), True, Bc=64)
    assert torch.equal(mapped, mha)
    mapped128 = hb.attention_fwd(hb.quantize_qkv(q, k, v, q_to_kv=head_map), True, Bc=128)
    mha128 = hb.attention_fwd(hb.quantize_qkv(q, k[:, idx].contiguous(), v[:, idx].contiguous()), True, Bc=128)
    assert torch.equal(mapped128, mha128)


@pytest.mark.parametrize("name", ["d128-bc64-causal-gqa", "d256-bc64-mild", "d64-bc64-causal-gqa-ragged"])
def test_output_dtypes_64_key_kernel(hb, par, name):
    """FP16 / BF16 outputs of the 64-key kernels are the FP32 output rounded once; reruns are bit-identical;
    rows past a ragged N are not written."""
    cfg = SMALL[name]
    q, k, v = synth.make_qkv(cfg)
    s, inv_s = par.calibrate(cfg, DEV)
    qkv = hb.quantize_qkv(q.to(DEV), k.to(DEV), v.to(DEV), s, inv_s)
    o32 = hb.attention_fwd(qkv, cfg.causal, Bc=64, out_dtype=hb.F32)
    assert torch.equal(o32, hb.attention_fwd(qkv, cfg.causal, Bc=64, out_dtype=hb.F32))
    assert torch.isfinite(o32).all()
    o16 = hb.attention_fwd(qkv, cfg.causal, Bc=64, out_dtype=hb.F16)
    ob16 = hb.attention_fwd(qkv, cfg.causal, Bc=64, out_dtype=hb.BF16)
    assert torch.equal(o16, o32.to(torch.float16)) and torch.equal(ob16, o32.to(torch.bfloat16))
    # a caller-provided output buffer with a guard region after it stays untouched beyond [B,Hq,N,d]
    n = o32.numel()
    buf = torch.full((n + 4096,), 7.0, dtype=torch.float32, device=DEV)
    hb.attention_fwd(qkv, cfg.causal, Bc=64, out_dtype=hb.F32, out=buf[:n].view_as(o32))
    assert torch.equal(buf[:n].view_as(o32), o32) and bool((buf[n:] == 7.0).all())


@pytest.mark.parametrize("d,Bc,normalizer", [(128, 64, 0), (256, 64, 0), (128, 128, 0), (64, 128, 0), (128, 64, 1)])
def test_nonzero_status_word_makes_every_kernel_family_a_no_op(hb, par, d, Bc, normalizer):
    """A call whose status word already holds an error does nothing: every CTA reads the word once,
    all of its roles agree on the verdict and leave through the common exit (which still frees tensor
    memory), the output buffer is untouched and the word is preserved.  The next ordinary call on the
    same device works, i.e. no tensor memory leaked and no barrier was left armed."""
    cfg = synth.config("C3", N=384, Hq=2, Hkv=1, d=d, Bc=Bc)
    q, k, v = (t.to(DEV) for t in synth.make_qkv(cfg))
    qkv = hb.quantize_qkv(q, k, v)
    status = torch.full((1,), 77, dtype=torch.int32, device=DEV)
    out = torch.full((cfg.B, cfg.Hq, cfg.N, cfg.d), 5.0, dtype=torch.float32, device=DEV)
    for _ in range(3):                                         # several launches: leaked tensor memory would block
        hb.attention_fwd(qkv, True, Bc=Bc, out=out, d_status=status, normalizer=normalizer)
    torch.cuda.synchronize()
    assert int(status.item()) == 77 and bool((out == 5.0).all())
    status.zero_()
    good = hb.attention_fwd(qkv, True, Bc=Bc, d_status=status, normalizer=normalizer)
    hb.attention_fwd(qkv, True, Bc=Bc, out=out, d_status=status, normalizer=normalizer)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(out, good) and torch.isfinite(out).all()


def test_expired_device_wait_is_reported_and_leaves_the_device_usable(hb, par):
    """The failure path of the bounded device-side waits, exercised without hanging or faulting anything: the
    self-test instantiation withholds the arrival that releases P V, the issuer's wait runs out after 2^12 polls,
    the status word reads HIFA4_ERR_TIMEOUT + 16 * site (site 7 = that wait), the call returns, the output buffer
    is untouched, and the next ordinary call on the same buffers passes parity (tensor memory was freed, no
    barrier stayed armed)."""
    cfg = synth.config("C3", N=128, Hq=1, Hkv=1, causal=False)           # one CTA, two key tiles
    q, k, v = (t.to(DEV) for t in synth.make_qkv(cfg))
    qkv = hb.quantize_qkv(q, k, v)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = torch.full((1, 1, cfg.N, cfg.d), 3.0, dtype=torch.float32, device=DEV)
    hb.selftest_wait_timeout(qkv, False, status, out=out)
    torch.cuda.synchronize()
    assert int(status.item()) == 6 + 16 * 7
    assert hb.status_string(6).lower().find("wait") >= 0 or hb.status_string(6)
    assert bool((out == 3.0).all())
    # a call that finds the status word set does nothing either; after clearing it everything works again
    hb.attention_fwd(qkv, False, Bc=64, out=out, d_status=status)
    torch.cuda.synchronize()
    assert bool((out == 3.0).all()) and int(status.item()) == 6 + 16 * 7
    res = par.run_case(cfg, DEV)
    print(par.assert_within_bars(res, "after the expired wait"))
    with pytest.raises(hb.Hifa4Error):                                  # the self-test refuses shapes it was not built for
        hb.selftest_wait_timeout(hb.quantize_qkv(*(t.to(DEV) for t in synth.make_qkv(synth.config("C3", N=128, Hq=1, Hkv=1, d=64)))),
                                 False, status)


@pytest.mark.parametrize("dtype,smooth,causal,p_dtype", [("bf16", True, True, "f16"), ("fp16", True, False, "f16"),
                                                         ("bf16", False, True, "f16"), ("fp16", True, True, "f32")])
def test_in_kernel_query_quantization_is_bit_identical(hb, par, dtype, smooth, causal, p_dtype):
    """hifa4_attention_fwd_qraw smooths and HIF4-quantizes Q inside the attention kernel (Algorithm 1 line 1 per CTA,
    in shared memory).  Both the stand-alone quantizer and the in-kernel one take the same exact arithmetic, so the
    output must equal, bit for bit, that of quantize_qkv + attention_fwd (which the other tests hold against the
    oracle), for both input types, with and without Smooth-QK factors, with GQA, a ragged last query block (N = 320)
    and an outlier-heavy K.  The K / V buffers written without Q must equal those written with it."""
    cfg = synth.config("C2", B=2, Hq=4, Hkv=2, N=320, dtype=dtype, causal=causal)
    q, k, v = (t.to(DEV) for t in synth.make_qkv(cfg))
    s, inv_s = par.calibrate(cfg, DEV) if smooth else (None, None)
    pd = hb.F32 if p_dtype == "f32" else hb.F16
    full = hb.quantize_qkv(q, k, v, s, inv_s)
    ref = hb.attention_fwd(full, causal, p_dtype=pd)
    kv = hb.quantize_qkv(None, k, v, s, inv_s, Hq=cfg.Hq)
    assert torch.equal(kv.k_mma, full.k_mma) and torch.equal(kv.v_mma, full.v_mma)
    assert torch.equal(kv.k_codes, full.k_codes) and torch.equal(kv.v_meta, full.v_meta)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for out_dtype in (hb.F32, hb.F16):
        got = hb.attention_fwd_qraw(q, s, kv, causal, out_dtype=out_dtype, p_dtype=pd, d_status=status)
        want = ref if out_dtype == hb.F32 else hb.attention_fwd(full, causal, out_dtype=out_dtype, p_dtype=pd)
        assert torch.equal(got, want)
    assert int(status.item()) == 0
    # a set status word makes the launch a no-op
    status.fill_(9)
    out = torch.full_like(ref, 2.0)
    hb.attention_fwd_qraw(q, s, kv, causal, out=out, p_dtype=pd, d_status=status)
    torch.cuda.synchronize()
    assert bool((out == 2.0).all()) and int(status.item()) == 9


def test_in_kernel_query_quantization_full_size_and_refusals(hb, par):
    """The headline shape through hifa4_attention_fwd_raw (which quantizes K and V into the workspace and Q inside the
    attention kernel from 64k query rows up) equals the two-call path; configurations the in-kernel quantizer was
    not built for are refused without a launch."""
    cfg = synth.config("C2")
    q, k, v = synth.make_qkv_device(cfg, DEV)
    s, inv_s = par.calibrate(cfg, DEV)
    full = hb.quantize_qkv(q, k, v, s, inv_s)
    want = hb.attention_fwd(full, True)
    before = hb.get_counters()
    got = hb.attention_fwd_raw(q, k, v, s, inv_s, True)
    after = hb.get_counters()
    assert torch.equal(got, want)
    assert after["launches"] - before["launches"] == 2          # K/V quantizer + attention
    kv = hb.quantize_qkv(None, k, v, s, inv_s, Hq=cfg.Hq)
    assert torch.equal(hb.attention_fwd_qraw(q, s, kv, True), want)
    c64 = synth.config("C3", N=128, Hq=1, Hkv=1, d=64)
    q6, k6, v6 = (t.to(DEV) for t in synth.make_qkv(c64))
    with pytest.raises(hb.Hifa4Error):
        hb.attention_fwd_qraw(q6, None, hb.quantize_qkv(None, k6, v6, Hq=1), True)


def test_calls_are_capturable_in_a_cuda_graph_and_replay_bit_identically(hb, par):
    """The entry points allocate nothing, synchronise nothing and only enqueue work on the caller's stream, so a
    quantize + attention pair (the grid with programmatic stream serialization included) and the raw entry point
    can be captured in a CUDA graph; replays write the same bits as the eager calls, also after the inputs changed
    in place."""
    cfg = synth.config("C2", B=1, Hq=8, Hkv=2, N=1024)
    q, k, v = (t.to(DEV) for t in synth.make_qkv(cfg))
    s, inv_s = par.calibrate(cfg, DEV)
    qkv = hb.quantize_qkv(q, k, v, s, inv_s)
    want = hb.attention_fwd(qkv, True)                                   # eager: also opts the kernels in
    want_raw = hb.attention_fwd_raw(q, k, v, s, inv_s, True)
    assert torch.equal(want, want_raw)
    out = torch.zeros_like(want)
    out_raw = torch.zeros_like(want)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = torch.empty(hb.attention_raw_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.N, cfg.d, qkv.in_dtype, True, 64),
                     dtype=torch.uint8, device=DEV)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=torch.cuda.Stream(device=DEV)):
        hb.quantize_qkv(q, k, v, s, inv_s, out=qkv, d_status=status)
        hb.attention_fwd(qkv, True, out=out, d_status=status)
        hb.attention_fwd_raw(q, k, v, s, inv_s, True, out=out_raw, workspace=ws, d_status=status)
    g.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(out, want) and torch.equal(out_raw, want)
    q2 = q.flip(2).contiguous()
    want2 = hb.attention_fwd(hb.quantize_qkv(q2, k, v, s, inv_s), True)
    q.copy_(q2)                                                          # same buffers, new contents
    g.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(out, want2) and torch.equal(out_raw, want2)
    assert not torch.equal(want, want2)


def test_concurrent_host_threads_on_their_own_streams(hb, par):
    """Two host threads call the library at the same time, each on its own stream and buffers (the per-device
    shared-memory opt-in and the tensor-map encoder look-up are guarded): both get the serial result."""
    import threading
    cfgs = [synth.config("C2", B=1, Hq=4, Hkv=2, N=512, seed=11), synth.config("C3", B=1, Hq=4, Hkv=1, N=768, seed=12)]
    data = [tuple(t.to(DEV) for t in synth.make_qkv(c)) for c in cfgs]
    want = [hb.attention_fwd(hb.quantize_qkv(*d), c.causal) for c, d in zip(cfgs, data)]
    torch.cuda.synchronize()
    got, errs = [None, None], []

    def work(i):
        try:
            with torch.cuda.stream(torch.cuda.Stream(device=DEV)):
                for _ in range(20):
                    got[i] = hb.attention_fwd_raw(*data[i], None, None, cfgs[i].causal)
                torch.cuda.current_stream().synchronize()
        except Exception as e:                                           # surfaced below
            errs.append(e)

    ts = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    assert not errs, errs
    assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1])
