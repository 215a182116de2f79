"""Parity of the FP8 linear layer in front of the attention (per-row quantiser, e4m3 GEMM, qkv projection with the
block quantiser fused into its epilogue) against the CPU oracle, through the C-ABI binding."""
import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc
from paper_2605_11354_b200 import binding as lt
from paper_2605_11354_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu


def activations(seed, rows, cols, dtype):
    g = np.random.default_rng(seed)
    x = (g.standard_normal((rows, cols)) * g.uniform(0.05, 8.0, size=(rows, 1))).astype(np.float32)
    if dtype == "bf16":
        x = wk.round_to_bf16(x)
    return x


@pytest.mark.parametrize("dtype,rows,cols", [("bf16", 333, 1024), ("f32", 65, 256), ("bf16", 7, 4096), ("f32", 1000, 16)])
def test_row_quantiser_is_bit_exact(dtype, rows, cols):
    x = activations(1, rows, cols, "f32")
    x[3] = 0.0
    x[4, 5] = 7.0e4
    x[5] *= 1e-7
    x[6, 0] = -0.0
    if dtype == "bf16":
        x = wk.round_to_bf16(x)
    codes, scales = lt.lite3r_quantize_rows_fp8(pu.to_device(x, dtype))
    torch.cuda.synchronize()
    ref_codes, ref_scales = orc.quantize_fp8_rows(x)
    assert np.array_equal(codes.cpu().numpy(), ref_codes)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), ref_scales.view(np.uint32))


def test_row_quantiser_strided_rows():
    x = activations(2, 50, 128, "f32")
    wide = torch.zeros((50, 200), device="cuda")
    wide[:, :128] = torch.from_numpy(x).cuda()
    codes, scales = lt.lite3r_quantize_rows_fp8(wide[:, :128])
    torch.cuda.synchronize()
    ref_codes, ref_scales = orc.quantize_fp8_rows(x)
    assert np.array_equal(codes.cpu().numpy(), ref_codes) and np.array_equal(scales.cpu().numpy(), ref_scales)


@pytest.mark.parametrize("rows,d_in,d_out,out_dtype,with_bias", [(300, 256, 192, torch.float32, True),
                                                                 (1, 128, 64, torch.float32, False),
                                                                 (513, 1024, 320, torch.bfloat16, True),
                                                                 (128, 384, 128, torch.float16, False)])
def test_linear_fp8_against_the_oracle(rows, d_in, d_out, out_dtype, with_bias):
    """y = x_q W_q^T + b: the e4m3 products are exact in fp32, so only the accumulation order separates the tensor-core
    result from the oracle's fp64 sum: 1e-5 of the largest output is ample (a few fp32 ulps over <= 1024 terms); the
    16-bit outputs add their own half ulp."""
    g = np.random.default_rng(3)
    x = activations(4, rows, d_in, "bf16")
    w = (g.standard_normal((d_out, d_in)) / np.sqrt(d_in)).astype(np.float32)
    b = g.standard_normal(d_out).astype(np.float32) if with_bias else None
    xc, xs = lt.lite3r_quantize_rows_fp8(pu.to_device(x, "bf16"))
    wc, ws = lt.lite3r_quantize_rows_fp8(torch.from_numpy(w).cuda())
    y = torch.full((rows, d_out), float("nan"), dtype=out_dtype, device="cuda")
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    lt.lite3r_linear_fp8(xc, xs, wc, ws, torch.from_numpy(b).cuda() if with_bias else None, y, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rxc, rxs = orc.quantize_fp8_rows(x)
    rwc, rws = orc.quantize_fp8_rows(w)
    ref = orc.linear_fp8(rxc, rxs, rwc, rws, b)
    got = y.float().cpu().numpy().astype(np.float64)
    half_ulp = {torch.float32: 0.0, torch.bfloat16: 2.0 ** -8, torch.float16: 2.0 ** -11}[out_dtype]
    err = np.abs(got - ref)
    print(f"linear {rows}x{d_in}x{d_out}: max err {err.max():.3e} of {np.abs(ref).max():.3e}")
    assert (err <= 1e-5 * np.abs(ref).max() + half_ulp * np.abs(ref)).all()


@pytest.mark.parametrize("block,tokens,batch,heads,d_model", [(64, 300, 2, 2, 256), (128, 300, 2, 2, 256),
                                                              (64, 1374, 1, 4, 512), (128, 129, 3, 2, 128)])
def test_fused_qkv_projection_against_the_oracle(block, tokens, batch, heads, d_model):
    """The projection with the block quantiser in its epilogue.  Each value is formed in fp32 from an accumulator whose
    summation order is the tensor core's, so it can differ from the oracle's fp64 value in the last fp32 bits; the
    tile maximum then moves the scale by an ulp or two and a value next to an e4m3 rounding boundary can take the
    neighbouring code.  Judged: scales within 4 fp32 ulps; dequantised values within 0.52 code steps of the oracle's
    exact value (half a step is the quantiser's own error bound); codes equal except for a counted fraction below
    0.5 %, each differing by one step; column sums exactly the sums of the GPU's own codes; padded rows zero."""
    g = np.random.default_rng(5)
    x = activations(6, batch * tokens, d_model, "bf16")
    w = (g.standard_normal((3 * heads * 64, d_model)) / np.sqrt(d_model)).astype(np.float32)
    b = (0.1 * g.standard_normal(3 * heads * 64)).astype(np.float32)
    xc, xs = lt.lite3r_quantize_rows_fp8(pu.to_device(x, "bf16"))
    wc, ws = lt.lite3r_quantize_rows_fp8(torch.from_numpy(w).cuda())
    shape = lt.Shape(batch, heads, tokens, 64, block)
    outs = [lt.alloc_fp8(shape, "cuda:0") for _ in range(3)]
    for o in outs:
        o.codes.fill_(0xAB)
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    lt.lite3r_qkv_project_fp8(xc, xs, wc, ws, torch.from_numpy(b).cuda(), shape, *outs, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    q, k, v, _ = orc.qkv_project_fp8(x.reshape(batch, tokens, d_model), w, heads, b)
    nb = -(-tokens // block)
    tab = orc.e4m3_value_table()
    total = flips = 0
    for name, ref, out in (("q", q, outs[0]), ("k", k, outs[1]), ("v", v, outs[2])):
        ref_codes, ref_scales = orc.quantize_fp8_blocks(ref.astype(np.float32), block)
        codes = out.codes.cpu().numpy()
        scales = out.scales.cpu().numpy()
        assert not codes[:, :, tokens:].any(), name  # padded rows
        ulps = np.abs(scales.view(np.int32).astype(np.int64) - ref_scales.view(np.int32).astype(np.int64))
        assert ulps.max() <= 4, (name, ulps.max())
        vals = tab[codes[:, :, :tokens]] * np.repeat(scales.astype(np.float64), block, axis=2)[:, :, :tokens, None]
        step = np.repeat(ref_scales.astype(np.float64), block, axis=2)[:, :, :tokens, None] * np.maximum(
            2.0 ** (np.floor(np.log2(np.maximum(np.abs(tab[ref_codes[:, :, :tokens]]), 2.0 ** -6))) - 3), 2.0 ** -9)
        assert (np.abs(vals - ref) <= 0.52 * step + 1e-12).all(), name
        diff = codes != ref_codes
        total += diff.size
        flips += int(diff.sum())
        if diff.any():  # a differing code is the neighbouring one (sign-magnitude codes: distance one)
            assert (np.abs(codes[diff].astype(np.int32) - ref_codes[diff].astype(np.int32)) == 1).all(), name
        colsum = out.colsum.cpu().numpy().astype(np.int64)
        assert np.array_equal(colsum, pu.colsum_units(codes, block)), name
    print(f"fused qkv block {block}: {flips} of {total} codes differ by one step")
    assert flips <= 0.005 * total
    # the tensors feed the attention path like the stand-alone quantiser's
    eng = lt.SlaForward(batch, heads, tokens, block, 0.3, 0.3)
    eng.q8, eng.k8, eng.v8 = outs
    eng.make_plan()
    proj = torch.from_numpy((g.standard_normal((heads, 64, 64)) / 8).astype(np.float32)).cuda()
    out = eng.forward(proj)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    qh, kh, vh = (orc.dequantize(o.codes.cpu().numpy(), o.scales.cpu().numpy(), tokens, block) for o in outs)
    ref_out = orc.sla_forward(qh, kh, vh, proj.cpu().numpy(), eng.plan.cls.cpu().numpy(), block)
    rel, mx = pu.output_errors(out.cpu().numpy(), ref_out)
    assert rel <= pu.REL_L2_TOL and mx <= pu.MAX_ABS_TOL * max(1.0, float(np.abs(ref_out).max()))


def test_attention_output_requantised_for_the_out_projection():
    """The step after the attention: its output, written token-major in bf16 ([B, N, H*64] seen as [B, H, N, 64]), is
    quantised per token for the attention block's output projection and multiplied by the e4m3 weight (Algorithm 2
    again).  Codes and scales are bit-exact for the bf16 values the forward stored; the product matches the oracle."""
    from test_gpu_parity import small_workload
    wl = small_workload("requant", tokens=500, heads=4, batch=2)
    inputs = wk.make_inputs(wl)
    eng, _ = pu.run_gpu(inputs, wl)
    proj = torch.from_numpy(inputs["proj"]).cuda()
    buf = torch.empty((wl.batch, wl.tokens, wl.heads, 64), dtype=torch.bfloat16, device="cuda")
    eng.forward(proj, out=buf.permute(0, 2, 1, 3))
    a = buf.view(wl.batch * wl.tokens, wl.heads * 64)
    ac, asc = lt.lite3r_quantize_rows_fp8(a)
    g = np.random.default_rng(11)
    w = (g.standard_normal((256, 256)) / 16).astype(np.float32)
    wc, ws = lt.lite3r_quantize_rows_fp8(torch.from_numpy(w).cuda())
    y = torch.empty((a.shape[0], 256), device="cuda")
    lt.lite3r_linear_fp8(ac, asc, wc, ws, None, y, eng.status)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    a_np = a.float().cpu().numpy()
    rc, rs = orc.quantize_fp8_rows(a_np)
    assert np.array_equal(ac.cpu().numpy(), rc) and np.array_equal(asc.cpu().numpy(), rs)
    rwc, rws = orc.quantize_fp8_rows(w)
    ref = orc.linear_fp8(rc, rs, rwc, rws)
    assert np.abs(y.cpu().numpy() - ref).max() <= 1e-5 * np.abs(ref).max()
