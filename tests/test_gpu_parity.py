"""Parity of the CUDA path (through the C-ABI binding) against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc
from paper_2605_11354_b200 import binding as lt
from paper_2605_11354_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu


def small_workload(name, **kw):
    base = dict(cfg_id=90, batch=1, heads=2, tokens=1000, head_dim=64, block=64, crit=0.25, neg=0.4, centres=16,
                sigma=0.3, src_dtype="bf16")
    base.update(kw)
    return wk.Workload(name, **base)


def oracle_subset(inputs, wl, heads, crit=None, neg=None, phi="softmax", cls=None, query_blocks=None):
    crit = wl.crit if crit is None else crit
    neg = wl.neg if neg is None else neg
    sl = [np.ascontiguousarray(inputs[n][:, heads]) for n in ("q", "k", "v")]
    return orc.sla_forward_from_source(*sl, inputs["proj"][heads], wl.block, crit, neg, phi=phi, cls=cls,
                                       query_blocks=query_blocks)


def check_quantized(eng, ref, wl, heads):
    for name, t in (("q", eng.q8), ("k", eng.k8), ("v", eng.v8)):
        codes = t.codes.cpu().numpy()[:, heads]
        scales = t.scales.cpu().numpy()[:, heads]
        assert np.array_equal(codes, ref[name + "_codes"]), name
        assert np.array_equal(scales.view(np.uint32), ref[name + "_scales"].view(np.uint32)), name
        if t.colsum is not None:
            colsum = t.colsum.cpu().numpy()[:, heads]
            assert np.array_equal(colsum.astype(np.int64), pu.colsum_units(ref[name + "_codes"], wl.block)), name


def full_parity(wl, inputs, heads=None, phi="softmax", crit=None, neg=None, query_blocks=None):
    heads = list(range(wl.heads)) if heads is None else heads
    eng, out = pu.run_gpu(inputs, wl, phi=phi, crit=crit, neg=neg)
    ref = oracle_subset(inputs, wl, heads, crit, neg, phi, query_blocks=[])
    check_quantized(eng, ref, wl, heads)
    flips, cls = pu.compare_plan(eng, ref["scores"], ref["cls"], heads)
    if flips:
        print(f"{wl.name}: {flips} class entries differ at pooled-score ties <= {pu.TIE_TOL}")
    ref_out = orc.sla_forward(ref["qhat"], ref["khat"], ref["vhat"], inputs["proj"][heads], cls, wl.block, phi,
                              query_blocks)
    rel, mx = pu.output_errors(out.cpu().numpy()[:, heads], ref_out)
    print(f"{wl.name}: rel_l2={rel:.3e} max_abs={mx:.3e} flips={flips}")
    assert rel <= pu.REL_L2_TOL and mx <= pu.MAX_ABS_TOL
    return eng, out


# ------------------------------------------------------------------------------------------------ small, complete
def test_tiny_config_full():
    wl = wk.WORKLOADS["tiny"]
    full_parity(wl, wk.make_inputs(wl))


@pytest.mark.parametrize("tokens,block", [(1000, 64), (1000, 128), (1024, 64), (65, 64), (64, 64), (129, 128), (7, 64)])
def test_ragged_and_small_shapes(tokens, block):
    wl = small_workload(f"small-{tokens}-{block}", tokens=tokens, block=block)
    full_parity(wl, wk.make_inputs(wl))


@pytest.mark.parametrize("crit,neg", [(1.0, 0.0), (0.0, 0.0), (0.0, 0.5), (0.3, 0.7), (0.05, 0.0), (0.0, 1.0)])
def test_degenerate_class_mixes(crit, neg):
    wl = small_workload(f"mix-{crit}-{neg}", tokens=700, crit=crit, neg=neg)
    full_parity(wl, wk.make_inputs(wl))


@pytest.mark.parametrize("block", [64, 128])
def test_elu_feature_map(block):
    wl = small_workload(f"elu-{block}", tokens=900, block=block)
    full_parity(wl, wk.make_inputs(wl), phi="elu1")


def test_fp32_source_and_strided_layout():
    """Sources laid out [B, N, H, D] (token-major) give the same codes as the contiguous [B, H, N, D] copy."""
    wl = small_workload("strided", tokens=777, src_dtype="f32", batch=2, heads=3)
    inputs = wk.make_inputs(wl)
    eng, _ = pu.run_gpu(inputs, wl)
    shape = eng.shape
    x = torch.from_numpy(inputs["k"]).cuda()
    x_bnhd = x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)  # same values, strides of a [B,N,H,D] buffer
    assert not x_bnhd.is_contiguous()
    alt = lt.alloc_fp8(shape, "cuda:0")
    lt.lite3r_quantize_fp8(x_bnhd, shape, alt)
    torch.cuda.synchronize()
    assert torch.equal(alt.codes, eng.k8.codes) and torch.equal(alt.scales, eng.k8.scales)
    assert torch.equal(alt.colsum, eng.k8.colsum)
    codes, scales = orc.quantize_fp8_blocks(inputs["k"], wl.block)
    assert np.array_equal(alt.codes.cpu().numpy(), codes)
    assert np.array_equal(alt.scales.cpu().numpy(), scales)


def test_qkv_launch_matches_single_launches():
    """lite3r_quantize_fp8_qkv (one launch for Q, K, V, different strides) is bit-identical to three single calls."""
    wl = small_workload("qkv", tokens=1111, batch=2, heads=3)
    inputs = wk.make_inputs(wl)
    shape = lt.Shape(wl.batch, wl.heads, wl.tokens, 64, wl.block)
    q, k, v = (pu.to_device(inputs[n], wl.src_dtype) for n in ("q", "k", "v"))
    k = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)  # token-major strides for one of the three
    single = [lt.alloc_fp8(shape, "cuda:0") for _ in range(3)]
    for x, out in zip((q, k, v), single):
        lt.lite3r_quantize_fp8(x, shape, out)
    fused = [lt.alloc_fp8(shape, "cuda:0") for _ in range(3)]
    lt.lite3r_quantize_fp8_qkv(q, k, v, shape, *fused)
    torch.cuda.synchronize()
    for a, b in zip(single, fused):
        assert torch.equal(a.codes, b.codes) and torch.equal(a.scales, b.scales) and torch.equal(a.colsum, b.colsum)
    codes, scales = orc.quantize_fp8_blocks(inputs["v"], wl.block)
    assert np.array_equal(fused[2].codes.cpu().numpy(), codes)
    assert np.array_equal(fused[2].scales.cpu().numpy().view(np.uint32), scales.view(np.uint32))


def test_quantizer_extremes():
    """All-zero tile, a single huge outlier, tiny magnitudes, negative zero: codes and scales bit-exact."""
    g = np.random.default_rng(5)
    x = g.standard_normal((1, 2, 300, 64)).astype(np.float32)
    x[0, 0, :64] = 0.0
    x[0, 0, 70, 3] = 3.0e4
    x[0, 1, 128:192] *= 1e-6
    x[0, 1, 200, 5] = -0.0
    wl = small_workload("extremes", tokens=300, src_dtype="f32")
    shape = lt.Shape(1, 2, 300, 64, 64)
    out = lt.alloc_fp8(shape, "cuda:0")
    lt.lite3r_quantize_fp8(torch.from_numpy(x).cuda(), shape, out)
    torch.cuda.synchronize()
    codes, scales = orc.quantize_fp8_blocks(x, 64)
    assert np.array_equal(out.codes.cpu().numpy(), codes)
    assert np.array_equal(out.scales.cpu().numpy().view(np.uint32), scales.view(np.uint32))
    assert np.array_equal(out.colsum.cpu().numpy().astype(np.int64), pu.colsum_units(codes, 64))


def test_shared_projection_and_determinism():
    wl = small_workload("shared-proj", tokens=640)
    inputs = wk.make_inputs(wl)
    eng, out = pu.run_gpu(inputs, wl)
    first = out.clone()
    proj = torch.from_numpy(inputs["proj"]).cuda()
    again = eng.forward(proj).clone()
    torch.cuda.synchronize()
    assert torch.equal(first, again)  # bit-identical on a re-run
    shared = eng.forward(proj[1].contiguous()).clone()
    torch.cuda.synchronize()
    ref = oracle_subset({**inputs, "proj": np.stack([inputs["proj"][1]] * 2)}, wl, [0, 1],
                        cls=eng.plan.cls.cpu().numpy())
    rel, mx = pu.output_errors(shared.cpu().numpy(), ref["out"])
    assert rel <= pu.REL_L2_TOL and mx <= pu.MAX_ABS_TOL


def test_ties_resolve_to_lower_index():
    """Duplicated key blocks give exactly equal pooled scores; the lower block index must rank first."""
    wl = small_workload("ties", tokens=640, heads=1, src_dtype="f32", crit=0.3, neg=0.3)
    inputs = wk.make_inputs(wl)
    k = inputs["k"]
    for dst, src in ((3, 1), (5, 1), (8, 2)):
        k[0, 0, dst * 64:(dst + 1) * 64] = k[0, 0, src * 64:(src + 1) * 64]
        inputs["v"][0, 0, dst * 64:(dst + 1) * 64] = inputs["v"][0, 0, src * 64:(src + 1) * 64]
    eng, _ = pu.run_gpu(inputs, wl)
    ref = oracle_subset(inputs, wl, [0], query_blocks=[])
    s = ref["scores"][0, 0]
    assert (s[:, 3] == s[:, 1]).all() and (s[:, 8] == s[:, 2]).all()
    assert np.array_equal(eng.plan.cls.cpu().numpy(), ref["cls"])


@pytest.mark.parametrize("seed", [7, 23])
def test_random_shapes_against_the_oracle(seed):
    """Seeded sweep over shapes, block sizes, class mixes, feature maps, source types and input structure: every case
    is checked like the fixed ones (codes, scales, column sums, plan, output)."""
    rng = np.random.default_rng(seed)
    for case in range(24):
        wl = wk.Workload(f"sweep{seed}-{case}", cfg_id=200 + case, batch=int(rng.integers(1, 4)),
                         heads=int(rng.integers(1, 4)), tokens=int(rng.integers(1, 2600)), head_dim=64,
                         block=int(rng.choice([64, 128])), crit=float(rng.choice([0.0, 0.05, 0.1, 0.3, 0.6, 1.0])),
                         neg=float(rng.choice([0.0, 0.2, 0.5, 0.9])), centres=int(rng.choice([0, 8, 32])), sigma=0.3,
                         src_dtype=str(rng.choice(["bf16", "f32"])))
        phi = str(rng.choice(["softmax", "elu1"]))
        blocks = None
        if wl.n_blocks * wl.batch * wl.heads > 40:
            blocks = pu.sample_blocks(wl, list(range(wl.heads)), 24, seed=case)
        full_parity(wl, wk.make_inputs(wl), phi=phi, query_blocks=blocks)


def test_all_scores_tied_in_a_long_row():
    """Zero queries make every pooled score of a row equal (one bucket holding all 150 blocks, more than the
    candidate list keeps): the selection must fall back to index order, exactly as the oracle ranks them."""
    wl = small_workload("alltied", tokens=150 * 64, heads=1, src_dtype="bf16", crit=0.2, neg=0.5)
    inputs = wk.make_inputs(wl)
    inputs["q"][:] = 0.0
    eng, _ = pu.run_gpu(inputs, wl)
    ref = oracle_subset(inputs, wl, [0], query_blocks=[])
    assert (ref["scores"] == 0).all()
    cls = eng.plan.cls.cpu().numpy()
    assert np.array_equal(cls, ref["cls"])
    k_c, k_m = eng.plan.k_crit, eng.plan.k_marg
    assert (cls[0, 0, :, :k_c] == 2).all() and (cls[0, 0, :, k_c:k_c + k_m] == 1).all()


def test_plan_of_a_very_long_sequence():
    """3000 blocks: the 64-bit row keys of eight query blocks no longer fit in shared memory, so the plan runs on the
    kernel that keeps single-precision scores and recomputes the exact keys at the selection thresholds.  Quantiser
    and plan are compared in full, the output on a few sampled query blocks."""
    wl = small_workload("long", tokens=3000 * 64 - 17, heads=1, src_dtype="bf16", crit=0.01, neg=0.95)
    inputs = wk.make_inputs(wl)
    full_parity(wl, inputs, query_blocks=pu.sample_blocks(wl, [0], 6, seed=5))


@pytest.fixture
def plan_variant():
    """Forces one of the plan kernels for the duration of a test (the library chooses by size otherwise)."""
    yield lt.lite3r_plan_variant
    lt.lite3r_plan_variant(0)


def plan_only(inputs, wl, crit=None, neg=None):
    """Quantises and plans on the GPU; returns the class matrix and the index lists as the oracle lays them out."""
    crit = wl.crit if crit is None else crit
    neg = wl.neg if neg is None else neg
    eng = lt.SlaForward(wl.batch, wl.heads, wl.tokens, wl.block, crit, neg)
    eng.quantize(*[pu.to_device(inputs[n], wl.src_dtype) for n in ("q", "k", "v")])
    eng.make_plan()
    torch.cuda.synchronize()
    return eng


@pytest.mark.parametrize("variant", [1, 2, 3, 4])
def test_every_plan_kernel_on_ties_and_near_ties(variant, plan_variant):
    """The four plan kernels (64-bit keys, single-precision scores with 8 or 16 rows per CTA, staged column sums) must
    give the oracle's plan bit for bit on the cases that separate them: exact ties (duplicated key blocks), rows
    whose scores are all equal (every entry in one place of the selection histogram: the keys are recomputed pass by
    pass), a crowded histogram bucket that only the refinement separates, ragged last blocks, and empty classes."""
    plan_variant(variant)
    # duplicated key blocks in a ragged sequence of 300 blocks
    wl = small_workload(f"var{variant}-ties", tokens=300 * 64 - 21, heads=2, src_dtype="f32", crit=0.1, neg=0.45)
    inputs = wk.make_inputs(wl)
    for dst, src in ((3, 1), (5, 1), (8, 2), (299, 7), (150, 149)):
        n = min(64, wl.tokens - dst * 64)
        inputs["k"][:, :, dst * 64:dst * 64 + n] = inputs["k"][:, :, src * 64:src * 64 + n]
    for crit, neg in ((0.1, 0.45), (0.0, 0.5), (0.37, 0.63), (1.0, 0.0), (0.02, 0.0)):
        eng = plan_only(inputs, wl, crit, neg)
        ref = oracle_subset(inputs, wl, [0, 1], crit, neg, query_blocks=[])
        flips, _ = pu.compare_plan(eng, ref["scores"], ref["cls"], [0, 1])
        assert flips == 0, (variant, crit, neg, flips)
    # all scores of every row equal, then nearly equal: keys that differ only far below single precision
    wl = small_workload(f"var{variant}-flat", tokens=400 * 64, heads=1, src_dtype="f32", crit=0.2, neg=0.5)
    inputs = wk.make_inputs(wl)
    inputs["q"][:] = 0.0
    eng = plan_only(inputs, wl)
    ref = oracle_subset(inputs, wl, [0], query_blocks=[])
    assert np.array_equal(eng.plan.cls.cpu().numpy(), ref["cls"])
    # a crowded bucket: 390 key blocks with scores within 5 % of each other and ten a hundred times larger, which
    # stretch the histogram's range so that the 390 share one of its 256 buckets (far more than the candidate list
    # keeps) and only the 16-bit refinement separates them
    g = np.random.default_rng(variant)
    inputs["q"][:] = 1.0
    level = (1.0 + 0.05 * g.uniform(-1.0, 1.0, 400)).astype(np.float32)
    level[g.choice(400, 10, replace=False)] = 100.0
    inputs["k"][0, 0] = np.repeat(level, 64)[:, None]
    for crit, neg in ((0.2, 0.5), (0.5, 0.1), (0.02, 0.9)):
        eng = plan_only(inputs, wl, crit, neg)
        ref = oracle_subset(inputs, wl, [0], crit, neg, query_blocks=[])
        flips, _ = pu.compare_plan(eng, ref["scores"], ref["cls"], [0])
        assert flips == 0, (variant, crit, neg)


@pytest.mark.parametrize("variant", [1, 2, 3, 4])
def test_every_plan_kernel_on_random_shapes(variant, plan_variant):
    plan_variant(variant)
    rng = np.random.default_rng(100 + variant)
    for case in range(10):
        wl = wk.Workload(f"planvar{variant}-{case}", cfg_id=300 + case, batch=int(rng.integers(1, 3)),
                         heads=int(rng.integers(1, 4)), tokens=int(rng.integers(1, 40000)), head_dim=64,
                         block=int(rng.choice([64, 128])), crit=float(rng.choice([0.0, 0.02, 0.1, 0.3, 1.0])),
                         neg=float(rng.choice([0.0, 0.2, 0.6, 0.9])), centres=int(rng.choice([0, 8, 64])), sigma=0.3,
                         src_dtype="bf16")
        inputs = wk.make_inputs(wl)
        eng = plan_only(inputs, wl)
        heads = list(range(wl.heads))
        ref = oracle_subset(inputs, wl, heads, query_blocks=[])
        flips, _ = pu.compare_plan(eng, ref["scores"], ref["cls"], heads)
        if flips:
            print(f"{wl.name}: {flips} class entries differ at pooled-score ties <= {pu.TIE_TOL}")


# ------------------------------------------------------------------------------------------------ benchmark shapes
def test_vggt8_two_heads_every_block():
    wl = wk.scaled_down(wk.WORKLOADS["vggt8"], heads=2)
    full_parity(wl, wk.make_inputs(wl))


def test_da3l_cut_every_block():
    wl = wk.scaled_down(wk.WORKLOADS["da3l"], heads=2, batch=1, tokens=6 * wk.TOKENS_PER_FRAME)
    full_parity(wl, wk.make_inputs(wl))


def test_frame_attention_cut_every_block():
    """Frame attention (one short sequence per frame, batch = frames): three frames, two heads, every query block."""
    wl = wk.scaled_down(wk.WORKLOADS["frame32"], heads=2, batch=3)
    full_parity(wl, wk.make_inputs(wl))


@pytest.mark.parametrize("name,oracle_heads,samples", [("vggt8", [0, 7, 15], 40), ("vggt32", [3, 12], 32),
                                                       ("da3l", [5], 32), ("frame32", [4, 11], 48)])
def test_full_size_configs_on_sampled_blocks(name, oracle_heads, samples):
    """The launch configuration the benchmark times, checked on a seeded sample of query blocks (always block 0,
    the ragged last block and one block per checked head); quantiser and plan are compared in full for those heads."""
    wl = wk.WORKLOADS[name]
    inputs = wk.make_inputs(wl)
    qb = pu.sample_blocks(wl, list(range(len(oracle_heads))), samples, seed=wl.cfg_id)
    full_parity(wl, inputs, heads=oracle_heads, query_blocks=qb)


@pytest.mark.parametrize("crit,neg", wk.STRESS_SWEEP[:4])
def test_stress_sweep_on_sampled_blocks(crit, neg):
    """All four sparsity points of the 100-frame sweep (critical 2 / 5 / 10 / 25 %, negligible 60 %)."""
    wl = wk.WORKLOADS["stress100"]
    inputs = wk.make_inputs(wl)
    qb = pu.sample_blocks(wl, [0], 12, seed=17)
    full_parity(wl, inputs, heads=[9], crit=crit, neg=neg, query_blocks=qb)


def test_stress_dense_equivalent_point():
    """Critical fraction 1.0 at 137 400 tokens: every key block is critical, the sparse branch is dense attention
    (2147 key steps per query tile) and the linear branch vanishes."""
    wl = wk.WORKLOADS["stress100"]
    inputs = wk.make_inputs(wl)
    qb = pu.sample_blocks(wl, [0], 4, seed=23)
    full_parity(wl, inputs, heads=[4], crit=1.0, neg=0.0, query_blocks=qb)


def test_overlapped_run_matches_the_in_order_run():
    """lite3r_sla_forward_begin on a side stream beside the plan, then lite3r_sla_forward_finish: bit-identical to the
    three calls in order, also when the two ways alternate on one engine."""
    wl = small_workload("overlap", tokens=5 * 1374, heads=4, batch=2)
    inputs = wk.make_inputs(wl)
    eng, expected = pu.run_gpu(inputs, wl)
    expected = expected.clone()
    q, k, v = (pu.to_device(inputs[n], wl.src_dtype) for n in ("q", "k", "v"))
    proj = torch.from_numpy(inputs["proj"]).cuda()
    for overlap in (True, True, False, True):
        eng.out.fill_(float("nan"))
        out = eng.run(q, k, v, proj, overlap=overlap)
        torch.cuda.synchronize()
        assert int(eng.status.item()) == 0
        assert torch.equal(out, expected), overlap


def test_token_major_output_layout():
    """The output may be a [B, N, H, D] buffer viewed as [B, H, N, D]: only the strides change."""
    wl = small_workload("out-strides", tokens=450, batch=2, heads=3)
    inputs = wk.make_inputs(wl)
    eng, out = pu.run_gpu(inputs, wl)
    proj = torch.from_numpy(inputs["proj"]).cuda()
    buf = torch.full((wl.batch, wl.tokens, wl.heads, 64), float("nan"), device="cuda")
    view = buf.permute(0, 2, 1, 3)
    lt.lite3r_sla_forward(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, view, eng.workspace, eng.status)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    assert torch.equal(view, out)


def test_device_waits_are_bounded():
    """A wait that can never be satisfied gives up after its limit, reports through device_status and leaves the
    context usable (the forward still runs and matches afterwards)."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    lt.selftest_wait_expiry(status, 2_000_000)  # 2 ms
    t1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 999
    assert 1.0 <= t0.elapsed_time(t1) < 200.0
    wl = wk.WORKLOADS["tiny"]
    full_parity(wl, wk.make_inputs(wl))


# ------------------------------------------------------------------------------------------------ boundary options
def bf16_round(x: np.ndarray) -> np.ndarray:
    return wk.round_to_bf16(x.astype(np.float32)).astype(np.float64)


@pytest.mark.parametrize("dtype,block", [(torch.bfloat16, 64), (torch.float16, 64), (torch.bfloat16, 128)])
def test_sixteen_bit_output(dtype, block):
    """out_dtype bf16 / fp16: the stored values are the fp32 result rounded to nearest even.  Checked two ways: bit for
    bit against the fp32 run's values cast by torch, and against the oracle within the fp32 tolerance plus half an
    ulp of the output type (bf16: 2^-8 relative, fp16: 2^-11)."""
    wl = small_workload(f"out16-{block}", tokens=1100, block=block, heads=3, batch=2)
    inputs = wk.make_inputs(wl)
    eng, out32 = pu.run_gpu(inputs, wl)
    proj = torch.from_numpy(inputs["proj"]).cuda()
    buf = torch.full((wl.batch, wl.heads, wl.tokens, 64), float("nan"), dtype=dtype, device="cuda")
    lt.lite3r_sla_forward(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, buf, eng.workspace, eng.status)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    assert torch.equal(buf, out32.to(dtype))
    ref = oracle_subset(inputs, wl, list(range(wl.heads)), cls=eng.plan.cls.cpu().numpy())
    got = buf.float().cpu().numpy().astype(np.float64)
    half_ulp = 2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -11
    err = np.abs(got - ref["out"])
    assert (err <= pu.MAX_ABS_TOL + half_ulp * np.abs(ref["out"])).all()
    rel, _ = pu.output_errors(got, ref["out"])
    assert rel <= pu.REL_L2_TOL + half_ulp  # rounding alone is at most half an ulp relative on every element


def test_token_major_sixteen_bit_output():
    wl = small_workload("out16-strides", tokens=450, batch=2, heads=3)
    inputs = wk.make_inputs(wl)
    eng, out = pu.run_gpu(inputs, wl)
    proj = torch.from_numpy(inputs["proj"]).cuda()
    buf = torch.full((wl.batch, wl.tokens, wl.heads, 64), float("nan"), dtype=torch.bfloat16, device="cuda")
    view = buf.permute(0, 2, 1, 3)
    lt.lite3r_sla_forward(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, view, eng.workspace, eng.status)
    torch.cuda.synchronize()
    assert torch.equal(view, out.to(torch.bfloat16))


@pytest.mark.parametrize("block,crit,neg", [(64, 0.25, 0.4), (128, 0.1, 0.5), (64, 0.0, 0.3), (64, 1.0, 0.0)])
def test_forward_builds_its_own_plan(block, crit, neg):
    """plan == NULL: lite3r_sla_forward classifies the blocks itself (inside its workspace) from the fractions; the
    result is bit-identical to lite3r_sla_plan followed by the forward, and the plan it left in the workspace is the
    one lite3r_sla_plan writes."""
    wl = small_workload(f"selfplan-{block}", tokens=1500, block=block, heads=2, batch=2, crit=crit, neg=neg)
    inputs = wk.make_inputs(wl)
    eng, expected = pu.run_gpu(inputs, wl)
    inside = lt.SlaForward(wl.batch, wl.heads, wl.tokens, wl.block, crit, neg, plan_inside=True)
    q, k, v = (pu.to_device(inputs[n], wl.src_dtype) for n in ("q", "k", "v"))
    proj = torch.from_numpy(inputs["proj"]).cuda()
    inside.workspace.fill_(0xEE)
    out = inside.run(q, k, v, proj)
    torch.cuda.synchronize()
    assert int(inside.status.item()) == 0
    assert torch.equal(out, expected)
    off = lt.lite3r_workspace_layout(inside.shape, crit, neg, plan_inside=True)
    nb, tiles = wl.n_blocks, wl.batch * wl.heads * wl.n_blocks
    cls = inside.workspace[off[4]:off[4] + tiles * nb].view(torch.int8).view(wl.batch, wl.heads, nb, nb)
    assert torch.equal(cls, eng.plan.cls)
    if eng.plan.k_crit:
        lists = inside.workspace[off[5]:off[5] + tiles * eng.plan.k_crit * 4].view(torch.int32)
        assert torch.equal(lists.view(wl.batch, wl.heads, nb, eng.plan.k_crit), eng.plan.crit_idx)


# ------------------------------------------------------------------------------------------------ memory safety
@pytest.mark.parametrize("tokens,block,batch,heads,crit,neg", [(7, 64, 1, 1, 0.5, 0.2), (1000, 64, 1, 2, 0.25, 0.4),
                                                                (1000, 128, 2, 1, 0.25, 0.4), (1374, 64, 3, 2, 0.25, 0.5),
                                                                (200, 64, 1, 1, 1.0, 0.0), (200, 128, 1, 1, 0.0, 0.0)])
def test_no_write_outside_the_buffers(tokens, block, batch, heads, crit, neg):
    """Every buffer the library writes (codes, scales, column sums, classes, both index lists, workspace, output) sits
    between two bands of a known byte pattern; after quantise + plan + forward the bands must be untouched.  Stands
    in for a memory checker: a kernel that writes a few bytes past a buffer fails here."""
    wl = small_workload("bands", tokens=tokens, block=block, batch=batch, heads=heads, crit=crit, neg=neg)
    inputs = wk.make_inputs(wl)
    shape = lt.Shape(batch, heads, tokens, 64, block)
    band = 4096
    guarded = []

    def banded(nbytes, dtype, shp):
        raw = torch.full((nbytes + 2 * band + 256,), 0xA5, dtype=torch.uint8, device="cuda")
        start = band + (-(raw.data_ptr() + band)) % 256
        guarded.append((raw, start, nbytes))
        return raw[start:start + nbytes].view(dtype).view(shp)

    codes_b, scales_b, colsum_b = lt.lite3r_fp8_sizes(shape)
    nb = wl.n_blocks
    fp8 = []
    for _ in range(3):
        fp8.append(lt.Fp8Tensor(banded(codes_b, torch.uint8, (batch, heads, nb * block, 64)),
                                banded(scales_b, torch.float32, (batch, heads, nb)),
                                banded(colsum_b, torch.int32, (batch, heads, nb, 64))))
    cls_b, crit_b, marg_b, kc, km, kn = lt.lite3r_plan_sizes(shape, crit, neg)
    plan = lt.PlanBuffers(banded(cls_b, torch.int8, (batch, heads, nb, nb)),
                          banded(max(crit_b, 4), torch.int32, (-1,))[:batch * heads * nb * kc].view(batch, heads, nb, kc),
                          banded(max(marg_b, 4), torch.int32, (-1,))[:batch * heads * nb * km].view(batch, heads, nb, km),
                          kc, km, kn)
    ws = banded(lt.lite3r_forward_workspace(shape, crit, neg), torch.uint8, (-1,))
    out = banded(batch * heads * tokens * 64 * 4, torch.float32, (batch, heads, tokens, 64))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q, k, v = (pu.to_device(inputs[n], wl.src_dtype) for n in ("q", "k", "v"))
    proj = torch.from_numpy(inputs["proj"]).cuda()
    lt.lite3r_quantize_fp8_qkv(q, k, v, shape, *fp8)
    lt.lite3r_sla_plan(fp8[0], fp8[1], shape, crit, neg, plan)
    lt.lite3r_sla_forward(fp8[0], fp8[1], fp8[2], proj, shape, lt.PHI_SOFTMAX, plan, out, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for raw, start, nbytes in guarded:
        assert bool((raw[:start] == 0xA5).all()) and bool((raw[start + nbytes:] == 0xA5).all())
    # and the run is the ordinary one
    eng, expected = pu.run_gpu(inputs, wl, crit=crit, neg=neg)
    assert torch.equal(out, expected)


# ------------------------------------------------------------------------------------------------ intermediates
@pytest.mark.parametrize("block,phi", [(64, "softmax"), (128, "softmax"), (64, "elu1")])
def test_workspace_intermediates_against_the_oracle(block, phi):
    """The linear branch's intermediates as the kernels leave them in the workspace: per-key-block summaries
    ((H_j W)^T | z_j), their sums over the marginal blocks (G_i^T W-folded | zeta_i) and the fp16 copy of V, against
    the oracle's kv_summaries (times W) at the precision they are stored in (bf16: 2^-9 relative per element)."""
    wl = small_workload(f"ws-{block}-{phi}", tokens=1000, block=block, heads=2, batch=1)
    inputs = wk.make_inputs(wl)
    eng, _ = pu.run_gpu(inputs, wl, phi=phi)
    ref = oracle_subset(inputs, wl, [0, 1], phi=phi, cls=eng.plan.cls.cpu().numpy(), query_blocks=[])
    Hs, zs = orc.kv_summaries(ref["khat"], ref["vhat"], block, phi)
    W = inputs["proj"].astype(np.float64)
    HW = np.einsum("bhjde,hef->bhjdf", Hs, W)  # H_j W, [d][f]
    off = lt.lite3r_workspace_layout(eng.shape, wl.crit, wl.neg)
    nb, tiles = wl.n_blocks, wl.heads * wl.n_blocks
    ws = eng.workspace
    hws = ws[off[0]:off[0] + tiles * 4160 * 2].view(torch.bfloat16).float().cpu().numpy().reshape(1, wl.heads, nb, 4160)
    got_hw_t = hws[..., :4096].reshape(1, wl.heads, nb, 64, 64)  # [f][d]
    got_z = hws[..., 4096:]

    def close(got, want, rel, what):
        scale = np.abs(want).max()
        err = np.abs(got - want).max()
        assert err <= rel * scale, (what, err, scale)

    close(got_hw_t, np.swapaxes(HW, -1, -2), 6e-3, "summaries")  # fp16 operands, bf16 storage
    close(got_z, zs, 4e-3, "normalisers")
    cls = eng.plan.cls.cpu().numpy()
    marg = (cls == 1).astype(np.float64)
    G = np.einsum("bhij,bhjdf->bhidf", marg, HW)
    zeta = np.einsum("bhij,bhjd->bhid", marg, zs)
    g16 = ws[off[1]:off[1] + tiles * 4096 * 2].view(torch.bfloat16).float().cpu().numpy().reshape(1, wl.heads, nb, 64, 64)
    zt = ws[off[2]:off[2] + tiles * 64 * 4].view(torch.float32).cpu().numpy().reshape(1, wl.heads, nb, 64)
    close(g16, np.swapaxes(G, -1, -2), 8e-3, "aggregates")
    close(zt, zeta, 4e-3, "zeta")
    v16 = ws[off[3]:off[3] + tiles * block * 64 * 2].view(torch.float16).float().cpu().numpy()
    v16 = v16.reshape(1, wl.heads, nb * block, 64)[:, :, :wl.tokens]
    assert np.abs(v16 - ref["vhat"]).max() <= 2.0 ** -11 * np.abs(ref["vhat"]).max()


@pytest.mark.parametrize("phi,vscale,kscale", [("softmax", 300.0, 1.0), ("elu1", 100.0, 3.0), ("softmax", 1e-3, 20.0)])
def test_large_and_small_magnitudes(phi, vscale, kscale):
    """Values far from unit scale (V in the hundreds, K several times larger, V tiny): inside the documented range the
    fp16 / bf16 intermediates neither overflow nor lose the result; checked against the oracle with the tolerance
    scaled by the output's magnitude."""
    wl = small_workload(f"mag-{phi}", tokens=900, heads=2, src_dtype="f32")
    inputs = wk.make_inputs(wl)
    inputs["v"] = (inputs["v"] * np.float32(vscale)).astype(np.float32)
    inputs["k"] = (inputs["k"] * np.float32(kscale)).astype(np.float32)
    eng, out = pu.run_gpu(inputs, wl, phi=phi)
    ref = oracle_subset(inputs, wl, [0, 1], phi=phi, cls=eng.plan.cls.cpu().numpy())
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    rel, mx = pu.output_errors(got, ref["out"])
    assert rel <= pu.REL_L2_TOL and mx <= pu.MAX_ABS_TOL * max(1.0, vscale)


def test_step_replayed_as_a_cuda_graph():
    """SlaForward.run_graph (one captured step) gives the bits of the stream-ordered run, on replay after replay and
    after new values were written into the captured source tensors."""
    wl = small_workload("graph", tokens=3 * 1374, heads=4, batch=2)
    inputs = wk.make_inputs(wl)
    eng, expected = pu.run_gpu(inputs, wl)
    expected = expected.clone()
    q, k, v = (pu.to_device(inputs[n], wl.src_dtype) for n in ("q", "k", "v"))
    proj = torch.from_numpy(inputs["proj"]).cuda()
    for _ in range(3):
        eng.out.fill_(float("nan"))
        out = eng.run_graph(q, k, v, proj)
        torch.cuda.synchronize()
        assert int(eng.status.item()) == 0 and torch.equal(out, expected)
    other = wk.make_inputs(small_workload("graph2", tokens=3 * 1374, heads=4, batch=2, cfg_id=92))
    for n, t in (("q", q), ("k", k), ("v", v)):
        t.copy_(pu.to_device(other[n], wl.src_dtype))
    out = eng.run_graph(q, k, v, proj).clone()
    torch.cuda.synchronize()
    ref = eng.run(q, k, v, proj)
    torch.cuda.synchronize()
    assert torch.equal(out, ref) and not torch.equal(out, expected)


@pytest.mark.parametrize("tokens,block,dtype,token_major", [(1000, 64, torch.float32, False), (7, 64, torch.float32, False),
                                                            (1000, 128, torch.bfloat16, False), (129, 128, torch.float32, True),
                                                            (1374, 64, torch.float16, True), (704, 64, torch.float32, False)])
def test_plain_stores_and_tma_stores_write_the_same(tokens, block, dtype, token_major):
    """The attention kernel's two ways of writing the output (TMA stores; plain vector stores, which it falls back to
    when no tensor map can describe the output) must give the same bytes, ragged tails, odd block counts (the copy of
    the last block in a pair is not stored), 16-bit types and token-major layouts included; and neither may touch
    anything outside the rows and columns of the output."""
    wl = small_workload(f"stores-{tokens}-{block}", tokens=tokens, block=block, batch=2, heads=3)
    inputs = wk.make_inputs(wl)
    eng, _ = pu.run_gpu(inputs, wl)
    proj = torch.from_numpy(inputs["proj"]).cuda()
    results = []
    try:
        for plain in (False, True):
            lt.lite3r_attention_plain_stores(plain)
            if token_major:  # [B, N, H, 80]: rows 80 wide, the kernel writes the first 64 columns
                buf = torch.full((wl.batch, wl.tokens, wl.heads, 80), 7.0, dtype=dtype, device="cuda")
                out = buf[..., :64].permute(0, 2, 1, 3)
            else:
                buf = torch.full((wl.batch, wl.heads, wl.tokens + 3, 64), 7.0, dtype=dtype, device="cuda")
                out = buf[:, :, :wl.tokens]
            eng.forward(proj, out=out)
            torch.cuda.synchronize()
            assert int(eng.status.item()) == 0
            results.append(buf.clone())
    finally:
        lt.lite3r_attention_plain_stores(False)
    assert torch.equal(results[0], results[1])
    if token_major:
        assert (results[0][..., 64:] == 7.0).all()
    else:
        assert (results[0][:, :, wl.tokens:] == 7.0).all()
    assert torch.isfinite(results[0].float()).all()
