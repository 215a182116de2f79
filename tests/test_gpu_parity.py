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
    """3000 blocks: the row keys of eight query blocks no longer fit in shared memory, so the plan kernel runs with
    four rows per CTA, staged column sums and the whole selection in the radix select.  Quantiser and plan are
    compared in full, the output on a few sampled query blocks."""
    wl = small_workload("long", tokens=3000 * 64 - 17, heads=1, src_dtype="bf16", crit=0.01, neg=0.95)
    inputs = wk.make_inputs(wl)
    full_parity(wl, inputs, query_blocks=pu.sample_blocks(wl, [0], 6, seed=5))


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
