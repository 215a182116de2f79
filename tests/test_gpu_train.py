"""Parity of the training side of the linear-branch projection (linear branch alone, MSE distillation term and its
gradient, gradient of the projection) against the CPU oracle, through the C-ABI binding."""
import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc
from paper_2605_11354_b200 import binding as lt
from paper_2605_11354_b200 import workloads as wk

import parity_util as pu
from test_gpu_parity import oracle_subset, small_workload

pytestmark = pytest.mark.gpu


def aligned_bytes(nbytes):
    raw = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    off = (-raw.data_ptr()) % 256
    return raw[off:off + nbytes]


@pytest.mark.parametrize("block,phi,tokens", [(64, "softmax", 1000), (128, "softmax", 700), (64, "elu1", 333)])
def test_linear_branch_alone(block, phi, tokens):
    wl = small_workload(f"olin-{block}-{phi}", tokens=tokens, block=block, heads=2, batch=2)
    inputs = wk.make_inputs(wl)
    eng, _ = pu.run_gpu(inputs, wl, phi=phi)
    ws = aligned_bytes(lt.lite3r_train_workspace(eng.shape, wl.crit, wl.neg))
    o_lin = torch.full((wl.batch, wl.heads, wl.tokens, 64), float("nan"), device="cuda")
    lt.lite3r_sla_linear_branch(eng.q8, eng.k8, eng.v8, eng.shape, eng.phi, eng.plan, o_lin, ws, eng.status)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    ref = oracle_subset(inputs, wl, [0, 1], phi=phi, cls=eng.plan.cls.cpu().numpy(), query_blocks=[])
    _, _, o_li = orc.sla_forward(ref["qhat"], ref["khat"], ref["vhat"], inputs["proj"], eng.plan.cls.cpu().numpy(), block,
                                 phi, parts=True)
    rel, mx = pu.output_errors(o_lin.cpu().numpy(), o_li)
    print(f"O_lin {block} {phi}: rel_l2={rel:.3e} max_abs={mx:.3e}")
    assert rel <= pu.REL_L2_TOL and mx <= pu.MAX_ABS_TOL


@pytest.mark.parametrize("dtype,count", [(torch.float32, 8 * 12345), (torch.bfloat16, 8 * 70001), (torch.float32, 8)])
def test_mse_distillation_term(dtype, count):
    g = np.random.default_rng(7)
    s = g.standard_normal(count).astype(np.float32)
    t = (s + 0.3 * g.standard_normal(count)).astype(np.float32)
    if dtype == torch.bfloat16:
        s, t = wk.round_to_bf16(s), wk.round_to_bf16(t)
    ds = pu.to_device(s, "bf16" if dtype == torch.bfloat16 else "f32")
    dt = pu.to_device(t, "bf16" if dtype == torch.bfloat16 else "f32")
    grad = torch.empty(count, dtype=torch.bfloat16, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = aligned_bytes(16384)
    lt.lite3r_mse_distill(ds, dt, grad, loss, ws)
    torch.cuda.synchronize()
    ref_loss, ref_grad = orc.mse_distill(s, t)
    # differences and their squares are fp32 on the device, the sum is fp64: 1e-6 relative covers the fp32 squares
    assert abs(float(loss.item()) - ref_loss) <= 1e-6 * ref_loss
    got = grad.float().cpu().numpy().astype(np.float64)
    assert (np.abs(got - ref_grad) <= 2.0 ** -8 * np.abs(ref_grad) + 1e-30).all()  # bf16 rounding of the gradient


@pytest.mark.parametrize("batch,heads,tokens", [(2, 3, 1000), (1, 2, 64), (1, 1, 7), (3, 2, 4111)])
def test_projection_gradient(batch, heads, tokens):
    """d_proj = O_lin^T dO against the oracle on the same bf16 operands: the products are exact in fp32, only the
    accumulation order differs (1e-5 of the largest entry)."""
    g = np.random.default_rng(8)
    o = wk.round_to_bf16(g.standard_normal((batch, heads, tokens, 64)).astype(np.float32))
    d = wk.round_to_bf16((g.standard_normal((batch, heads, tokens, 64)) / tokens).astype(np.float32))
    shape = lt.Shape(batch, heads, tokens, 64, 64)
    ws = aligned_bytes(lt.lite3r_train_workspace(shape, 0.1, 0.5))
    dw = torch.full((heads, 64, 64), float("nan"), device="cuda")
    status = torch.ones(1, dtype=torch.int32, device="cuda")
    lt.lite3r_proj_lin_backward(pu.to_device(o, "bf16"), pu.to_device(d, "bf16"), shape, dw, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = orc.proj_lin_backward(o, d)
    got = dw.cpu().numpy().astype(np.float64)
    assert np.abs(got - ref).max() <= 1e-5 * np.abs(ref).max()
    again = torch.empty_like(dw)
    lt.lite3r_proj_lin_backward(pu.to_device(o, "bf16"), pu.to_device(d, "bf16"), shape, again, ws, status)
    torch.cuda.synchronize()
    assert torch.equal(again, dw)  # fixed summation order


def test_one_distillation_step_end_to_end():
    """Forward, MSE term against a teacher output, gradient of the projection: the chain a training step of the
    method runs through this library, against the same chain in the oracle."""
    wl = small_workload("distill", tokens=900, heads=2, batch=1)
    inputs = wk.make_inputs(wl)
    eng, out = pu.run_gpu(inputs, wl)
    g = np.random.default_rng(9)
    teacher_np = (out.cpu().numpy() + 0.1 * g.standard_normal(out.shape)).astype(np.float32)
    teacher = torch.from_numpy(teacher_np).cuda()
    ws = aligned_bytes(lt.lite3r_train_workspace(eng.shape, wl.crit, wl.neg))
    o_lin = torch.empty(out.shape, dtype=torch.bfloat16, device="cuda")
    lt.lite3r_sla_linear_branch(eng.q8, eng.k8, eng.v8, eng.shape, eng.phi, eng.plan, o_lin, ws, eng.status)
    grad = torch.empty(out.shape, dtype=torch.bfloat16, device="cuda")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    lt.lite3r_mse_distill(out.contiguous(), teacher, grad, loss, ws)
    dw = torch.empty((wl.heads, 64, 64), device="cuda")
    lt.lite3r_proj_lin_backward(o_lin, grad, eng.shape, dw, ws, eng.status)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    ref = oracle_subset(inputs, wl, [0, 1], cls=eng.plan.cls.cpu().numpy(), query_blocks=[])
    r_out, _, r_lin = orc.sla_forward(ref["qhat"], ref["khat"], ref["vhat"], inputs["proj"], eng.plan.cls.cpu().numpy(),
                                      wl.block, parts=True)
    r_loss, r_grad = orc.mse_distill(r_out, teacher_np)
    r_dw = orc.proj_lin_backward(r_lin, r_grad)
    assert abs(float(loss.item()) - r_loss) <= 2e-3 * r_loss
    got = dw.cpu().numpy().astype(np.float64)
    rel = np.sqrt(((got - r_dw) ** 2).sum() / (r_dw ** 2).sum())
    print(f"dW rel_l2={rel:.3e}")
    assert rel <= 1e-2  # bf16 operands (2^-9 each) and the forward's own 2e-3 enter the gradient
