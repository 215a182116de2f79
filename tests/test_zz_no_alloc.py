"""The allocation-free forward (`lite3r_sla_forward_static_scratch`) against the regular entry point.

Callers that cannot allocate device memory where they call the library (plug-ins inside another runtime's
pre-planned arena, allocator-free real-time loops) use the variant whose scratch is a fixed array inside the
library.  It must give the same output as `lite3r_sla_forward`, also when called twice in a row on the array
the previous call left dirty, and must refuse shapes that do not fit its 32 MiB limit.
This file sorts last so that every other test has already run if it fails."""
import numpy as np
import pytest
import torch

from paper_2605_11354_b200 import binding as lt
from paper_2605_11354_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu


def prepared(wl):
    inputs = wk.make_inputs(wl)
    eng, out = pu.run_gpu(inputs, wl)
    proj = torch.from_numpy(inputs["proj"]).cuda()
    return eng, out.clone(), proj


@pytest.mark.parametrize("name,heads", [("tiny", 2), ("vggt8", 2)])
def test_static_scratch_matches_regular_forward_twice(name, heads):
    wl = wk.scaled_down(wk.WORKLOADS[name], heads=heads)
    eng, expected, proj = prepared(wl)
    assert lt.lite3r_forward_workspace(eng.shape, wl.crit, wl.neg) <= lt.STATIC_SCRATCH_BYTES
    ref = expected.cpu().numpy().astype(np.float64)
    free_after_first = None
    for call in range(3):
        out = torch.full_like(expected, float("nan"))
        lt.lite3r_sla_forward_static_scratch(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, out,
                                             eng.status)
        torch.cuda.synchronize()
        # the first call on a device may make CUDA load the array; every later call must leave the device's free
        # memory exactly where it was (nothing allocated, nothing freed)
        free_now = torch.cuda.mem_get_info()[0]
        if call >= 1:
            assert free_now == free_after_first, (call, free_now, free_after_first)
        free_after_first = free_now
        assert int(eng.status.item()) == 0
        rel, mx = pu.output_errors(out.cpu().numpy(), ref)
        assert rel <= pu.REL_L2_TOL and mx <= pu.MAX_ABS_TOL, (call, rel, mx)
        assert torch.equal(out, expected), f"call {call}: not bit-identical to lite3r_sla_forward"
    # a different problem in between leaves other contents in the shared array; the next call must not care
    other = wk.scaled_down(wk.WORKLOADS["tiny"], heads=1)
    eng2, expected2, proj2 = prepared(other)
    out2 = torch.empty_like(expected2)
    lt.lite3r_sla_forward_static_scratch(eng2.q8, eng2.k8, eng2.v8, proj2, eng2.shape, eng2.phi, eng2.plan, out2)
    out = torch.empty_like(expected)
    lt.lite3r_sla_forward_static_scratch(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, out)
    torch.cuda.synchronize()
    assert torch.equal(out2, expected2) and torch.equal(out, expected)


def test_static_scratch_rejects_oversized_shapes():
    wl = wk.scaled_down(wk.WORKLOADS["vggt8"], heads=8)  # 1376 tiles > the 1344 that fit in 32 MiB
    eng = lt.SlaForward(wl.batch, wl.heads, wl.tokens, wl.block, wl.crit, wl.neg)
    assert lt.lite3r_forward_workspace(eng.shape, wl.crit, wl.neg) > lt.STATIC_SCRATCH_BYTES
    proj = torch.zeros((wl.heads, 64, 64), device="cuda")
    with pytest.raises(lt.Lite3rError, match="workspace too small"):
        lt.lite3r_sla_forward_static_scratch(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, eng.out)


@pytest.mark.parametrize("blocks,fits", [(1012, True), (1013, False)])
def test_static_scratch_limit_at_block_128(blocks, fits):
    """At block 128 a tile takes more scratch (the fp16 copy of V doubles): 1012 tiles fit, 1013 do not."""
    wl = wk.Workload("limit128", cfg_id=91, batch=1, heads=1, tokens=blocks * 128 - 5, head_dim=64, block=128,
                     crit=0.01, neg=0.9, centres=8, sigma=0.3, src_dtype="bf16")
    if not fits:
        eng = lt.SlaForward(wl.batch, wl.heads, wl.tokens, wl.block, wl.crit, wl.neg)
        proj = torch.zeros((1, 64, 64), device="cuda")
        with pytest.raises(lt.Lite3rError, match="workspace too small"):
            lt.lite3r_sla_forward_static_scratch(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, eng.out)
        return
    eng, expected, proj = prepared(wl)
    out = torch.empty_like(expected)
    lt.lite3r_sla_forward_static_scratch(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, out, eng.status)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0 and torch.equal(out, expected)


def test_static_scratch_sixteen_bit_output():
    wl = wk.scaled_down(wk.WORKLOADS["tiny"], heads=2)
    eng, expected, proj = prepared(wl)
    out = torch.empty(expected.shape, dtype=torch.bfloat16, device="cuda")
    lt.lite3r_sla_forward_static_scratch(eng.q8, eng.k8, eng.v8, proj, eng.shape, eng.phi, eng.plan, out, eng.status)
    torch.cuda.synchronize()
    assert torch.equal(out, expected.to(torch.bfloat16))
