"""Shared pieces of the GPU parity tests: upload seeded inputs, run the CUDA path through the C-ABI binding,
run the oracle on the same arrays, and compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import sla_oracle as orc
from paper_2605_11354_b200 import binding as lt
from paper_2605_11354_b200 import workloads as wk

REL_L2_TOL = 2e-3  # output tolerance of the benchmark contract
MAX_ABS_TOL = 1e-2
TIE_TOL = 1e-6  # class flips are tolerated only between pooled scores closer than this


def to_device(x: np.ndarray, src_dtype: str, device="cuda:0") -> torch.Tensor:
    if src_dtype == "bf16":
        bits = torch.from_numpy(wk.bf16_bits(x).view(np.int16)).to(device)
        return bits.view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(device)


def colsum_units(codes: np.ndarray, block: int) -> np.ndarray:
    """Per-tile column sums of the oracle's code values in units of 2^-9 (exact integers)."""
    B, H, Np, D = codes.shape
    vals = np.rint(orc.e4m3_decode(codes) * 512.0).astype(np.int64)
    return vals.reshape(B, H, Np // block, block, D).sum(axis=3)


def run_gpu(inputs: dict, wl, phi="softmax", crit=None, neg=None, device="cuda:0"):
    crit = wl.crit if crit is None else crit
    neg = wl.neg if neg is None else neg
    eng = lt.SlaForward(wl.batch, wl.heads, wl.tokens, wl.block, crit, neg, phi=phi, device=device)
    q, k, v = (to_device(inputs[n], wl.src_dtype, device) for n in ("q", "k", "v"))
    proj = torch.from_numpy(inputs["proj"]).to(device)
    out = eng.run(q, k, v, proj)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    return eng, out


def compare_plan(eng, oracle_scores: np.ndarray, oracle_cls: np.ndarray, heads=None):
    """Bit-exact class matrix except where the differing entries' oracle scores lie within TIE_TOL of the
    class boundary they straddle; returns the number of such tie flips.  Also checks the index lists."""
    cls = eng.plan.cls.cpu().numpy()
    crit_idx = eng.plan.crit_idx.cpu().numpy()
    marg_idx = eng.plan.marg_idx.cpu().numpy()
    if heads is not None:
        cls, crit_idx, marg_idx = cls[:, heads], crit_idx[:, heads], marg_idx[:, heads]
    flips = 0
    diff = np.argwhere((cls != oracle_cls).any(axis=-1))
    for (b, h, i) in diff:
        row_g, row_o, s = cls[b, h, i], oracle_cls[b, h, i], oracle_scores[b, h, i]
        for c in (0, 1, 2):
            assert (row_g == c).sum() == (row_o == c).sum()
        bad = np.flatnonzero(row_g != row_o)
        # every misplaced entry must be within TIE_TOL of an entry of the class it was swapped with
        for j in bad:
            partners = bad[row_g[bad] == row_o[j]]
            assert partners.size and np.abs(s[partners] - s[j]).min() <= TIE_TOL, (b, h, i, j)
        flips += bad.size
    # index lists of EVERY row: ascending positions of the class in the GPU's own class matrix
    for lists, c in ((crit_idx, orc.CLASS_CRITICAL), (marg_idx, orc.CLASS_MARGINAL)):
        k = lists.shape[-1]
        if k == 0:
            continue
        member = cls == c
        assert (member.sum(axis=-1) == k).all()
        # nonzero walks rows in order and columns ascending, so a reshape gives the expected lists
        expected = np.nonzero(member)[-1].reshape(*cls.shape[:-1], k)
        assert np.array_equal(lists, expected)
    return flips, cls


def output_errors(got: np.ndarray, ref: np.ndarray):
    mask = ~np.isnan(ref)
    d = got[mask].astype(np.float64) - ref[mask]
    ref_sq = float((ref[mask] ** 2).sum())
    rel_l2 = float(np.sqrt((d ** 2).sum() / ref_sq)) if ref_sq > 0 else float(np.abs(d).max() > 0)
    return rel_l2, float(np.abs(d).max())


def sample_blocks(wl, heads, count, seed=0):
    """Seeded sample of query blocks: block 0, the (possibly ragged) last block and one block per head always."""
    g = np.random.default_rng(seed)
    nb = wl.n_blocks
    picks = {(0, heads[0], 0), (wl.batch - 1, heads[-1], nb - 1)}
    for h in heads:
        picks.add((int(g.integers(wl.batch)), h, int(g.integers(nb))))
    while len(picks) < count:
        picks.add((int(g.integers(wl.batch)), int(g.choice(heads)), int(g.integers(nb))))
    return sorted(picks)
