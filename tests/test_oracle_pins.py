"""Pins for the CPU oracle: every part of it is checked against something other than itself
(closed forms, library routines, brute force, invariants).  No GPU needed."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def small_problem(seed, B=1, H=2, N=100, D=8, block=16, scale=1.0):
    g = rng(seed)
    q = (g.standard_normal((B, H, N, D)) * scale).astype(np.float32)
    k = (g.standard_normal((B, H, N, D)) * scale).astype(np.float32)
    v = g.standard_normal((B, H, N, D)).astype(np.float32)
    w = (g.standard_normal((H, D, D)) / math.sqrt(D)).astype(np.float32)
    return q, k, v, w


# ------------------------------------------------------------------ P1: e4m3 codec
def test_e4m3_landmarks_from_format_definition():
    table = orc.e4m3_value_table()
    with open(os.path.join(GOLDEN, "e4m3_landmarks.txt")) as fh:
        rows = [ln.split("#")[0].split() for ln in fh if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 10
    for code, value in rows:
        assert table[int(code, 16)] == float(value)
    assert np.isnan(table[0x7F]) and np.isnan(table[0xFF])
    finite = table[:0x7F]
    assert np.all(np.diff(finite) > 0)


def test_e4m3_decode_matches_torch_float8():
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    mine = orc.e4m3_value_table()
    ok = np.isnan(ref) == np.isnan(mine)
    assert ok.all()
    m = ~np.isnan(ref)
    assert np.array_equal(ref[m], mine[m])
    assert np.array_equal(np.signbit(ref[m]), np.signbit(mine[m]))


def test_e4m3_roundtrip_midpoints_saturation():
    table = orc.e4m3_value_table()
    codes = np.array([c for c in range(256) if not np.isnan(table[c])], dtype=np.uint8)
    assert np.array_equal(orc.e4m3_encode_rne(table[codes].astype(np.float32)), codes)
    pos = table[:0x7F]
    mids = (0.5 * (pos[:-1] + pos[1:])).astype(np.float32)  # exact in fp32
    got = orc.e4m3_encode_rne(mids)
    expect = np.array([c if c % 2 == 0 else c + 1 for c in range(0x7E)], dtype=np.uint8)  # even mantissa wins
    assert np.array_equal(got, expect)
    assert np.array_equal(orc.e4m3_encode_rne(-mids), expect | 0x80)
    # just off the midpoint goes to the nearer neighbour
    up = np.nextafter(mids, np.float32(np.inf))
    dn = np.nextafter(mids, np.float32(-np.inf))
    assert np.array_equal(orc.e4m3_encode_rne(up), np.arange(1, 0x7F, dtype=np.uint8))
    assert np.array_equal(orc.e4m3_encode_rne(dn), np.arange(0, 0x7E, dtype=np.uint8))
    assert orc.e4m3_encode_rne(np.float32(448.0)) == 0x7E
    assert orc.e4m3_encode_rne(np.float32(1e9)) == 0x7E
    assert orc.e4m3_encode_rne(np.float32(-1e9)) == 0xFE


def test_e4m3_encode_matches_torch_cast():
    g = rng(1)
    y = np.concatenate([
        g.uniform(-448, 448, 200000), g.standard_normal(200000) * 3, g.standard_normal(100000) * 0.02,
        np.linspace(-448, 448, 114689), np.array([0.0, -0.0, 1e-30, -1e-30, 448.0, -448.0])]).astype(np.float32)
    ref = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(orc.e4m3_encode_rne(y), ref)


# ------------------------------------------------------------------ quantiser
def test_quantizer_tile_by_tile_definition():
    """Re-derive each tile with scalar fp32 operations and torch's fp8 cast."""
    q, _, _, _ = small_problem(2, N=75, D=8, block=16, scale=3.0)
    codes, scales = orc.quantize_fp8_blocks(q, 16)
    B, H, N, D = q.shape
    assert codes.shape == (B, H, 80, D) and scales.shape == (B, H, 5)
    for h in range(H):
        for i in range(5):
            tile = q[0, h, i * 16:min(N, (i + 1) * 16)]
            amax = np.float32(np.abs(tile).max())
            s = np.float32(np.float32(amax + np.float32(1e-8)) / np.float32(448.0))
            assert scales[0, h, i] == s
            y = torch.from_numpy((tile / s).astype(np.float32)).clamp(-448, 448)
            ref = y.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
            assert np.array_equal(codes[0, h, i * 16:i * 16 + tile.shape[0]], ref)
    assert not codes[:, :, N:].any()  # padded tail is zero
    # the tile maximum lands on +-448 and the error obeys the format's half-ulp bound
    xhat = orc.dequantize(codes, scales, N, 16)
    tab = np.abs(orc.e4m3_decode(codes[:, :, :N]))
    assert (tab.reshape(B, H, -1).max(axis=2) == 448).all()
    ulp = np.where(tab < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(tab, 2.0 ** -6))) - 3))
    sc = np.repeat(scales.astype(np.float64), 16, axis=2)[:, :, :N, None]
    assert (np.abs(xhat - q) <= 0.5 * ulp * sc * (1 + 1e-6) + 1e-12).all()


def test_quantizer_zero_tile_and_outlier():
    x = np.zeros((1, 1, 32, 4), dtype=np.float32)
    x[0, 0, 20, 1] = 1000.0
    x[0, 0, 21, 2] = -0.5
    codes, scales = orc.quantize_fp8_blocks(x, 16)
    assert not codes[0, 0, :16].any()
    assert scales[0, 0, 0] == np.float32(np.float32(1e-8) / np.float32(448.0))
    assert codes[0, 0, 20, 1] == 0x7E
    assert scales[0, 0, 1] == np.float32(np.float32(1000.0) / np.float32(448.0))
    # -0.5 / (1000/448) = -0.224 -> nearest e4m3 value is -0.21875 (0x80|0x26)
    assert orc.e4m3_decode(codes[0, 0, 21, 2]) == -0.21875


def test_quantizer_power_of_two_invariance():
    q, _, _, _ = small_problem(3, N=64, D=8, block=16)
    c1, s1 = orc.quantize_fp8_blocks(q, 16)
    # the 1e-8 guard is absorbed by fp32 rounding once amax >= 0.25, so the scale is then exactly amax / 448
    for kpow in (-2, 5, 9):
        c2, s2 = orc.quantize_fp8_blocks(q * np.float32(2.0 ** kpow), 16)
        assert np.array_equal(c1, c2)
        assert np.array_equal(s2, s1 * np.float32(2.0 ** kpow))


# ------------------------------------------------------------------ helpers for the forward pins
def quantized(q, k, v, block):
    N = q.shape[2]
    out = []
    for x in (q, k, v):
        c, s = orc.quantize_fp8_blocks(x, block)
        out.append(orc.dequantize(c, s, N, block))
    return out


def dense_attention_torch(qh, kh, vh):
    t = [torch.from_numpy(np.ascontiguousarray(a)) for a in (qh, kh, vh)]
    return torch.nn.functional.scaled_dot_product_attention(*t).numpy()


# ------------------------------------------------------------------ P2: crit = 1 is dense attention
@pytest.mark.parametrize("N,block", [(96, 16), (100, 16), (70, 64)])
def test_all_critical_equals_dense_attention(N, block):
    q, k, v, w = small_problem(4, N=N, block=block)
    qh, kh, vh = quantized(q, k, v, block)
    cls = orc.classify(orc.pooled_scores(qh, kh, block), 1.0, 0.0)
    assert (cls == orc.CLASS_CRITICAL).all()
    out = orc.sla_forward(qh, kh, vh, w, cls, block)
    ref = dense_attention_torch(qh, kh, vh)
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ P3: crit = 0, neg = 0 is global linear attention
@pytest.mark.parametrize("phi", ["softmax", "elu1"])
def test_all_marginal_equals_linear_attention_closed_form(phi):
    q, k, v, w = small_problem(5, N=100, block=16)
    qh, kh, vh = quantized(q, k, v, 16)
    cls = orc.classify(orc.pooled_scores(qh, kh, 16), 0.0, 0.0)
    assert (cls == orc.CLASS_MARGINAL).all()
    out = orc.sla_forward(qh, kh, vh, w, cls, 16, phi=phi)
    tq, tk, tv, tw = (torch.from_numpy(np.ascontiguousarray(a)).double() for a in (qh, kh, vh, w))
    if phi == "softmax":
        fq, fk = torch.softmax(tq, -1), torch.softmax(tk, -1)
    else:
        fq, fk = torch.nn.functional.elu(tq) + 1, torch.nn.functional.elu(tk) + 1
    T = fk.transpose(-1, -2) @ tv  # phi(K)^T V   (Algorithm 1, KV summary)
    z = fk.sum(dim=-2)  # phi(K)^T 1   (normaliser)
    lin = (fq @ T) / (fq @ z.unsqueeze(-1))  # linear output
    ref = (lin @ tw.unsqueeze(0)).numpy()  # projection and sum with O_sparse = 0
    assert np.allclose(out, ref, rtol=1e-11, atol=1e-13)


# ------------------------------------------------------------------ P4: brute force per query token
def brute_force(qh, kh, vh, w, block, crit, neg, phi):
    """Scalar loops only: block means, ranking, then per query token explicit sums over keys."""
    B, H, N, D = qh.shape
    Nb = -(-N // block)
    k_c, k_m, k_n = orc.class_counts(Nb, crit, neg)

    def feat(x):
        if phi == "softmax":
            e = [math.exp(t - max(x)) for t in x]
            return [t / sum(e) for t in e]
        return [t + 1.0 if t > 0 else math.exp(t) for t in x]

    out = np.zeros((B, H, N, D))
    for b in range(B):
        for h in range(H):
            means = []
            for src in (qh, kh):
                mm = []
                for i in range(Nb):
                    toks = range(i * block, min(N, (i + 1) * block))
                    mm.append([sum(src[b, h, t, d] for t in toks) / len(toks) for d in range(D)])
                means.append(mm)
            fk = [feat(list(kh[b, h, s])) for s in range(N)]
            for i in range(Nb):
                sc = [sum(means[0][i][d] * means[1][j][d] for d in range(D)) / math.sqrt(D) for j in range(Nb)]
                order = sorted(range(Nb), key=lambda j: (-sc[j], j))
                crit_set, neg_set = set(order[:k_c]), set(order[Nb - k_n:] if k_n else [])
                for t in range(i * block, min(N, (i + 1) * block)):
                    keys_c = [s for s in range(N) if s // block in crit_set]
                    keys_m = [s for s in range(N) if s // block not in crit_set and s // block not in neg_set]
                    o = [0.0] * D
                    if keys_c:
                        logit = [sum(qh[b, h, t, d] * kh[b, h, s, d] for d in range(D)) / math.sqrt(D) for s in keys_c]
                        mx = max(logit)
                        e = [math.exp(x - mx) for x in logit]
                        for s, ws in zip(keys_c, e):
                            for d in range(D):
                                o[d] += ws / sum(e) * vh[b, h, s, d]
                    if keys_m:
                        fq = feat(list(qh[b, h, t]))
                        sim = [sum(fq[d] * fk[s][d] for d in range(D)) for s in keys_m]
                        lin = [sum(ws * vh[b, h, s, e_] for s, ws in zip(keys_m, sim)) / sum(sim) for e_ in range(D)]
                        for e_ in range(D):
                            o[e_] += sum(lin[d] * w[h, d, e_] for d in range(D))
                    out[b, h, t] = o
    return out


@pytest.mark.parametrize("N,D,block,crit,neg,phi", [
    (100, 4, 16, 0.3, 0.4, "softmax"),
    (100, 4, 16, 0.3, 0.4, "elu1"),
    (96, 6, 8, 0.25, 0.5, "softmax"),
    (37, 4, 8, 0.2, 0.8, "softmax"),  # no marginal blocks
    (37, 4, 8, 0.0, 0.4, "softmax"),  # no critical blocks
])
def test_forward_matches_brute_force(N, D, block, crit, neg, phi):
    q, k, v, w = small_problem(6, H=2, N=N, D=D, block=block, scale=1.5)
    qh, kh, vh = quantized(q, k, v, block)
    cls = orc.classify(orc.pooled_scores(qh, kh, block), crit, neg)
    out = orc.sla_forward(qh, kh, vh, w, cls, block, phi=phi)
    ref = brute_force(qh, kh, vh, w.astype(np.float64), block, crit, neg, phi)
    assert np.allclose(out, ref, rtol=1e-10, atol=1e-12)


# ------------------------------------------------------------------ P5: constant V
def test_constant_value_rows_give_c_plus_cW():
    q, k, v, w = small_problem(7, N=100, block=16)
    c = rng(70).standard_normal(v.shape[-1])
    qh, kh, _ = quantized(q, k, v, 16)
    vh = np.broadcast_to(c, qh.shape).copy()
    cls = orc.classify(orc.pooled_scores(qh, kh, 16), 0.3, 0.3)
    out = orc.sla_forward(qh, kh, vh, w, cls, 16)
    for h in range(out.shape[1]):
        expect = c + c @ w[h].astype(np.float64)
        assert np.allclose(out[0, h], expect, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ P6: summary normalisation
def test_softmax_phi_summaries_count_valid_tokens():
    q, k, v, w = small_problem(8, N=100, block=16)
    _, kh, vh = quantized(q, k, v, 16)
    Hs, zs = orc.kv_summaries(kh, vh, 16)
    counts = np.array([16] * 6 + [4], dtype=np.float64)
    assert np.allclose(zs.sum(axis=-1), counts[None, None], rtol=1e-13)
    # H_j against an explicit token loop for one block, orientation [d_key, d_value]
    j = 6
    ref = np.zeros((8, 8))
    for s in range(96, 100):
        e = np.exp(kh[0, 1, s] - kh[0, 1, s].max())
        ref += np.outer(e / e.sum(), vh[0, 1, s])
    assert np.allclose(Hs[0, 1, j], ref, rtol=1e-13, atol=1e-15)


def test_forward_uses_sum_of_marginal_summaries():
    q, k, v, w = small_problem(9, N=100, block=16)
    qh, kh, vh = quantized(q, k, v, 16)
    cls = orc.classify(orc.pooled_scores(qh, kh, 16), 0.3, 0.3)
    Hs, zs = orc.kv_summaries(kh, vh, 16)
    _, _, o_lin = orc.sla_forward(qh, kh, vh, w, cls, 16, parts=True)
    b, h, i = 0, 1, 3
    marg = np.flatnonzero(cls[b, h, i] == orc.CLASS_MARGINAL)
    G, zeta = Hs[b, h, marg].sum(axis=0), zs[b, h, marg].sum(axis=0)
    pq = orc.phi_softmax(qh[b, h, 48:64])
    assert np.allclose(o_lin[b, h, 48:64], (pq @ G) / (pq @ zeta)[:, None], rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ P7: order independence
def test_permuting_tokens_inside_key_blocks_changes_nothing():
    q, k, v, w = small_problem(10, N=96, block=16)
    qh, kh, vh = quantized(q, k, v, 16)
    cls = orc.classify(orc.pooled_scores(qh, kh, 16), 0.3, 0.3)
    out = orc.sla_forward(qh, kh, vh, w, cls, 16)
    perm = np.concatenate([j * 16 + rng(100 + j).permutation(16) for j in range(6)])
    cls2 = orc.classify(orc.pooled_scores(qh, kh[:, :, perm], 16), 0.3, 0.3)
    assert np.array_equal(cls, cls2) or np.allclose(
        orc.pooled_scores(qh, kh, 16), orc.pooled_scores(qh, kh[:, :, perm], 16), rtol=1e-13)
    out2 = orc.sla_forward(qh, kh[:, :, perm], vh[:, :, perm], w, cls, 16)
    assert np.allclose(out, out2, rtol=1e-11, atol=1e-13)


# ------------------------------------------------------------------ P8: block size 1 is token-level top-k
def test_block_one_equals_token_level_topk_attention():
    N, D, lam = 40, 8, 0.25
    q, k, v, w = small_problem(11, H=1, N=N, D=D, block=1)
    qh, kh, vh = quantized(q, k, v, 1)
    cls = orc.classify(orc.pooled_scores(qh, kh, 1), lam, 1.0 - lam)
    assert orc.class_counts(N, lam, 1.0 - lam) == (10, 0, 30)
    out = orc.sla_forward(qh, kh, vh, w, cls, 1)
    S = qh[0, 0] @ kh[0, 0].T / math.sqrt(D)  # Algorithm 1, scores
    ref = np.zeros((N, D))
    for t in range(N):
        keep = sorted(range(N), key=lambda s: (-S[t, s], s))[:10]  # TopKMask
        e = np.exp(S[t, keep] - S[t, keep].max())  # sparse softmax with masked entries excluded
        ref[t] = (e / e.sum()) @ vh[0, 0, keep]  # sparse output
    assert np.allclose(out[0, 0], ref, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ P9: classification
def test_class_counts_table():
    # (Nb, crit, neg) -> counts, from the configurations' block counts
    assert orc.class_counts(8, 0.25, 0.50) == (2, 2, 4)
    assert orc.class_counts(172, 0.10, 0.60) == (17, 52, 103)
    assert orc.class_counts(687, 0.05, 0.75) == (34, 138, 515)
    assert orc.class_counts(172, 0.08, 0.70) == (14, 38, 120)
    assert orc.class_counts(2147, 0.02, 0.60) == (43, 816, 1288)
    assert orc.class_counts(2147, 0.25, 0.60) == (537, 322, 1288)
    assert orc.class_counts(2147, 1.0, 0.0) == (2147, 0, 0)
    assert orc.class_counts(10, 0.01, 0.0) == (1, 9, 0)  # non-zero fraction keeps one block
    assert orc.class_counts(10, 0.0, 1.0) == (0, 0, 10)
    assert orc.class_counts(10, 0.6, 0.9) == (6, 0, 4)  # critical has priority
    assert orc.class_counts(2, 0.25, 0.0) == (1, 1, 0)  # 0.5 rounds half up


def test_classification_partitions_and_orders_rows():
    g = rng(12)
    s = g.standard_normal((2, 3, 23, 23))
    cls = orc.classify(s, 0.2, 0.5)
    k_c, k_m, k_n = orc.class_counts(23, 0.2, 0.5)
    assert ((cls == 2).sum(-1) == k_c).all() and ((cls == 1).sum(-1) == k_m).all() and ((cls == 0).sum(-1) == k_n).all()
    big = np.where(cls == 2, s, np.inf).min(-1)
    mid_hi = np.where(cls == 1, s, -np.inf).max(-1)
    mid_lo = np.where(cls == 1, s, np.inf).min(-1)
    low = np.where(cls == 0, s, -np.inf).max(-1)
    assert (big >= mid_hi).all() and (mid_lo >= low).all()
    crit_idx, marg_idx = orc.index_lists(cls)
    assert crit_idx.shape[-1] == k_c and marg_idx.shape[-1] == k_m
    assert (np.diff(crit_idx, axis=-1) > 0).all() and (np.diff(marg_idx, axis=-1) > 0).all()


def test_ties_go_to_lower_key_block_index():
    s = np.array([[[[1.0, 3.0, 3.0, 3.0, 0.5, 0.5, 0.5, 0.5]]]])
    cls = orc.classify(np.repeat(s, 8, axis=2), 0.25, 0.375)  # k_c=2, k_n=3
    assert cls[0, 0, 0].tolist() == [1, 2, 2, 1, 1, 0, 0, 0]


def test_pooled_scores_use_valid_tokens_only():
    q, k, v, w = small_problem(13, H=1, N=20, D=4, block=16)
    qh, kh, _ = quantized(q, k, v, 16)
    sc = orc.pooled_scores(qh, kh, 16)
    ref = (qh[0, 0, 16:20].sum(0) / 4) @ (kh[0, 0, :16].sum(0) / 16) / 2.0
    assert np.isclose(sc[0, 0, 1, 0], ref, rtol=1e-13)


def test_subset_of_query_blocks_and_external_plan():
    q, k, v, w = small_problem(14, N=100, block=16)
    full = orc.sla_forward_from_source(q, k, v, w, 16, 0.3, 0.3)
    part = orc.sla_forward_from_source(q, k, v, w, 16, 0.3, 0.3, cls=full["cls"], query_blocks=[(0, 1, 6), (0, 0, 0)])
    assert np.array_equal(part["out"][0, 1, 96:], full["out"][0, 1, 96:])
    assert np.array_equal(part["out"][0, 0, :16], full["out"][0, 0, :16])
    assert np.isnan(part["out"][0, 0, 16:]).all()


# ------------------------------------------------------------------ the composed path used by every GPU parity test
def torch_quantize(x, block):
    """Independent quantiser: scalar fp32 scale per tile, torch's float8_e4m3fn cast, decode through torch's view."""
    B, H, N, D = x.shape
    nb = -(-N // block)
    codes = np.zeros((B, H, nb * block, D), dtype=np.uint8)
    scales = np.zeros((B, H, nb), dtype=np.float32)
    xhat = np.zeros((B, H, N, D))
    for b in range(B):
        for h in range(H):
            for i in range(nb):
                sl = slice(i * block, min(N, (i + 1) * block))
                tile = x[b, h, sl]
                s = np.float32(np.float32(np.float32(np.abs(tile).max()) + np.float32(1e-8)) / np.float32(448.0))
                f8 = torch.from_numpy((tile / s).astype(np.float32)).clamp(-448, 448).to(torch.float8_e4m3fn)
                codes[b, h, sl] = f8.view(torch.uint8).numpy()
                scales[b, h, i] = s
                xhat[b, h, sl] = f8.to(torch.float64).numpy() * float(s)
    return codes, scales, xhat


@pytest.mark.parametrize("phi", ["softmax", "elu1"])
def test_from_source_composition_against_independent_pieces(phi):
    """sla_forward_from_source (the function the GPU parity tests take their expected values from) against pieces that
    do not come from the oracle: torch's cast for the codes, the scalar brute force (which pools, ranks and sums on
    its own) for the output.  K and V have visibly different magnitudes and crit != neg, so swapped operands,
    swapped fractions or a wrong block size cannot pass."""
    block, crit, neg = 16, 0.3, 0.15
    q, k, v, w = small_problem(21, H=2, N=100, D=4, block=block, scale=1.5)
    k = (k * np.float32(3.0)).astype(np.float32)
    v = (v * np.float32(0.2) + np.float32(0.7)).astype(np.float32)
    res = orc.sla_forward_from_source(q, k, v, w, block, crit, neg, phi=phi)
    indep = {n: torch_quantize(x, block) for n, x in (("q", q), ("k", k), ("v", v))}
    for n in ("q", "k", "v"):
        codes, scales, xhat = indep[n]
        assert np.array_equal(res[n + "_codes"], codes)
        assert np.array_equal(res[n + "_scales"], scales)
        assert np.array_equal(res[n + "hat"], xhat)
    # the three quantised tensors are different things
    assert not np.array_equal(res["k_scales"], res["v_scales"]) and not np.array_equal(res["q_scales"], res["k_scales"])
    qh, kh, vh = indep["q"][2], indep["k"][2], indep["v"][2]
    nb = -(-100 // block)
    # scores: explicit block means of the valid tokens
    for (h, i, j) in ((0, 0, 0), (1, 6, 2), (0, 3, 6), (1, 6, 6)):
        mq = qh[0, h, i * block:min(100, (i + 1) * block)].mean(axis=0)
        mk = kh[0, h, j * block:min(100, (j + 1) * block)].mean(axis=0)
        assert np.isclose(res["scores"][0, h, i, j], float(mq @ mk) / 2.0, rtol=1e-12)
    assert not np.allclose(res["scores"], np.swapaxes(res["scores"], -1, -2))
    # classes: the counts of these fractions, critical = the largest scores
    k_c, k_m, k_n = orc.class_counts(nb, crit, neg)
    assert (k_c, k_m, k_n) == (2, 4, 1)
    for h in range(2):
        for i in range(nb):
            order = sorted(range(nb), key=lambda j: (-res["scores"][0, h, i, j], j))
            assert set(np.flatnonzero(res["cls"][0, h, i] == 2)) == set(order[:k_c])
            assert set(np.flatnonzero(res["cls"][0, h, i] == 0)) == set(order[nb - k_n:])
    ref = brute_force(qh, kh, vh, w.astype(np.float64), block, crit, neg, phi)
    assert np.allclose(res["out"], ref, rtol=1e-10, atol=1e-12)
    # and the brute force with the fractions swapped is a different answer (the test would notice the swap)
    swapped = brute_force(qh, kh, vh, w.astype(np.float64), block, neg, crit, phi)
    assert not np.allclose(res["out"], swapped, rtol=1e-3, atol=1e-3)


# ------------------------------------------------------------------ FP8 linear layer (Algorithm 2)
def test_row_quantizer_against_torch_cast():
    g = rng(31)
    x = (g.standard_normal((37, 48)) * g.uniform(0.01, 30.0, size=(37, 1))).astype(np.float32)
    x[5] = 0.0
    x[6, 3] = 1.0e4
    codes, scales = orc.quantize_fp8_rows(x)
    for i in range(x.shape[0]):
        s = np.float32(np.float32(np.float32(np.abs(x[i]).max()) + np.float32(1e-8)) / np.float32(448.0))
        assert scales[i] == s
        ref = torch.from_numpy((x[i] / s).astype(np.float32)).clamp(-448, 448).to(torch.float8_e4m3fn)
        assert np.array_equal(codes[i], ref.view(torch.uint8).numpy())
    assert not codes[5].any() and codes[6, 3] == 0x7E
    # every non-zero row reaches +-448, and a power-of-two factor per row only moves the scale
    assert (np.abs(orc.e4m3_decode(codes[np.abs(x).max(axis=1) > 0])).max(axis=1) == 448).all()
    factor = np.float32(2.0) ** g.integers(-3, 6, size=(37, 1)).astype(np.float32)
    c2, s2 = orc.quantize_fp8_rows(x * factor)
    keep = np.abs(x).max(axis=1) >= 0.25  # the 1e-8 guard is absorbed from there on
    assert np.array_equal(c2[keep], codes[keep]) and np.array_equal(s2[keep], (scales * factor[:, 0])[keep])


def test_fp8_linear_against_torch_matmul_and_scalar_loops():
    g = rng(32)
    N, din, dout = 23, 40, 17
    x = g.standard_normal((N, din)).astype(np.float32) * 3
    w = (g.standard_normal((dout, din)) / math.sqrt(din)).astype(np.float32)
    b = g.standard_normal(dout).astype(np.float32)
    xc, xs = orc.quantize_fp8_rows(x)
    wc, ws = orc.quantize_fp8_rows(w)
    y = orc.linear_fp8(xc, xs, wc, ws, b)
    # library routine on operands dequantised through torch's float8 view
    xq = torch.from_numpy(xc).view(torch.float8_e4m3fn).to(torch.float64) * torch.from_numpy(xs.astype(np.float64))[:, None]
    wq = torch.from_numpy(wc).view(torch.float8_e4m3fn).to(torch.float64) * torch.from_numpy(ws.astype(np.float64))[:, None]
    ref = torch.nn.functional.linear(xq, wq, torch.from_numpy(b.astype(np.float64))).numpy()
    assert np.allclose(y, ref, rtol=1e-13, atol=1e-13)
    # scalar loops, scales applied outside the integer-like sum as a kernel would
    tab = orc.e4m3_value_table()
    for (n, o) in ((0, 0), (22, 16), (7, 3)):
        acc = sum(float(tab[xc[n, k]]) * float(tab[wc[o, k]]) for k in range(din))
        assert np.isclose(y[n, o], acc * float(xs[n]) * float(ws[o]) + float(b[o]), rtol=1e-12)
    # not symmetric in its operands, and the quantised product stays close to the unquantised one
    assert y.shape == (N, dout)
    exact = x.astype(np.float64) @ w.astype(np.float64).T + b
    assert np.abs(y - exact).max() < 0.08 * np.abs(exact).max()
    assert np.allclose(orc.linear_fp8(xc, xs, wc, ws), y - b[None, :], rtol=1e-12, atol=1e-12)


def test_qkv_projection_layout_and_identity_weight():
    """Output rows are ordered (q | k | v) x head x D; with a weight that copies input channels, each head's q / k /
    v is the per-token-quantised input slice times the (exactly representable) weight."""
    g = rng(33)
    B, N, H, D = 2, 19, 3, 4
    dm = H * D
    x = g.standard_normal((B, N, dm)).astype(np.float32)
    w = np.zeros((3 * H * D, dm), dtype=np.float32)
    for part, gain in enumerate((1.0, 2.0, -0.5)):
        for o in range(H * D):
            w[part * H * D + o, o] = gain
    q, k, v, ops = orc.qkv_project_fp8(x, w, H)
    assert q.shape == (B, H, N, D)
    xq = orc.dequantize_rows(ops["x_codes"], ops["x_scales"]).reshape(B, N, H, D).transpose(0, 2, 1, 3)
    # a weight row with a single entry g dequantises to sign(g) * 448 * scale_row (its code is +-448), g up to fp32 rounding
    gq = [math.copysign(448.0 * float(ops["w_scales"][part * H * D]), gain) for part, gain in enumerate((1.0, 2.0, -0.5))]
    assert all(abs(a / b - 1.0) < 1e-6 for a, b in zip(gq, (1.0, 2.0, -0.5)))
    assert np.allclose(q, gq[0] * xq, rtol=1e-12, atol=0) and np.allclose(k, gq[1] * xq, rtol=1e-12, atol=0)
    assert np.allclose(v, gq[2] * xq, rtol=1e-12, atol=0)
    # a general weight: equals the plain linear layer reshaped
    w2 = (g.standard_normal((3 * H * D, dm)) / 3).astype(np.float32)
    q2, k2, v2, ops2 = orc.qkv_project_fp8(x, w2, H)
    y = orc.linear_fp8(ops2["x_codes"], ops2["x_scales"], ops2["w_codes"], ops2["w_scales"])
    assert np.array_equal(k2[1, 2, 5], y[1 * N + 5, H * D + 2 * D:H * D + 3 * D])
    assert np.array_equal(v2[0, 0, 18], y[18, 2 * H * D:2 * H * D + D])


# ------------------------------------------------------------------ training side of proj_lin (Eq. 3, selective freezing)
def test_mse_distill_against_torch_autograd():
    g = rng(41)
    a = torch.from_numpy(g.standard_normal((2, 3, 17, 8))).requires_grad_(True)
    t = torch.from_numpy(g.standard_normal((2, 3, 17, 8)))
    loss = torch.nn.functional.mse_loss(a, t)
    loss.backward()
    mine_loss, mine_grad = orc.mse_distill(a.detach().numpy(), t.numpy())
    assert np.isclose(mine_loss, float(loss), rtol=1e-14)
    assert np.allclose(mine_grad, a.grad.numpy(), rtol=1e-13, atol=0)
    assert orc.mse_distill(t.numpy(), t.numpy())[0] == 0.0


def test_proj_lin_gradient_by_finite_differences():
    """dW = O_lin^T dO pinned against what it must be the derivative of: the distillation loss of the whole SLA
    forward as a function of W, differentiated numerically (central differences) on a small problem.  The loss is
    quadratic in W, so central differences are exact up to round-off."""
    q, k, v, w = small_problem(42, H=2, N=70, D=4, block=16)
    qh, kh, vh = quantized(q, k, v, 16)
    cls = orc.classify(orc.pooled_scores(qh, kh, 16), 0.25, 0.25)
    teacher = rng(43).standard_normal(qh.shape)
    w = w.astype(np.float64)
    out, o_sp, o_li = orc.sla_forward(qh, kh, vh, w, cls, 16, parts=True)
    loss, d_out = orc.mse_distill(out, teacher)
    dw = orc.proj_lin_backward(o_li, d_out)
    assert dw.shape == w.shape
    eps = 1e-4
    for (h, i, j) in ((0, 0, 0), (1, 3, 2), (0, 2, 3), (1, 1, 1)):
        wp, wm = w.copy(), w.copy()
        wp[h, i, j] += eps
        wm[h, i, j] -= eps
        lp = orc.mse_distill(orc.sla_forward(qh, kh, vh, wp, cls, 16), teacher)[0]
        lm = orc.mse_distill(orc.sla_forward(qh, kh, vh, wm, cls, 16), teacher)[0]
        assert np.isclose((lp - lm) / (2 * eps), dw[h, i, j], rtol=1e-7, atol=1e-12), (h, i, j)
    # against the library routine and a transposed-operand mistake
    ref = torch.einsum("bhtd,bhte->hde", torch.from_numpy(o_li), torch.from_numpy(d_out)).numpy()
    assert np.allclose(dw, ref, rtol=1e-13, atol=1e-15)
    assert not np.allclose(dw, np.swapaxes(dw, 1, 2), rtol=1e-3, atol=1e-9)
