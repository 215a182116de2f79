"""CPU oracle for the FP8 Sparse Linear Attention (SLA) forward.  TEST INFRASTRUCTURE.

A plain, slow, fp64 restatement of what the method computes, written from the
paper's definition (Eq. 1 and Algorithm 1 for the attention, the appendix
"FP8 E4M3 Format" / "Scaled FP8 Quantization" equations for the quantiser) in
the block-level form this library implements.  It shares no code with the CUDA
path and is imported only by the tests, the smoke check and the benchmark's
CPU-baseline leg; the product never routes through it.

Conventions
-----------
* Tensors are ``[B, H, N, D]`` (batch, heads, tokens, head_dim); a *block* is
  ``block`` consecutive tokens of one (b, h); ``Nb = ceil(N / block)``; the last
  block may be ragged and only its valid tokens take part in anything.
* The quantiser's three operations (scale, divide, clamp) run in fp32 because
  the paper's quantiser is an fp32 program whose integer result must be
  reproduced bit for bit; everything after the codes is fp64.
* The FP8 linear layer in front of the attention (per-token / per-output-row scaled e4m3 operands, Algorithm 2 in its
  deployed form) follows the same rule: scale, divide and clamp in fp32, the product in fp64.
* Pins (checked in tests/test_oracle_pins.py): the e4m3 codec against the
  closed-form format definition and torch's float8_e4m3fn cast; crit=1 against
  dense softmax attention; crit=0,neg=0 against the global linear-attention
  closed form (Algorithm 1, its linear branch, projection and sum); brute-force per-query evaluation on
  tiny inputs; constant-V, phi-summary and permutation invariants; block=1
  against Algorithm 1's score, mask and sparse-softmax steps evaluated per token.  Beyond those pins the
  output values of the general three-class case rest on the definition itself
  (the paper prints no worked numeric example): parity unpinned past the pins.
"""
from __future__ import annotations

import math

import numpy as np

FP8_MAX = 448.0  # appendix "Scaled FP8 Quantization": FP8_MAX = 448
SCALE_EPS = 1e-8  # appendix "Implementation Details": epsilon added to scale factors

CLASS_NEGLIGIBLE, CLASS_MARGINAL, CLASS_CRITICAL = 0, 1, 2


# --------------------------------------------------------------------------- e4m3 format
def e4m3_value_table() -> np.ndarray:
    """Value of each of the 256 e4m3 ("fn") codes: 1 sign, 4 exponent, 3 mantissa bits,
    bias 7, subnormals at exponent field 0, no infinities, S.1111.111 is NaN
    (appendix "FP8 E4M3 Format")."""
    table = np.empty(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e = (code >> 3) & 0xF
        m = code & 0x7
        if e == 0:
            mag = 2.0 ** -6 * (m / 8.0)
        elif e == 15 and m == 7:
            mag = float("nan")
        else:
            mag = 2.0 ** (e - 7) * (1.0 + m / 8.0)
        table[code] = sign * mag
    return table


_TABLE = e4m3_value_table()
_POS = _TABLE[:0x7F].copy()  # codes 0x00..0x7E: 0 .. 448 ascending


def e4m3_encode_rne(y: np.ndarray) -> np.ndarray:
    """Cast finite values to e4m3 codes: nearest representable value, ties to the code
    with an even mantissa, saturating at +-448 (never the NaN code); the sign bit
    follows the sign of the input even when the magnitude rounds to zero."""
    y = np.asarray(y)
    a = np.minimum(np.abs(y).astype(np.float64), FP8_MAX)
    hi = np.searchsorted(_POS, a, side="left")  # smallest code whose value >= a
    lo = np.maximum(hi - 1, 0)
    mid = 0.5 * (_POS[lo] + _POS[hi])  # exact: both are multiples of 2**-9
    pick_hi = (a > mid) | ((a == mid) & ((hi & 1) == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return code | (np.signbit(y).astype(np.uint8) << 7)


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    return _TABLE[np.asarray(codes, dtype=np.uint8)]


# --------------------------------------------------------------------------- quantiser
def n_blocks(tokens: int, block: int) -> int:
    return -(-tokens // block)


def quantize_fp8_blocks(x: np.ndarray, block: int):
    """Scaled FP8 quantisation with one scale per (b, h, token-block) tile of block x D.

    Appendix "Scaled FP8 Quantization": scale = max|x| / 448 (plus the 1e-8 guard of
    "Implementation Details", applied as (amax + 1e-8) / 448), x_scaled = clamp(x / scale,
    -448, 448), code = FP8(x_scaled).  All three steps in fp32.

    Returns (codes uint8 [B,H,Nb*block,D] with the padded tail zero, scales fp32 [B,H,Nb]).
    """
    x = np.asarray(x, dtype=np.float32)
    B, H, N, D = x.shape
    Nb = n_blocks(N, block)
    xp = np.zeros((B, H, Nb * block, D), dtype=np.float32)
    xp[:, :, :N] = x
    tiles = xp.reshape(B, H, Nb, block, D)
    amax = np.abs(tiles).max(axis=(3, 4)).astype(np.float32)
    scales = ((amax + np.float32(SCALE_EPS)) / np.float32(FP8_MAX)).astype(np.float32)
    y = (tiles / scales[:, :, :, None, None]).astype(np.float32)
    y = np.minimum(np.maximum(y, np.float32(-FP8_MAX)), np.float32(FP8_MAX))
    codes = e4m3_encode_rne(y).reshape(B, H, Nb * block, D)
    codes[:, :, N:] = 0
    return codes, scales


def dequantize(codes: np.ndarray, scales: np.ndarray, tokens: int, block: int) -> np.ndarray:
    """x_hat = value(code) * scale in fp64 (exact), valid tokens only: [B,H,N,D]."""
    B, H, Np, D = codes.shape
    Nb = Np // block
    vals = e4m3_decode(codes).reshape(B, H, Nb, block, D)
    vals = vals * scales.astype(np.float64)[:, :, :, None, None]
    return vals.reshape(B, H, Np, D)[:, :, :tokens]


# --------------------------------------------------------------------------- plan
def block_means(xhat: np.ndarray, block: int) -> np.ndarray:
    """Mean over the valid tokens of each block: [B,H,Nb,D]."""
    B, H, N, D = xhat.shape
    Nb = n_blocks(N, block)
    out = np.empty((B, H, Nb, D), dtype=np.float64)
    for i in range(Nb):
        out[:, :, i] = xhat[:, :, i * block:min(N, (i + 1) * block)].mean(axis=2)
    return out


def pooled_scores(qhat: np.ndarray, khat: np.ndarray, block: int) -> np.ndarray:
    """Compressed scores s_ij = (mean_i(q) . mean_j(k)) / sqrt(D): [B,H,Nb,Nb]
    (the score step of Algorithm 1 applied to block means)."""
    D = qhat.shape[-1]
    return np.einsum("bhid,bhjd->bhij", block_means(qhat, block), block_means(khat, block)) / math.sqrt(D)


def class_counts(nb: int, crit: float, neg: float):
    """(k_crit, k_marg, k_neg) key blocks per query block.  Fractions of Nb are rounded
    half up; a non-zero critical fraction keeps at least one block; critical has
    priority over negligible."""
    k_c = 0 if crit == 0 else min(nb, max(1, int(math.floor(crit * nb + 0.5))))
    k_n = min(nb - k_c, int(math.floor(neg * nb + 0.5)))
    return k_c, nb - k_c - k_n, k_n


def classify(scores: np.ndarray, crit: float, neg: float) -> np.ndarray:
    """Row-wise top-k (the TopKMask step of Algorithm 1, per query block): rank the key blocks of each row
    by score descending, ties to the lower key-block index; the first k_crit are critical (2),
    the last k_neg negligible (0), the rest marginal (1).  Returns int8 [B,H,Nb,Nb]."""
    nb = scores.shape[-1]
    k_c, _, k_n = class_counts(nb, crit, neg)
    order = np.argsort(-scores, axis=-1, kind="stable")
    rank = np.empty_like(order)
    np.put_along_axis(rank, order, np.broadcast_to(np.arange(nb), order.shape), axis=-1)
    cls = np.full(scores.shape, CLASS_MARGINAL, dtype=np.int8)
    cls[rank < k_c] = CLASS_CRITICAL
    cls[rank >= nb - k_n] = CLASS_NEGLIGIBLE
    return cls


def index_lists(cls: np.ndarray):
    """Ascending key-block indices of the critical and of the marginal blocks of every row.
    Every row must hold the same counts.  Returns (int32 [B,H,Nb,k_c], int32 [B,H,Nb,k_m])."""
    B, H, Nb, _ = cls.shape
    k_c = int((cls[0, 0, 0] == CLASS_CRITICAL).sum())
    k_m = int((cls[0, 0, 0] == CLASS_MARGINAL).sum())
    crit = np.empty((B, H, Nb, k_c), dtype=np.int32)
    marg = np.empty((B, H, Nb, k_m), dtype=np.int32)
    for b in range(B):
        for h in range(H):
            for i in range(Nb):
                crit[b, h, i] = np.flatnonzero(cls[b, h, i] == CLASS_CRITICAL)
                marg[b, h, i] = np.flatnonzero(cls[b, h, i] == CLASS_MARGINAL)
    return crit, marg


# --------------------------------------------------------------------------- feature maps
def phi_softmax(x: np.ndarray) -> np.ndarray:
    """Feature map of the benchmark contract: softmax over the head_dim components."""
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def phi_elu1(x: np.ndarray) -> np.ndarray:
    """Feature map of Algorithm 1: ELU(x) + 1."""
    return np.where(x > 0, x + 1.0, np.exp(np.minimum(x, 0.0)))


PHI = {"softmax": phi_softmax, "elu1": phi_elu1}


# --------------------------------------------------------------------------- linear-branch summaries
def kv_summaries(khat: np.ndarray, vhat: np.ndarray, block: int, phi: str = "softmax"):
    """Per key block j: H_j = phi(K_j)^T V_j [D,D] and z_j = phi(K_j)^T 1 [D]
    (the KV-summary and normaliser steps of Algorithm 1 restricted to one block), valid tokens only."""
    B, H, N, D = khat.shape
    Nb = n_blocks(N, block)
    f = PHI[phi]
    Hs = np.empty((B, H, Nb, D, D), dtype=np.float64)
    zs = np.empty((B, H, Nb, D), dtype=np.float64)
    for j in range(Nb):
        sl = slice(j * block, min(N, (j + 1) * block))
        pk = f(khat[:, :, sl])
        Hs[:, :, j] = np.einsum("bhsd,bhse->bhde", pk, vhat[:, :, sl])
        zs[:, :, j] = pk.sum(axis=2)
    return Hs, zs


# --------------------------------------------------------------------------- forward
def sla_forward(qhat, khat, vhat, proj, cls, block, phi="softmax", query_blocks=None, parts=False):
    """A_SLA = A_sparse + Proj(A_lin) (Eq. 1), block-level classes taken from ``cls``.

    qhat/khat/vhat: dequantised fp64 [B,H,N,D]; proj: [H,D,D] (or [D,D] shared), applied as
    O_lin @ W (the projection-and-sum step of Algorithm 1, no bias); cls: int8 [B,H,Nb,Nb].
    For the query tokens of block i of (b, h):
      sparse branch (Algorithm 1's masked softmax and its product with V): softmax over exactly the valid keys of the critical blocks of
        (q . k) / sqrt(D), times V; zero when there is no critical block;
      linear branch (Algorithm 1's feature map, summaries and normalised output) over the valid keys of the marginal blocks only:
        (phi(q) G_i) / (phi(q) . zeta_i) with G_i, zeta_i the sums of the per-block
        summaries; zero when there is no marginal block.
    ``query_blocks``: iterable of (b, h, i) to evaluate (default all).  Returns fp64 [B,H,N,D]
    (rows of blocks not evaluated stay NaN); with ``parts`` also (O_sparse, O_lin)."""
    B, H, N, D = qhat.shape
    Nb = n_blocks(N, block)
    f = PHI[phi]
    proj = np.asarray(proj, dtype=np.float64)
    if proj.ndim == 2:
        proj = np.broadcast_to(proj, (H, D, D))
    out = np.full((B, H, N, D), np.nan)
    o_sp = np.full((B, H, N, D), np.nan)
    o_li = np.full((B, H, N, D), np.nan)
    if query_blocks is None:
        query_blocks = [(b, h, i) for b in range(B) for h in range(H) for i in range(Nb)]
    inv_sqrt_d = 1.0 / math.sqrt(D)

    def tokens_of(blocks):
        return np.concatenate([np.arange(j * block, min(N, (j + 1) * block)) for j in blocks])

    for (b, h, i) in query_blocks:
        rows = slice(i * block, min(N, (i + 1) * block))
        q = qhat[b, h, rows]
        crit = np.flatnonzero(cls[b, h, i] == CLASS_CRITICAL)
        marg = np.flatnonzero(cls[b, h, i] == CLASS_MARGINAL)
        if crit.size:
            t = tokens_of(crit)
            s = (q @ khat[b, h, t].T) * inv_sqrt_d
            p = np.exp(s - s.max(axis=1, keepdims=True))
            sparse = (p / p.sum(axis=1, keepdims=True)) @ vhat[b, h, t]
        else:
            sparse = np.zeros_like(q)
        if marg.size:
            t = tokens_of(marg)
            pk = f(khat[b, h, t])
            G = pk.T @ vhat[b, h, t]  # = sum over marginal blocks of H_j
            zeta = pk.sum(axis=0)  # = sum of z_j
            pq = f(q)
            lin = (pq @ G) / (pq @ zeta)[:, None]
        else:
            lin = np.zeros_like(q)
        o_sp[b, h, rows] = sparse
        o_li[b, h, rows] = lin
        out[b, h, rows] = sparse + lin @ proj[h]
    return (out, o_sp, o_li) if parts else out


def sla_forward_from_source(q, k, v, proj, block, crit, neg, phi="softmax", cls=None, query_blocks=None):
    """Whole path from unquantised fp32 sources: quantise, plan (unless ``cls`` is given), forward.
    Returns a dict of every intermediate the parity tests compare."""
    qc, qs = quantize_fp8_blocks(q, block)
    kc, ks = quantize_fp8_blocks(k, block)
    vc, vs = quantize_fp8_blocks(v, block)
    N = q.shape[2]
    qhat, khat, vhat = (dequantize(c, s, N, block) for c, s in ((qc, qs), (kc, ks), (vc, vs)))
    scores = pooled_scores(qhat, khat, block)
    if cls is None:
        cls = classify(scores, crit, neg)
    out = sla_forward(qhat, khat, vhat, proj, cls, block, phi, query_blocks)
    return {"q_codes": qc, "q_scales": qs, "k_codes": kc, "k_scales": ks, "v_codes": vc, "v_scales": vs,
            "qhat": qhat, "khat": khat, "vhat": vhat, "scores": scores, "cls": cls, "out": out}


# --------------------------------------------------------------------------- FP8 linear layer (Algorithm 2, deployed form)
def quantize_fp8_rows(x: np.ndarray):
    """Scaled FP8 quantisation with one scale per row of a matrix [R, C]: per token for activations, per output
    row for weights (appendix "Per-Tensor Dynamic Scaling").  scale_i = (max_j |x_ij| + 1e-8) / 448, codes =
    e4m3(clamp(x / scale, -448, 448)); the three steps in fp32 as in quantize_fp8_blocks.
    Returns (codes uint8 [R, C], scales fp32 [R])."""
    x = np.asarray(x, dtype=np.float32)
    amax = np.abs(x).max(axis=1).astype(np.float32)
    scales = ((amax + np.float32(SCALE_EPS)) / np.float32(FP8_MAX)).astype(np.float32)
    y = (x / scales[:, None]).astype(np.float32)
    y = np.minimum(np.maximum(y, np.float32(-FP8_MAX)), np.float32(FP8_MAX))
    return e4m3_encode_rne(y), scales


def dequantize_rows(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """value(code) * scale of its row, fp64 (exact)."""
    return e4m3_decode(codes) * scales.astype(np.float64)[:, None]


def linear_fp8(x_codes, x_scales, w_codes, w_scales, bias=None) -> np.ndarray:
    """y = x_q W_q^T + b (the linear transformation of Algorithm 2) on the quantised operands: x_q [N, d_in] with
    per-token scales, W_q [d_out, d_in] with per-output-row scales.  fp64 [N, d_out]."""
    y = dequantize_rows(x_codes, x_scales) @ dequantize_rows(w_codes, w_scales).T
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y


def qkv_project_fp8(x, w_qkv, heads: int, bias=None):
    """The qkv projection of an attention block as an FP8 linear layer (Eq. 2: W_q = Q_fp8(W), X_q = Q_fp8(X),
    Y = Linear(X_q, W_q)): x [B, N, d_model], w_qkv [3 * heads * D, d_model] with the output rows ordered
    (q | k | v) x head x D.  Returns (q, k, v) fp64 [B, heads, N, D] and the quantised operands."""
    x = np.asarray(x, dtype=np.float32)
    B, N, dm = x.shape
    xc, xs = quantize_fp8_rows(x.reshape(B * N, dm))
    wc, ws = quantize_fp8_rows(w_qkv)
    y = linear_fp8(xc, xs, wc, ws, bias)
    D = w_qkv.shape[0] // (3 * heads)
    y = y.reshape(B, N, 3, heads, D)
    q, k, v = (np.ascontiguousarray(y[:, :, i].transpose(0, 2, 1, 3)) for i in range(3))
    return q, k, v, {"x_codes": xc, "x_scales": xs, "w_codes": wc, "w_scales": ws}


# --------------------------------------------------------------------------- training side of proj_lin (Sec. 3.3, Eq. 3)
def mse_distill(student: np.ndarray, teacher: np.ndarray):
    """One module's term of the partial attention distillation loss (Eq. 3): MSE(A_student, stopgrad(A_teacher)) =
    mean over all elements of (A_s - A_t)^2, and its gradient with respect to the student output,
    2 (A_s - A_t) / numel.  fp64."""
    s = np.asarray(student, dtype=np.float64)
    t = np.asarray(teacher, dtype=np.float64)
    d = s - t
    return float((d * d).mean()), 2.0 * d / d.size


def proj_lin_backward(o_lin: np.ndarray, d_out: np.ndarray) -> np.ndarray:
    """Gradient of a loss with respect to the linear-branch projection W (the only trained tensor, Sec. 3.3
    "selective freezing"): the output is O = O_sparse + O_lin W_h per head (Algorithm 1's last step), so
    dL/dW_h = sum over batch and tokens of O_lin[b,h,t,:]^T dO[b,h,t,:].  o_lin, d_out: [B,H,N,D]; returns [H,D,D]."""
    return np.einsum("bhtd,bhte->hde", np.asarray(o_lin, dtype=np.float64), np.asarray(d_out, dtype=np.float64))
