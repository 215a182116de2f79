"""Seeded synthetic inputs shaped like the multi-view attention workloads.

This module only draws random numbers and lays them out; it contains none of
the attention method's arithmetic (no quantisation, pooling, softmax or
feature map).  Both the CPU oracle's tests and the CUDA path's tests feed on
the arrays produced here, which is the only thing the two sides share.

Token layout: a sequence is ``frames`` consecutive frames of 1374 tokens
(1 camera + 4 register tokens, then 37 x 37 patch tokens), the per-frame token
count of the VGGT / Depth-Anything-3 backbones.  The paper's image datasets and
pretrained weights are not available, so query/key vectors are drawn from a
Gaussian cluster model instead: every token position inside a frame is tied to
one of ``centres`` cluster centres (the same centres in every frame and for
both Q and K) and receives independent Gaussian noise, which makes blocks at
the same position of different frames correlate the way cross-view
correspondences do.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

TOKENS_PER_FRAME = 1374  # 37*37 patches + 1 camera + 4 register tokens
SPECIAL_TOKENS = 5
PATCH_TOKENS = TOKENS_PER_FRAME - SPECIAL_TOKENS
SEED_BASE = 113540


@dataclass(frozen=True)
class Workload:
    """One benchmark/parity configuration."""

    name: str
    cfg_id: int
    batch: int
    heads: int
    tokens: int
    head_dim: int
    block: int
    crit: float
    neg: float
    centres: int  # 0 = iid N(0,1) queries/keys (no cluster structure)
    sigma: float
    src_dtype: str  # "f32" or "bf16"

    @property
    def n_blocks(self) -> int:
        return -(-self.tokens // self.block)

    @property
    def dense_equiv_flops(self) -> float:
        return 4.0 * self.batch * self.heads * float(self.tokens) ** 2 * self.head_dim


WORKLOADS = {
    "tiny": Workload("tiny", 1, 1, 2, 512, 64, 64, 0.25, 0.50, 0, 0.0, "f32"),
    "vggt8": Workload("vggt8", 2, 1, 16, 8 * TOKENS_PER_FRAME, 64, 64, 0.10, 0.60, 64, 0.3, "bf16"),
    "vggt32": Workload("vggt32", 3, 1, 16, 32 * TOKENS_PER_FRAME, 64, 64, 0.05, 0.75, 64, 0.3, "bf16"),
    "da3l": Workload("da3l", 4, 4, 16, 16 * TOKENS_PER_FRAME, 64, 128, 0.08, 0.70, 128, 0.5, "bf16"),
    "stress100": Workload("stress100", 5, 1, 16, 100 * TOKENS_PER_FRAME, 64, 64, 0.10, 0.60, 64, 0.3, "bf16"),
    # frame attention: every frame is a sequence of its own (batch = frames), 22 blocks of 64 tokens, the last one
    # with 30; the short-sequence regime where launch, plan and ragged-block costs weigh most
    "frame32": Workload("frame32", 6, 32, 16, TOKENS_PER_FRAME, 64, 64, 0.25, 0.50, 64, 0.3, "bf16"),
}
STRESS_SWEEP = ((0.02, 0.60), (0.05, 0.60), (0.10, 0.60), (0.25, 0.60), (1.00, 0.00))


def scaled_down(wl: Workload, *, heads: int | None = None, tokens: int | None = None,
                batch: int | None = None) -> Workload:
    """Same recipe on a smaller shape (used to keep CPU-side checks short)."""
    return replace(wl, heads=heads or wl.heads, tokens=tokens or wl.tokens,
                   batch=batch or wl.batch, name=wl.name + "-cut")


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays fp32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of fp32 values that are already bf16-representable."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return (u >> np.uint32(16)).astype(np.uint16)


def centre_of_token(tokens: int, centres: int) -> np.ndarray:
    """Cluster-centre index of every token position of a sequence."""
    p = np.arange(tokens, dtype=np.int64) % TOKENS_PER_FRAME
    patch = np.clip(p - SPECIAL_TOKENS, 0, None) * centres // PATCH_TOKENS
    return np.where(p < SPECIAL_TOKENS, p % centres, patch).astype(np.int64)


def make_inputs(wl: Workload) -> dict:
    """Draw q, k, v of shape [B, H, N, D] and proj of shape [H, D, D] (fp32 arrays).

    For ``src_dtype == "bf16"`` the q/k/v values are exactly representable in
    bf16 (use :func:`bf16_bits` for the 16-bit patterns).  ``proj`` is fp32.
    """
    s_centres, s_qn, s_kn, s_v, s_proj = np.random.SeedSequence(SEED_BASE + wl.cfg_id).spawn(5)
    B, H, N, D = wl.batch, wl.heads, wl.tokens, wl.head_dim
    shape = (B, H, N, D)

    def normal(seq, shp):
        return np.random.Generator(np.random.PCG64(seq)).standard_normal(shp, dtype=np.float32)

    v = normal(s_v, shape)
    proj = normal(s_proj, (H, D, D)) * np.float32(1.0 / np.sqrt(D))
    if wl.centres == 0:
        q = normal(s_qn, shape)
        k = normal(s_kn, shape)
    else:
        c = normal(s_centres, (H, wl.centres, D))
        base = c[:, centre_of_token(N, wl.centres), :]  # [H, N, D], shared by the batch
        q = normal(s_qn, shape)
        q *= np.float32(wl.sigma)
        q += base[None]
        k = normal(s_kn, shape)
        k *= np.float32(wl.sigma)
        k += base[None]
    if wl.src_dtype == "bf16":
        q, k, v = round_to_bf16(q), round_to_bf16(k), round_to_bf16(v)
    return {"q": q, "k": k, "v": v, "proj": proj.astype(np.float32)}
