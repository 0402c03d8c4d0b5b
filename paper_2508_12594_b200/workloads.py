"""Seeded synthetic inputs for the FLARE token mixer.

This module holds input recipes only: it draws latent queries, keys, values,
padding masks and upstream gradients with the shapes and value distributions
of the five benchmark workloads.  It contains none of the mixer's arithmetic
(no scores, no softmax, no contraction), so both the CPU oracle's tests and
the CUDA path's tests may import it without sharing any part of the method.

Layouts (the C-ABI's):  Q_lat [H, M, D];  K, V, dY [B, N, H, D];
key_mask [B, N] uint8 (1 = valid token, 0 = padding).

Every tensor is drawn in fp32 from a ``torch.Generator`` on the CPU seeded
with the workload's seed and then cast once to the workload dtype; the cast
values are what every consumer sees.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """One problem shape.  ``kind`` selects how K and V are drawn."""

    name: str
    B: int
    H: int
    N: int
    M: int
    D: int
    dtype: str          # "f32" | "bf16" | "f16"
    kind: str           # "iid" | "cloud2d" | "padded" | "cube" | "scaled"
    seed: int
    backward: bool = False
    scale: float = 1.0  # the paper's mixer uses s = 1 in both stages (Section 3.2)

    @property
    def tokens(self) -> int:
        return self.B * self.N

    def torch_dtype(self) -> torch.dtype:
        return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[self.dtype]

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five benchmark workloads.  "sweep" is a family: see sweep_point().
CONFIGS = {
    "tiny": Workload("tiny", B=1, H=2, N=1024, M=16, D=16, dtype="f32", kind="iid", seed=0),
    "mesh2d": Workload("mesh2d", B=4, H=8, N=65536, M=64, D=16, dtype="bf16", kind="cloud2d", seed=2),
    "padded": Workload("padded", B=32, H=4, N=4096, M=128, D=32, dtype="bf16", kind="padded", seed=3,
                       backward=True),
    "mesh3d_1m": Workload("mesh3d_1m", B=1, H=8, N=1048576, M=256, D=16, dtype="bf16", kind="cube", seed=4),
    # the shape of the paper's own million-point study (field-prediction appendix): C = 64, H = 8, hence D = 8,
    # with M between 128 and 2048 latents; not one of the five benchmark workloads
    "field_1m": Workload("field_1m", B=1, H=8, N=1048576, M=1024, D=8, dtype="bf16", kind="cube", seed=6, backward=True),
}

SWEEP_N = (16384, 131072, 1048576)
SWEEP_M = (32, 128, 512)


def sweep_point(N: int, M: int) -> Workload:
    """One (N, M) point of the training-step sweep (B=1, H=8, D=32, bf16)."""
    return Workload(f"sweep_N{N}_M{M}", B=1, H=8, N=N, M=M, D=32, dtype="bf16", kind="scaled", seed=5,
                    backward=True)


@dataclasses.dataclass
class Inputs:
    Q: torch.Tensor                    # [H, M, D]
    K: torch.Tensor                    # [B, N, H, D]
    V: torch.Tensor                    # [B, N, H, D]
    key_mask: Optional[torch.Tensor]   # [B, N] uint8 or None
    dY: Optional[torch.Tensor]         # [B, N, H, D] or None


def _projected_features(g: torch.Generator, B: int, N: int, C: int, coords: torch.Tensor):
    """Token features [coords | N(0,1) channels] of width 128 projected to K and V of width C.

    The projection weights are N(0, 1/128) (variance 1/128), drawn once per call and shared
    by all batch items; the products are formed in fp32.
    """
    F = 128
    ncoord = coords.shape[-1]
    X = torch.empty(B, N, F, dtype=torch.float32)
    X[..., :ncoord] = coords
    X[..., ncoord:] = torch.randn(B, N, F - ncoord, generator=g, dtype=torch.float32)
    Wk = torch.randn(F, C, generator=g, dtype=torch.float32) * (1.0 / F) ** 0.5
    Wv = torch.randn(F, C, generator=g, dtype=torch.float32) * (1.0 / F) ** 0.5
    return X @ Wk, X @ Wv


def make_inputs(w: Workload) -> Inputs:
    """Draw the inputs of workload ``w`` (CPU tensors, already cast to ``w.dtype``)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    B, H, N, M, D = w.B, w.H, w.N, w.M, w.D
    C = H * D
    dt = w.torch_dtype()
    Q = torch.randn(H, M, D, generator=g, dtype=torch.float32)
    mask = None
    if w.kind == "iid":
        K = torch.randn(B, N, C, generator=g, dtype=torch.float32)
        V = torch.randn(B, N, C, generator=g, dtype=torch.float32)
    elif w.kind == "cloud2d":
        # unstructured 2-D point cloud: xy ~ U(0,1)^2 per token, fresh per batch item
        xy = torch.rand(B, N, 2, generator=g, dtype=torch.float32)
        K, V = _projected_features(g, B, N, C, xy)
    elif w.kind == "cube":
        # points uniform on the surface of the unit cube: pick a face, two free coordinates
        face = torch.randint(0, 6, (B, N), generator=g)
        uv = torch.rand(B, N, 2, generator=g, dtype=torch.float32)
        axis = face // 2                       # which coordinate is pinned
        side = (face % 2).to(torch.float32)    # pinned to 0 or 1
        xyz = torch.zeros(B, N, 3, dtype=torch.float32)
        for a in range(3):
            free = [c for c in range(3) if c != a]
            sel = axis == a
            xyz[..., a] = torch.where(sel, side, xyz[..., a])
            xyz[..., free[0]] = torch.where(sel, uv[..., 0], xyz[..., free[0]])
            xyz[..., free[1]] = torch.where(sel, uv[..., 1], xyz[..., free[1]])
        K, V = _projected_features(g, B, N, C, xyz)
    elif w.kind in ("padded", "scaled"):
        K = torch.randn(B, N, C, generator=g, dtype=torch.float32) / D ** 0.5
        V = torch.randn(B, N, C, generator=g, dtype=torch.float32) / D ** 0.5
        if w.kind == "padded":
            # a random 10 % of the token indices of each batch item are padding
            npad = N // 10
            mask = torch.ones(B, N, dtype=torch.uint8)
            for b in range(B):
                idx = torch.randperm(N, generator=g)[:npad]
                mask[b, idx] = 0
            keep = mask.to(torch.float32).unsqueeze(-1)
            K = K * keep
            V = V * keep
    else:
        raise ValueError(f"unknown workload kind {w.kind!r}")
    K = K.reshape(B, N, H, D).to(dt).contiguous()
    V = V.reshape(B, N, H, D).to(dt).contiguous()
    Q = Q.to(dt).contiguous()
    dY = None
    if w.backward:
        dY = torch.randn(B, N, H, D, generator=g, dtype=torch.float32).to(dt).contiguous()
    return Inputs(Q=Q, K=K, V=V, key_mask=mask, dY=dY)


def make_random(B, H, N, M, D, dtype="f32", seed=0, masked_fraction=0.0, with_dy=False,
                k_std=1.0, q_std=1.0) -> Inputs:
    """Small i.i.d. Gaussian case for edge-shape tests; optional random padding mask."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    dt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[dtype]
    Q = (torch.randn(H, M, D, generator=g) * q_std).to(dt)
    K = (torch.randn(B, N, H, D, generator=g) * k_std).to(dt)
    V = torch.randn(B, N, H, D, generator=g).to(dt)
    mask = None
    if masked_fraction > 0.0:
        mask = (torch.rand(B, N, generator=g) >= masked_fraction).to(torch.uint8)
    dY = torch.randn(B, N, H, D, generator=g).to(dt) if with_dy else None
    return Inputs(Q=Q.contiguous(), K=K.contiguous(), V=V.contiguous(), key_mask=mask, dY=dY)
