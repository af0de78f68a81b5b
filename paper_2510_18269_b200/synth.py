"""Seeded synthetic kv streams shaped like LLaVA-OV kv-caches.

This module only draws random tensors; it contains none of the method's
arithmetic (no quantization, no means over tokens, no scoring).  Both the CUDA
tests and the CPU oracle's tests take their inputs from here, so that they see
the same bytes.

Recipe (per layer l, kv head h):
  * four "outlier" key channels are drawn once per (l, h) from the seed and
    every key value in those channels is scaled by 10;
  * K ~ N(0,1) (then outlier scaling), V ~ N(0,1);
  * a direction u[l, h, :] ~ N(0,1) is drawn; every query token of every query
    head of the GQA block of h is u[l, h, :] + q_noise * N(0,1);
  * `n_planted` groups per layer are overwritten with keys u[l, h, :] +
    0.1 * N(0,1) (every token of the group), so that retrieval has known
    strong matches while the remaining selections are decided by small score
    differences among ordinary groups.
Tensors are generated in the storage dtype (bf16 / fp16 / fp32) so that what
is consumed is exactly what is returned.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

DTYPES = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}


@dataclass
class Shape:
    """Geometry of one workload (names follow the paper: L, H_q, H_k, d, G, T, T_q, k)."""
    name: str
    L: int
    H_q: int
    H_k: int
    d: int
    G: int
    T: int            # stored groups (frames)
    T_q: int
    k: int
    dtype: str = "bf16"
    N_in: int = 0     # tokens per frame before the keep-mask (0: frames arrive already reduced to G)
    q_noise: float = 0.25
    seed: int = 0
    extra: dict = field(default_factory=dict)


# The five workloads of the benchmark definition (shapes only; values are synthetic).
C1 = Shape("C1-tiny", L=1, H_q=1, H_k=1, d=128, G=16, T=64, T_q=1, k=4, dtype="fp32", q_noise=0.0, seed=0)
C2 = Shape("C2-7B-layer", L=1, H_q=28, H_k=4, d=128, G=50, T=1024, T_q=8, k=32, seed=1236)
C3 = Shape("C3-7B-2h", L=28, H_q=28, H_k=4, d=128, G=50, T=7200, T_q=16, k=64, seed=1237)
C4 = Shape("C4-7B-interleave", L=28, H_q=28, H_k=4, d=128, G=50, T=3600, T_q=16, k=64, N_in=196, seed=1238)
C5 = Shape("C5-72B", L=80, H_q=64, H_k=8, d=128, G=50, T=3600, T_q=32, k=64, seed=1239)
CONFIGS = {s.name.split("-")[0]: s for s in (C1, C2, C3, C4, C5)}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def outlier_channels(shape: Shape, device="cpu") -> torch.Tensor:
    """[L][H_k][4] int64 channel ids, fixed by the seed (drawn on the CPU so every device agrees)."""
    g = _gen(shape.seed * 7919 + 1, "cpu")
    ids = torch.stack([torch.randperm(shape.d, generator=g)[:4] for _ in range(shape.L * shape.H_k)])
    return ids.view(shape.L, shape.H_k, 4).to(device)


def direction(shape: Shape, device="cpu") -> torch.Tensor:
    """u [L][H_k][d] float32 (drawn on the CPU so every device agrees)."""
    g = _gen(shape.seed * 7919 + 2, "cpu")
    return torch.randn(shape.L, shape.H_k, shape.d, generator=g).to(device)


def planted_groups(shape: Shape, n_planted: int | None = None) -> torch.Tensor:
    """[L][n_planted] int64 group ids per layer, sorted ascending."""
    n = shape.k // 2 if n_planted is None else n_planted
    if shape.name.startswith("C1"):
        n = shape.k if n_planted is None else n_planted
    g = _gen(shape.seed * 7919 + 3, "cpu")
    rows = [torch.sort(torch.randperm(shape.T, generator=g)[:n]).values for _ in range(shape.L)]
    return torch.stack(rows)


def queries(shape: Shape, device="cpu") -> torch.Tensor:
    """Q [L][H_q][T_q][d] in the storage dtype."""
    u = direction(shape, device)
    rep = shape.H_q // shape.H_k
    base = u.repeat_interleave(rep, dim=1)[:, :, None, :].expand(shape.L, shape.H_q, shape.T_q, shape.d)
    g = _gen(shape.seed * 7919 + 4, device)
    noise = torch.randn(shape.L, shape.H_q, shape.T_q, shape.d, generator=g, device=device)
    return (base + shape.q_noise * noise).to(DTYPES[shape.dtype]).contiguous()


def kv_chunk(shape: Shape, layer: int, frame_begin: int, frame_count: int, device="cpu",
             planted: torch.Tensor | None = None):
    """K, V for frames [frame_begin, frame_begin+frame_count) of one layer.

    Returns two tensors [frame_count][H_k][tokens][d] in the storage dtype,
    tokens = N_in if the shape has a keep-mask, else G.  Each (layer, frame)
    has its own generator state, so a chunk does not depend on how the stream
    was cut into chunks only through `frame_begin`/`frame_count` of THIS call.
    """
    tokens = shape.N_in or shape.G
    dt = DTYPES[shape.dtype]
    g = _gen((shape.seed * 1000003 + layer) * 1000003 + frame_begin, device)
    K = torch.randn(frame_count, shape.H_k, tokens, shape.d, generator=g, device=device)
    V = torch.randn(frame_count, shape.H_k, tokens, shape.d, generator=g, device=device)
    out = outlier_channels(shape, device)[layer]                     # [H_k][4]
    scale = torch.ones(shape.H_k, shape.d, device=device)
    scale.scatter_(1, out, 10.0)
    K = K * scale[None, :, None, :]
    if planted is None:
        planted = planted_groups(shape)
    ids = planted[layer]
    ids = ids[(ids >= frame_begin) & (ids < frame_begin + frame_count)] - frame_begin
    if ids.numel():
        u = direction(shape, device)[layer]                          # [H_k][d]
        noise = torch.randn(ids.numel(), shape.H_k, tokens, shape.d, generator=g, device=device)
        K[ids.to(device)] = u[None, :, None, :] + 0.1 * noise
    return K.to(dt).contiguous(), V.to(dt).contiguous()


def kv_stream(shape: Shape, device="cpu", frame_chunk: int = 256):
    """Whole stream: K, V [L][T][H_k][tokens][d] in the storage dtype (allocated once, filled in chunks)."""
    tokens = shape.N_in or shape.G
    dt = DTYPES[shape.dtype]
    K = torch.empty(shape.L, shape.T, shape.H_k, tokens, shape.d, dtype=dt, device=device)
    V = torch.empty_like(K)
    planted = planted_groups(shape)
    for l in range(shape.L):
        for f0 in range(0, shape.T, frame_chunk):
            n = min(frame_chunk, shape.T - f0)
            k, v = kv_chunk(shape, l, f0, n, device, planted)
            K[l, f0:f0 + n] = k
            V[l, f0:f0 + n] = v
    return K, V


def keep_mask(shape: Shape, frame_begin: int, frame_count: int) -> torch.Tensor:
    """token_idx [frame_count][G] int32: G of the N_in tokens of each frame, sorted (a seeded random mask)."""
    assert shape.N_in >= shape.G
    rows = []
    for f in range(frame_begin, frame_begin + frame_count):
        g = _gen(shape.seed * 7919 + 100 + f, "cpu")
        rows.append(torch.sort(torch.randperm(shape.N_in, generator=g)[:shape.G]).values)
    return torch.stack(rows).to(torch.int32)


def ctr_stream(T: int, N: int, D: int, seed: int, device="cpu", dtype: str = "bf16", frame_chunk: int = 256):
    """Vision-encoder features and saliency for the CTR steps: F [T][N][D] in the storage dtype, alpha [T][N] float32.

    A fixed scene (one base vector per patch position) seen by a camera that does not move: most positions repeat
    their base vector with a little noise (cosine similarity to the previous frame around 0.99: static); a block of
    adjacent positions that wanders over the frame is redrawn every frame (similarity around 0: dynamic); one
    position in eight drifts with noise chosen so that its similarity falls on both sides of 0.9.  The saliency is
    uniform noise, raised where the content changes.  No arithmetic of the method is done here.
    """
    dt = DTYPES[dtype]
    g0 = _gen(seed * 9973 + 1, device)
    base = torch.randn(N, D, generator=g0, device=device)
    drift = (torch.arange(N, device=device) % 8) == 3
    F = torch.empty(T, N, D, dtype=dt, device=device)
    alpha = torch.empty(T, N, dtype=torch.float32, device=device)
    width = max(1, N // 6)
    for f0 in range(0, T, frame_chunk):
        n = min(frame_chunk, T - f0)
        g = _gen(seed * 9973 + 7 + f0, device)
        noise = torch.randn(n, N, D, generator=g, device=device)
        x = base[None] + 0.1 * noise
        x[:, drift] = base[None, drift] + 0.33 * noise[:, drift]
        start = (torch.arange(f0, f0 + n, device=device) * 5) % max(1, N - width)          # [n]
        pos = torch.arange(N, device=device)[None, :]
        moving = (pos >= start[:, None]) & (pos < start[:, None] + width)                   # [n][N]
        x = torch.where(moving[:, :, None], 1.5 * noise, x)
        a = torch.rand(n, N, generator=g, device=device) * 0.6 + 0.4 * moving.float()
        F[f0:f0 + n] = x.to(dt)
        alpha[f0:f0 + n] = a.clamp_(0.0, 1.0)
    return F, alpha


def as_u16(t: torch.Tensor):
    """NumPy view for the oracle: uint16 bit patterns for bf16/fp16, float32 unchanged."""
    t = t.detach().cpu().contiguous()
    if t.dtype in (torch.bfloat16, torch.float16):
        import numpy as np
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
