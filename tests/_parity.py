"""Shared helpers of the GPU parity tests: run the same seeded inputs through the
CPU oracle and through the C-ABI CUDA library, and compare element by element.

Tolerances (stated here, used by every parity test):
  * packed 4-bit codes ........ bit-exact
  * scale s ................... bit-exact (two binary32 operations on both sides)
  * offset m .................. equal as numbers (+0 and -0 compare equal)
  * representative key ........ |d| <= 2^-24 * sum_g|x_g| + 2^-23 * |k-bar|   (binary32 summation of G terms
                                against the oracle's binary64 mean), norms to 1e-5 relative
  * scores .................... |d| <= 1e-5 absolute (scores lie in [-1, 1])
  * selected indices .......... identical, except members whose oracle score is within 1e-5 relative of the
                                oracle's K-th score (ties)
  * 16-bit metadata ........... s and m bit-exact after conversion to binary32; k-bar equal to the oracle's except
                                where the binary32 mean sits within its summation error of a rounding boundary of
                                the 16-bit type (then one 16-bit step apart; at most 0.5 % of the entries), and
                                the stored norm within 1e-5 relative of the norm of the key the library stored
  * dequantized values ........ |a - b| <= 1e-3 * max(|b|, s); in fact expected bit-identical (same fmaf, same
                                rounding), and the mismatch count is asserted to be 0
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2510_18269_b200 import synth

GUARD = 64  # sentinel elements kept after every output buffer


def dt_code(dtype: str) -> int:
    return {"bf16": 0, "fp16": 1, "fp32": 2}[dtype]


def contiguous_strides(sh, tokens):
    """Element strides (layer, group, head, token) of a [L][T][H_k][tokens][d] tensor."""
    return (sh.T * sh.H_k * tokens * sh.d, sh.H_k * tokens * sh.d, tokens * sh.d, sh.d)


def q_strides(sh):
    return (sh.H_q * sh.T_q * sh.d, sh.T_q * sh.d, sh.d)


def bits_of(sh) -> int:
    """Width of a code for this workload: 4 unless the shape asks for the 2-bit variant."""
    return int(sh.extra.get("bits", 4))


def meta_of(sh) -> str:
    """Storage type of s, m and k-bar for this workload: fp32 unless the shape asks for fp16 / bf16."""
    return str(sh.extra.get("meta", "fp32"))


def oracle_cfg(orc, sh, mode=0, cap=None):
    return orc.make_config(sh.L, sh.H_q, sh.H_k, sh.d, sh.G, cap or sh.T, bits_of(sh), dt_code(sh.dtype), mode,
                           dt_code(meta_of(sh)))


def gpu_cfg(oqm, sh, mode=0, cap=None):
    return oqm.make_config(sh.L, sh.H_q, sh.H_k, sh.d, sh.G, cap or sh.T, bits_of(sh), dt_code(sh.dtype), mode,
                           dt_code(meta_of(sh)))


_TORCH16 = {0: torch.bfloat16, 1: torch.float16}


def compare_store(gst, ost, K_f32, groups=None, layers=None):
    """gst: oqm.Store (device); ost: oracle Store (host); K_f32: float32 numpy [L][T][H][G][d] of the keys the
    representative key was averaged from (for its error bound)."""
    L = gst.cfg.n_layers
    layers = range(L) if layers is None else layers
    gsel = slice(None) if groups is None else groups
    meta16 = gst.cfg.meta_dtype != 2

    def meta_np(t):  # a device metadata array as float32 numpy (exact for every storage type)
        return t.to(torch.float32).cpu().numpy()

    for l in layers:
        for name in ("codes_k", "codes_v"):
            g = getattr(gst, name)[l, gsel].cpu().numpy()
            o = getattr(ost, name)[l, gsel]
            bad = int((g != o).sum())
            assert bad == 0, f"{name} layer {l}: {bad} packed bytes differ"
        for name in ("scale_k", "scale_v"):
            g = meta_np(getattr(gst, name)[l, gsel])
            o = getattr(ost, name)[l, gsel]
            assert np.array_equal(g.view(np.uint32), o.view(np.uint32)), f"{name} layer {l} not bit-exact"
        for name in ("zero_k", "zero_v"):
            g = meta_np(getattr(gst, name)[l, gsel])
            o = getattr(ost, name)[l, gsel]
            assert np.array_equal(g, o), f"{name} layer {l} differs"
        g = meta_np(gst.rep_key[l, gsel]).astype(np.float64)
        o = ost.rep_key[l, gsel].astype(np.float64)
        gn = gst.rep_norm2[l, gsel].cpu().numpy().astype(np.float64)
        on = ost.rep_norm2[l, gsel].astype(np.float64)
        if not meta16:
            absum = np.abs(K_f32[l, gsel]).astype(np.float64).sum(axis=-2)         # [T][H][d]
            tol = 2.0 ** -24 * absum + 2.0 ** -23 * np.abs(o) + 1e-30
            assert np.all(np.abs(g - o) <= tol), f"rep_key layer {l}: max excess {(np.abs(g - o) - tol).max()}"
            assert np.all(np.abs(gn - on) <= 1e-5 * np.abs(on) + 1e-30), f"rep_norm2 layer {l}"
        else:
            step = np.abs(o) * (2.0 ** -7 if gst.cfg.meta_dtype == 0 else 2.0 ** -10) + 2.0 ** -24
            assert np.all(np.abs(g - o) <= step), f"rep_key layer {l}: more than one 16-bit step apart"
            assert np.mean(g != o) <= 5e-3, f"rep_key layer {l}: {np.mean(g != o):.4f} of the entries differ"
            own = (g ** 2).sum(axis=-1)
            assert np.all(np.abs(gn - own) <= 1e-5 * own + 1e-30), f"rep_norm2 layer {l} is not the norm of the stored key"


def compare_scores(g_scores: torch.Tensor, o_scores: np.ndarray):
    g = g_scores.cpu().numpy().reshape(o_scores.shape)
    err = np.abs(g.astype(np.float64) - o_scores.astype(np.float64))
    assert err.max() <= 1e-5, f"scores differ by {err.max()}"


def compare_topk(g_idx: torch.Tensor, o_idx: np.ndarray, o_scores_rows: np.ndarray, k: int):
    """g_idx, o_idx: [rows][k]; o_scores_rows: [rows][n] oracle scores."""
    g = g_idx.cpu().numpy().reshape(o_idx.shape)
    n = o_scores_rows.shape[1]
    ksel = min(k, n)
    exact_rows = 0
    for r in range(o_idx.shape[0]):
        gr, orr = g[r], o_idx[r]
        assert np.all(gr[ksel:] == -1), "unused slots must be -1"
        sel = gr[:ksel]
        assert np.all((sel >= 0) & (sel < n)) and np.all(np.diff(sel) > 0), "selection must be ascending and in range"
        if np.array_equal(sel, orr[:ksel]):
            exact_rows += 1
            continue
        kth = o_scores_rows[r, orr[:ksel]].min()
        diff = np.setxor1d(sel, orr[:ksel])
        sc = o_scores_rows[r, diff]
        assert np.all(np.abs(sc - kth) <= 1e-5 * max(abs(kth), 1e-30)), \
            f"row {r}: selections differ beyond score ties: {diff}, scores {sc}, kth {kth}"
    return exact_rows


def compare_active(g16: np.ndarray, o16: np.ndarray, g_idx: np.ndarray, o_idx: np.ndarray, sys_len: int, G: int,
                   per_head: bool = False, min_same: float = 0.9):
    """Active caches [L][H][S][d] as 16-bit patterns: the library's (built from ITS selection g_idx) against the
    oracle's (built from the oracle's selection o_idx; nothing the library produced is fed to the oracle).  Slot j of
    a ranking row lands in tokens [sys_len + j*G, sys_len + (j+1)*G) and depends on idx[row][j] alone, so the slots
    where both sides selected the same group are compared bit for bit; they differ only behind a tie at the K-th
    score.  The system tokens in front and whatever lies behind the last slot must be identical.  Returns the rows
    whose selections agree completely."""
    L, H, S, d = o16.shape
    rows, k = o_idx.shape
    g_idx = g_idx.reshape(rows, k)
    same = g_idx == o_idx
    assert same.mean() >= min_same, f"only {same.mean():.3f} of the slots hold the same group on both sides"
    gr = g16.reshape(rows, -1, S, d) if per_head else g16.reshape(rows, H, S, d)
    orr = o16.reshape(gr.shape)
    assert np.array_equal(gr[:, :, :sys_len], orr[:, :, :sys_len]), "system tokens differ"
    assert np.array_equal(gr[:, :, sys_len + k * G:], orr[:, :, sys_len + k * G:]), "tokens behind the last slot differ"
    for r in range(rows):
        for j in range(k):
            if same[r, j]:
                a, b = sys_len + j * G, sys_len + (j + 1) * G
                assert np.array_equal(gr[r, :, a:b], orr[r, :, a:b]), f"row {r} slot {j}: reconstructed group differs"
    return same.all(axis=1)


def out_buffers(sh, layer_count, S_tokens, torch_dtype, device, sentinel):
    """Active cache [layer_count][H_k][S_tokens][d] with a guard band after it, filled with a sentinel."""
    n = layer_count * sh.H_k * S_tokens * sh.d
    flat = torch.full((n + GUARD,), sentinel, dtype=torch_dtype, device=device)
    return flat, flat[:n].view(layer_count, sh.H_k, S_tokens, sh.d)


def active_strides(sh, S_tokens):
    return (sh.H_k * S_tokens * sh.d, S_tokens * sh.d, sh.d)


def as_np16(t: torch.Tensor) -> np.ndarray:
    return synth.as_u16(t)


def f32_of(orc, arr: np.ndarray, dtype: str) -> np.ndarray:
    return arr if dtype == "fp32" else orc.to_f32(arr, dt_code(dtype))


def random_bank(orc, oqm, sh, mode, seed):
    """The same random bank in an oracle Store (NumPy) and in a device Store."""
    ocfg, gcfg = oracle_cfg(orc, sh, mode), gpu_cfg(oqm, sh, mode)
    ost, gst = orc.Store(ocfg), oqm.Store(gcfg)
    rng = np.random.default_rng(seed)
    ost.rep_key[...] = rng.standard_normal(ost.rep_key.shape, dtype=np.float32)
    # a few groups point along a common direction so that the head of the ranking is not pure noise
    u = rng.standard_normal((sh.L, 1, sh.H_k, sh.d), dtype=np.float32)
    pick = rng.choice(sh.T, size=max(1, min(sh.T, sh.k) // 2), replace=False)
    ost.rep_key[:, pick] = u + 0.3 * ost.rep_key[:, pick]
    ost.rep_norm2[...] = (ost.rep_key.astype(np.float64) ** 2).sum(-1).astype(np.float32)
    ost.codes_k[...] = rng.integers(0, 256, ost.codes_k.shape, dtype=np.uint8)
    ost.codes_v[...] = rng.integers(0, 256, ost.codes_v.shape, dtype=np.uint8)
    for name in ("scale_k", "scale_v"):
        getattr(ost, name)[...] = rng.uniform(0.01, 0.5, getattr(ost, name).shape).astype(np.float32)
    for name in ("zero_k", "zero_v"):
        getattr(ost, name)[...] = rng.standard_normal(getattr(ost, name).shape, dtype=np.float32)
    if ocfg.meta_dtype != 2:  # both sides hold the same values, representable in the 16-bit storage type
        t16 = _TORCH16[ocfg.meta_dtype]
        for name in ("scale_k", "zero_k", "scale_v", "zero_v", "rep_key"):
            a = getattr(ost, name)
            a[...] = torch.from_numpy(a).to(t16).to(torch.float32).numpy()
        ost.rep_norm2[...] = (ost.rep_key.astype(np.float64) ** 2).sum(-1).astype(np.float32)
    for name in ("codes_k", "codes_v", "scale_k", "zero_k", "scale_v", "zero_v", "rep_key", "rep_norm2"):
        dst = getattr(gst, name)
        dst.copy_(torch.from_numpy(getattr(ost, name)).to(dst.dtype))
    return ocfg, gcfg, ost, gst, u
