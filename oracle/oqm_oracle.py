"""ctypes loader for the CPU oracle (oqm_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, the smoke check and the
benchmark's CPU-baseline leg.  Nothing in the CUDA package imports this module
and this module imports nothing from the CUDA package.

All arrays are NumPy host arrays.  bf16 / fp16 tensors are carried as uint16
bit patterns (NumPy has no bfloat16); `to_f32` / `from_f32` convert.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "oqm_oracle.c"
_LIB = _HERE / "liboqm_oracle.so"

BF16, FP16, FP32 = 0, 1, 2
PER_LAYER, PER_HEAD = 0, 1


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no fused multiply-add contraction, no fast-math)."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
           str(_SRC), "-o", str(_LIB), "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "group_tokens",
        "capacity_groups", "bits", "kv_dtype", "score_mode", "meta_dtype")]


class _Store(C.Structure):
    _fields_ = [("codes_k", C.c_void_p), ("codes_v", C.c_void_p), ("scale_k", C.c_void_p),
                ("zero_k", C.c_void_p), ("scale_v", C.c_void_p), ("zero_v", C.c_void_p),
                ("rep_key", C.c_void_p), ("rep_norm2", C.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(str(_LIB))
        L.orc_bf16_to_f32.restype = C.c_float
        L.orc_bf16_to_f32.argtypes = [C.c_uint16]
        L.orc_f16_to_f32.restype = C.c_float
        L.orc_f16_to_f32.argtypes = [C.c_uint16]
        L.orc_f32_to_bf16.restype = C.c_uint16
        L.orc_f32_to_bf16.argtypes = [C.c_float]
        L.orc_f32_to_f16.restype = C.c_uint16
        L.orc_f32_to_f16.argtypes = [C.c_float]
        for name in ("orc_round_nearest", "orc_round_down", "orc_round_up"):
            getattr(L, name).restype = C.c_float
            getattr(L, name).argtypes = [C.c_float, C.c_int]
        L.orc_dequant_value.restype = C.c_float
        L.orc_dequant_value.argtypes = [C.c_int, C.c_float, C.c_float]
        L.orc_paper_ratio.restype = C.c_double
        L.orc_paper_ratio.argtypes = [C.c_int32] * 3
        L.orc_ratio_percent.restype = C.c_double
        L.orc_ratio_percent.argtypes = [C.c_int32] * 3
        L.orc_fp16_kv_bytes.restype = C.c_double
        L.orc_fp16_kv_bytes.argtypes = [C.c_int32, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32]
        L.orc_store_bytes.restype = C.c_double
        L.orc_store_bytes.argtypes = [C.POINTER(Config), C.c_int64, C.c_int32]
        L.orc_budget_to_k.restype = C.c_int32
        L.orc_budget_to_k.argtypes = [C.c_int64, C.c_int32, C.c_int32]
        L.orc_max_threads.restype = C.c_int32
        for name in ("orc_quantize_frame", "orc_score_groups", "orc_topk", "orc_dequant_gather", "orc_attend",
                     "orc_ctr_similarity", "orc_ctr_select"):
            getattr(L, name).restype = C.c_int32
        _lib = L
    return _lib


def _p(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


def make_config(n_layers, n_q_heads, n_kv_heads, head_dim, group_tokens, capacity_groups,
                bits=4, kv_dtype=BF16, score_mode=PER_LAYER, meta_dtype=FP32) -> Config:
    return Config(n_layers, n_q_heads, n_kv_heads, head_dim, group_tokens, capacity_groups,
                  bits, kv_dtype, score_mode, meta_dtype)


class Store:
    """Host-side memory bank: plain NumPy arrays, zero-initialised.  s, m and k-bar are float32 arrays whatever
    cfg.meta_dtype says: with 16-bit metadata they hold values that are exactly representable in that type."""

    def __init__(self, cfg: Config):
        L, T, H, G, d = cfg.n_layers, cfg.capacity_groups, cfg.n_kv_heads, cfg.group_tokens, cfg.head_dim
        rb = d * cfg.bits // 8
        self.cfg = cfg
        self.codes_k = np.zeros((L, T, H, G, rb), np.uint8)
        self.codes_v = np.zeros((L, T, H, G, rb), np.uint8)
        self.scale_k = np.zeros((L, T, H, d), np.float32)
        self.zero_k = np.zeros((L, T, H, d), np.float32)
        self.scale_v = np.zeros((L, T, H, d), np.float32)
        self.zero_v = np.zeros((L, T, H, d), np.float32)
        self.rep_key = np.zeros((L, T, H, d), np.float32)
        self.rep_norm2 = np.zeros((L, T, H), np.float32)

    def c(self) -> _Store:
        return _Store(*[a.ctypes.data for a in (
            self.codes_k, self.codes_v, self.scale_k, self.zero_k, self.scale_v, self.zero_v,
            self.rep_key, self.rep_norm2)])


# ---------------------------------------------------------------- formats

def to_f32(a: np.ndarray, dtype: int) -> np.ndarray:
    a = np.ascontiguousarray(a)
    out = np.empty(a.shape, np.float32)
    lib().orc_convert_to_f32(_p(a), C.c_int(dtype), C.c_int64(a.size), _p(out))
    return out


def from_f32(a: np.ndarray, dtype: int) -> np.ndarray:
    a = np.ascontiguousarray(a, np.float32)
    out = np.empty(a.shape, np.float32 if dtype == FP32 else np.uint16)
    lib().orc_convert_from_f32(_p(a), C.c_int(dtype), C.c_int64(a.size), _p(out))
    return out


# ---------------------------------------------------------------- pieces

def round_nearest(x: float, dtype: int) -> float:
    return float(lib().orc_round_nearest(C.c_float(x), dtype))


def round_down(x: float, dtype: int) -> float:
    return float(lib().orc_round_down(C.c_float(x), dtype))


def round_up(x: float, dtype: int) -> float:
    return float(lib().orc_round_up(C.c_float(x), dtype))


def quantize_group(X: np.ndarray, bits: int = 4, meta_dtype: int = FP32):
    """X [H][G][d] float32 -> (codes [H][G][d] uint8 unpacked, s [H][d], m [H][d])."""
    X = np.ascontiguousarray(X, np.float32)
    H, G, d = X.shape
    codes = np.empty((H, G, d), np.uint8)
    s = np.empty((H, d), np.float32)
    m = np.empty((H, d), np.float32)
    lib().orc_quantize_group(_p(X), C.c_int(H), C.c_int(G), C.c_int(d), C.c_int(bits), C.c_int(meta_dtype),
                             _p(codes), _p(s), _p(m))
    return codes, s, m


def pack_row(codes: np.ndarray, bits: int = 4) -> np.ndarray:
    codes = np.ascontiguousarray(codes, np.uint8)
    out = np.empty(codes.size * bits // 8, np.uint8)
    lib().orc_pack_row(_p(codes), C.c_int(codes.size), C.c_int(bits), _p(out))
    return out


def unpack_row(packed: np.ndarray, d: int, bits: int = 4) -> np.ndarray:
    packed = np.ascontiguousarray(packed, np.uint8)
    out = np.empty(d, np.uint8)
    lib().orc_unpack_row(_p(packed), C.c_int(d), C.c_int(bits), _p(out))
    return out


def dequant_value(code: int, s: float, m: float) -> float:
    return float(lib().orc_dequant_value(int(code), C.c_float(s), C.c_float(m)))


def rep_key(K: np.ndarray, meta_dtype: int = FP32):
    """K [H][G][d] float32 -> (k-bar [H][d] float32, |k-bar_h|^2 [H] float32)."""
    K = np.ascontiguousarray(K, np.float32)
    H, G, d = K.shape
    rep = np.empty((H, d), np.float32)
    n2 = np.empty((H,), np.float32)
    lib().orc_rep_key(_p(K), C.c_int(H), C.c_int(G), C.c_int(d), C.c_int(meta_dtype), _p(rep), _p(n2))
    return rep, n2


def query_embedding(cfg: Config, Q: np.ndarray, q_dtype: int) -> np.ndarray:
    """Q [H_q][T_q][d] (one layer, contiguous) -> q [H_k][d] float64."""
    Q = np.ascontiguousarray(Q)
    Hq, Tq, d = Q.shape
    out = np.empty((cfg.n_kv_heads, d), np.float64)
    lib().orc_query_embedding(C.byref(cfg), _p(Q), C.c_int(q_dtype), C.c_int64(0), C.c_int32(Tq),
                              C.c_int64(Tq * d), C.c_int64(d), _p(out))
    return out


# ---------------------------------------------------------------- the four calls (+ attend)

def quantize_frame(cfg: Config, store: Store, layer_begin, layer_count, group_begin, group_count,
                   K, V, strides, K_summary=None, token_idx=None, tokens_per_frame_in=0, n_threads=0):
    sl, sg, sh, stok = strides
    if token_idx is not None:
        token_idx = np.ascontiguousarray(token_idx, np.int32)
    st = store.c()
    return lib().orc_quantize_frame(
        C.byref(cfg), C.byref(st), C.c_int32(layer_begin), C.c_int32(layer_count), C.c_int32(group_begin),
        C.c_int32(group_count), _p(K), _p(V), C.c_int64(sl), C.c_int64(sg), C.c_int64(sh), C.c_int64(stok),
        _p(K_summary), _p(token_idx), C.c_int32(tokens_per_frame_in), C.c_int32(n_threads))


def score_groups(cfg: Config, store: Store, layer_begin, layer_count, n_groups, Q, T_q, q_strides,
                 n_threads=0) -> np.ndarray:
    ql, qh, qt = q_strides
    H = cfg.n_kv_heads
    shape = (layer_count, n_groups) if cfg.score_mode == PER_LAYER else (layer_count, H, n_groups)
    scores = np.zeros(shape, np.float32)
    st = store.c()
    rc = lib().orc_score_groups(C.byref(cfg), C.byref(st), C.c_int32(layer_begin), C.c_int32(layer_count),
                                C.c_int32(n_groups), _p(Q), C.c_int32(T_q), C.c_int64(ql), C.c_int64(qh),
                                C.c_int64(qt), _p(scores), C.c_int32(n_threads))
    if rc:
        raise ValueError(f"orc_score_groups -> {rc}")
    return scores


def topk(scores: np.ndarray, k: int):
    """scores [rows][n] -> (idx [rows][k] int32 ascending, -1 padded; sel scores; n_sel [rows])."""
    scores = np.ascontiguousarray(scores, np.float32)
    rows, n = scores.shape
    idx = np.empty((rows, k), np.int32)
    sc = np.empty((rows, k), np.float32)
    nsel = np.empty((rows,), np.int32)
    rc = lib().orc_topk(_p(scores), C.c_int32(rows), C.c_int32(n), C.c_int64(n), C.c_int32(k), _p(idx), _p(sc), _p(nsel))
    if rc:
        raise ValueError(f"orc_topk -> {rc}")
    return idx, sc, nsel


def budget_to_k(budget_tokens: int, G: int, stored_groups: int) -> int:
    return int(lib().orc_budget_to_k(budget_tokens, G, stored_groups))


def dequant_gather(cfg: Config, store: Store, layer_begin, layer_count, idx, k, n_groups, k_active, v_active,
                   out_dtype, strides, token_offset, n_threads=0):
    sl, sh, stok = strides
    idx = np.ascontiguousarray(idx, np.int32)
    st = store.c()
    return lib().orc_dequant_gather(
        C.byref(cfg), C.byref(st), C.c_int32(layer_begin), C.c_int32(layer_count), _p(idx), C.c_int32(k),
        C.c_int32(n_groups), _p(k_active), _p(v_active), C.c_int32(out_dtype), C.c_int64(sl), C.c_int64(sh),
        C.c_int64(stok), C.c_int32(token_offset), C.c_int32(n_threads))


def attend(H_q, H_k, d, q_dec, q_dtype, k_cache, v_cache, kv_dtype, stride_head, stride_token, n_tokens,
           softmax_scale, out_dtype=BF16) -> np.ndarray:
    out = np.empty((H_q, d), np.float32 if out_dtype == FP32 else np.uint16)
    rc = lib().orc_attend(C.c_int32(H_q), C.c_int32(H_k), C.c_int32(d), _p(q_dec), C.c_int32(q_dtype),
                          _p(k_cache), _p(v_cache), C.c_int32(kv_dtype), C.c_int64(stride_head),
                          C.c_int64(stride_token), C.c_int32(n_tokens), C.c_double(softmax_scale), _p(out),
                          C.c_int32(out_dtype))
    if rc:
        raise ValueError(f"orc_attend -> {rc}")
    return out


# ---------------------------------------------------------------- CTR

def ctr_similarity(F: np.ndarray, dtype: int, prev: np.ndarray | None = None) -> np.ndarray:
    """F [T][N][D] (contiguous; uint16 patterns for the 16-bit types), prev [N][D] or None -> sim [T][N] float32."""
    F = np.ascontiguousarray(F)
    T, N, D = F.shape
    if prev is not None:
        prev = np.ascontiguousarray(prev)
        assert prev.shape == (N, D) and prev.dtype == F.dtype
    sim = np.empty((T, N), np.float32)
    rc = lib().orc_ctr_similarity(_p(F), _p(prev), C.c_int(dtype), C.c_int32(T), C.c_int32(N), C.c_int32(D),
                                  C.c_int64(N * D), C.c_int64(D), _p(sim))
    if rc:
        raise ValueError(f"orc_ctr_similarity -> {rc}")
    return sim


def ctr_select(sim: np.ndarray, alpha: np.ndarray, G: int, tau_c: float):
    """sim, alpha [T][N] float32 -> (k_s [T], k_d [T], static_idx [T][N], dyn_idx [T][G]), int32, -1 padded."""
    sim = np.ascontiguousarray(sim, np.float32)
    alpha = np.ascontiguousarray(alpha, np.float32)
    T, N = sim.shape
    ks, kd = np.empty(T, np.int32), np.empty(T, np.int32)
    sidx, didx = np.empty((T, N), np.int32), np.empty((T, G), np.int32)
    rc = lib().orc_ctr_select(_p(sim), _p(alpha), C.c_int32(T), C.c_int32(N), C.c_int32(G), C.c_float(tau_c),
                              _p(ks), _p(kd), _p(sidx), _p(didx))
    if rc:
        raise ValueError(f"orc_ctr_select -> {rc}")
    return ks, kd, sidx, didx


def ctr_merge(F_frame: np.ndarray, dtype: int, S: np.ndarray, k_s: int, knn: int = 5):
    """One frame's Merge_{k_s} under this code's reading of the paper's density-based clustering.

    F_frame [N][D] (uint16 patterns for the 16-bit types), S: ascending static token indices.  Returns a dict:
    centre [k_s] (token indices, ascending), assign [n_s] (position of each static token's centre in `centre`),
    merged [k_s][D] float32 (member means), gamma [n_s] float64, margin_centres (relative gap between the last gamma
    taken and the first left out) and margin_assign [n_s] (relative gap between each token's nearest and second
    nearest centre): how far the integer decisions are from flipping."""
    F_frame = np.ascontiguousarray(F_frame)
    N, D = F_frame.shape
    S = np.ascontiguousarray(S, np.int32)
    n_s = int(S.shape[0])
    centre = np.full(max(k_s, 1), -1, np.int32)
    assign = np.full(max(n_s, 1), -1, np.int32)
    merged = np.zeros((max(k_s, 1), D), np.float32)
    gamma = np.zeros(max(n_s, 1), np.float64)
    margin = np.zeros(1 + max(n_s, 1), np.float64)
    rc = lib().orc_ctr_merge(_p(F_frame), C.c_int32(dtype), C.c_int32(N), C.c_int32(D), C.c_int64(D), _p(S),
                             C.c_int32(n_s), C.c_int32(k_s), C.c_int32(knn), _p(centre), _p(assign), _p(merged),
                             _p(gamma), _p(margin))
    if rc:
        raise ValueError(f"orc_ctr_merge -> {rc}")
    return {"centre": centre[:k_s], "assign": assign[:n_s], "merged": merged[:k_s], "gamma": gamma[:n_s],
            "margin_centres": float(margin[0]), "margin_assign": margin[1:1 + n_s]}


def ctr_retain(F_frame: np.ndarray, dtype: int, dyn: np.ndarray, centre: np.ndarray, merged: np.ndarray, G: int):
    """The frame's retained group: the selected dynamic rows and the merged rows in position order.
    Returns (retained [G][D] in the feature type, pos [G] int32)."""
    F_frame = np.ascontiguousarray(F_frame)
    N, D = F_frame.shape
    dyn = np.ascontiguousarray(dyn, np.int32)
    centre = np.ascontiguousarray(centre, np.int32)
    merged = np.ascontiguousarray(merged, np.float32)
    retained = np.zeros((G, D), F_frame.dtype)
    pos = np.full(G, -1, np.int32)
    rc = lib().orc_ctr_retain(_p(F_frame), C.c_int32(dtype), C.c_int32(N), C.c_int32(D), C.c_int64(D), _p(dyn),
                              C.c_int32(dyn.shape[0]), _p(centre), _p(merged), C.c_int32(centre.shape[0]), C.c_int32(G),
                              _p(retained), _p(pos))
    if rc:
        raise ValueError(f"orc_ctr_retain -> {rc}")
    return retained, pos


# ---------------------------------------------------------------- accounting

def paper_ratio(N, G, bits=4):
    return float(lib().orc_paper_ratio(N, G, bits))


def ratio_percent(N, G, bits):
    return float(lib().orc_ratio_percent(N, G, bits))


def fp16_kv_bytes(L, frames, N, H_kv, d_h, elem_bytes=2):
    return float(lib().orc_fp16_kv_bytes(L, frames, N, H_kv, d_h, elem_bytes))


def store_bytes(cfg: Config, groups: int, with_metadata: bool):
    return float(lib().orc_store_bytes(C.byref(cfg), groups, int(with_metadata)))


def max_threads() -> int:
    return int(lib().orc_max_threads())


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1
