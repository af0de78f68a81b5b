"""Thin Python binding of libstom_oqm.so (argument marshalling only).

Every step of the path runs in the library's CUDA kernels; PyTorch is used for
device memory and streams.  There is no CPU fallback: if the library is not
built, importing `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libstom_oqm.so"

BF16, FP16, FP32 = 0, 1, 2
PER_LAYER, PER_HEAD = 0, 1
FLAG_BAD_INDEX = 1
FLAG_TIMEOUT = 2
FLAG_DIRTY_WORKSPACE = 4

_TORCH_DTYPE = {BF16: torch.bfloat16, FP16: torch.float16, FP32: torch.float32}
_DTYPE_CODE = {v: k for k, v in _TORCH_DTYPE.items()}

EXPORTS = (
    "stom_oqm_store_layout", "stom_oqm_store_bind", "stom_oqm_budget_to_k", "stom_oqm_score_workspace_bytes",
    "stom_status_string", "stom_last_cuda_error", "stom_oqm_quantize_frame", "stom_oqm_score_groups",
    "stom_oqm_topk", "stom_oqm_dequant_gather", "stom_oqm_retrieve",
    "stom_oqm_quantize_host_scratch_bytes", "stom_oqm_quantize_frame_host",
    "stom_oqm_retrieve_host_scratch_bytes", "stom_oqm_retrieve_host",
    "stom_oqm_score_groups_noalloc", "stom_oqm_attend_workspace_bytes", "stom_oqm_attend",
    "stom_oqm_retrieve_workspace_bytes",
    "stom_ctr_similarity", "stom_ctr_select", "stom_ctr_reduce", "stom_ctr_merge", "stom_ctr_reduce_tokens",
)


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "group_tokens",
        "capacity_groups", "bits", "kv_dtype", "score_mode", "meta_dtype")]


class StoreDesc(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "codes_k", "codes_v", "scale_k", "zero_k", "scale_v", "zero_v", "rep_key", "rep_norm2")]


class Layout(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "bytes_total", "off_codes_k", "off_codes_v", "off_scale_k", "off_zero_k", "off_scale_v", "off_zero_v",
        "off_rep_key", "off_rep_norm2", "bytes_codes", "bytes_meta", "bytes_norm2")]


class StomError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().stom_status_string(code).decode()
        super().__init__(f"{where}: {msg} (status {code}, cuda error {lib().stom_last_cuda_error()})")


_lib = None


def lib():
    """The loaded C-ABI library.  Fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2510_18269_b200.build` "
                "(there is no fallback path)")
        L = C.CDLL(str(LIB_PATH))
        L.stom_status_string.restype = C.c_char_p
        L.stom_status_string.argtypes = [C.c_int32]
        L.stom_oqm_score_workspace_bytes.restype = C.c_int64
        L.stom_oqm_score_workspace_bytes.argtypes = [C.POINTER(Config), C.c_int32]
        L.stom_oqm_budget_to_k.argtypes = [C.c_int64, C.c_int32, C.c_int32]
        L.stom_oqm_attend_workspace_bytes.restype = C.c_int64
        L.stom_oqm_retrieve_workspace_bytes.restype = C.c_int64
        L.stom_oqm_quantize_host_scratch_bytes.restype = C.c_int64
        L.stom_oqm_retrieve_host_scratch_bytes.restype = C.c_int64
        for name in EXPORTS:
            fn = getattr(L, name)
            if fn.restype is C.c_int:
                fn.restype = C.c_int32
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(rc: int, where: str):
    if rc != 0:
        raise StomError(rc, where)


def make_config(n_layers, n_q_heads, n_kv_heads, head_dim, group_tokens, capacity_groups,
                bits=4, kv_dtype=BF16, score_mode=PER_LAYER, meta_dtype=FP32) -> Config:
    return Config(n_layers, n_q_heads, n_kv_heads, head_dim, group_tokens, capacity_groups,
                  bits, kv_dtype, score_mode, meta_dtype)


def dtype_code(t: torch.dtype) -> int:
    return _DTYPE_CODE[t]


def stom_oqm_store_layout(cfg: Config) -> Layout:
    lay = Layout()
    _check(lib().stom_oqm_store_layout(C.byref(cfg), C.byref(lay)), "stom_oqm_store_layout")
    return lay


def stom_oqm_budget_to_k(budget_tokens: int, group_tokens: int, stored_groups: int) -> int:
    return int(lib().stom_oqm_budget_to_k(budget_tokens, group_tokens, stored_groups))


def stom_oqm_score_workspace_bytes(cfg: Config, layer_count: int) -> int:
    return int(lib().stom_oqm_score_workspace_bytes(C.byref(cfg), layer_count))


class Store:
    """One device arena holding the memory bank, plus typed tensor views of its arrays."""

    def __init__(self, cfg: Config, device="cuda", zero: bool = True):
        self.cfg = cfg
        self.layout = stom_oqm_store_layout(cfg)
        alloc = torch.zeros if zero else torch.empty
        self.arena = alloc(self.layout.bytes_total + 256, dtype=torch.uint8, device=device)
        shift = (-self.arena.data_ptr()) % 256
        self.base = self.arena[shift:shift + self.layout.bytes_total]
        self.desc = StoreDesc()
        _check(lib().stom_oqm_store_bind(C.byref(cfg), C.c_void_p(self.base.data_ptr()), C.byref(self.desc)),
               "stom_oqm_store_bind")
        L, T, H, G, d = cfg.n_layers, cfg.capacity_groups, cfg.n_kv_heads, cfg.group_tokens, cfg.head_dim
        lay = self.layout

        def view(off, nbytes, dtype, shape):
            return self.base[off:off + nbytes].view(dtype).view(*shape)

        self.codes_k = view(lay.off_codes_k, lay.bytes_codes, torch.uint8, (L, T, H, G, d * cfg.bits // 8))
        self.codes_v = view(lay.off_codes_v, lay.bytes_codes, torch.uint8, (L, T, H, G, d * cfg.bits // 8))
        mt = _TORCH_DTYPE[cfg.meta_dtype]  # element type of s, m and k-bar
        self.scale_k = view(lay.off_scale_k, lay.bytes_meta, mt, (L, T, H, d))
        self.zero_k = view(lay.off_zero_k, lay.bytes_meta, mt, (L, T, H, d))
        self.scale_v = view(lay.off_scale_v, lay.bytes_meta, mt, (L, T, H, d))
        self.zero_v = view(lay.off_zero_v, lay.bytes_meta, mt, (L, T, H, d))
        self.rep_key = view(lay.off_rep_key, lay.bytes_meta, mt, (L, T, H, d))
        self.rep_norm2 = view(lay.off_rep_norm2, lay.bytes_norm2, torch.float32, (L, T, H))


def stom_oqm_quantize_frame(cfg: Config, store: Store, layer_begin, layer_count, group_begin, group_count,
                            K, V, strides, K_summary=None, token_idx=None, tokens_per_frame_in=0,
                            dev_flags=None, stream=None):
    """strides = (layer, group, head, token) in elements of K / V."""
    sl, sg, sh, st = strides
    rc = lib().stom_oqm_quantize_frame(
        C.byref(cfg), C.byref(store.desc), C.c_int32(layer_begin), C.c_int32(layer_count),
        C.c_int32(group_begin), C.c_int32(group_count), _ptr(K), _ptr(V),
        C.c_int64(sl), C.c_int64(sg), C.c_int64(sh), C.c_int64(st), _ptr(K_summary), _ptr(token_idx),
        C.c_int32(tokens_per_frame_in), _ptr(dev_flags), _stream(stream))
    _check(rc, "stom_oqm_quantize_frame")


def stom_oqm_score_groups(cfg: Config, store: Store, layer_begin, layer_count, n_groups, Q, T_q, q_strides,
                          scores, workspace, stream=None):
    ql, qh, qt = q_strides
    rc = lib().stom_oqm_score_groups(
        C.byref(cfg), C.byref(store.desc), C.c_int32(layer_begin), C.c_int32(layer_count), C.c_int32(n_groups),
        _ptr(Q), C.c_int32(T_q), C.c_int64(ql), C.c_int64(qh), C.c_int64(qt), _ptr(scores), _ptr(workspace),
        C.c_int64(0 if workspace is None else workspace.numel() * workspace.element_size()), _stream(stream))
    _check(rc, "stom_oqm_score_groups")


NOALLOC_SCRATCH_BYTES = 512 * 1024


def stom_oqm_score_groups_noalloc(cfg: Config, store: Store, layer_begin, layer_count, n_groups, Q, T_q, q_strides,
                                  scores, stream=None):
    """Scores without caller scratch, for hosts that cannot allocate device memory (for example a server whose
    memory pool owns all of HBM, or code that may not call cudaMalloc because it would stall the device).

    Same result as stom_oqm_score_groups.  The intermediate question embeddings live in a NOALLOC_SCRATCH_BYTES
    array inside the library that all calls on a GPU share: keep such calls ordered on the GPU (one stream, or
    events), make the first call on each GPU outside of stream capture, and split the layer range when the call
    reports that the array is too small."""
    ql, qh, qt = q_strides
    rc = lib().stom_oqm_score_groups_noalloc(
        C.byref(cfg), C.byref(store.desc), C.c_int32(layer_begin), C.c_int32(layer_count), C.c_int32(n_groups),
        _ptr(Q), C.c_int32(T_q), C.c_int64(ql), C.c_int64(qh), C.c_int64(qt), _ptr(scores), _stream(stream))
    _check(rc, "stom_oqm_score_groups_noalloc")


def stom_oqm_topk(scores, rows, n, row_stride, k, idx_out, score_out=None, n_sel_out=None, stream=None):
    rc = lib().stom_oqm_topk(_ptr(scores), C.c_int32(rows), C.c_int32(n), C.c_int64(row_stride), C.c_int32(k),
                             _ptr(idx_out), _ptr(score_out), _ptr(n_sel_out), _stream(stream))
    _check(rc, "stom_oqm_topk")


def stom_oqm_dequant_gather(cfg: Config, store: Store, layer_begin, layer_count, idx, k, n_groups,
                            k_active, v_active, out_dtype, strides, token_offset, dev_flags=None, stream=None):
    """strides = (layer, head, token) in elements of the active cache."""
    sl, sh, st = strides
    rc = lib().stom_oqm_dequant_gather(
        C.byref(cfg), C.byref(store.desc), C.c_int32(layer_begin), C.c_int32(layer_count), _ptr(idx),
        C.c_int32(k), C.c_int32(n_groups), _ptr(k_active), _ptr(v_active), C.c_int32(out_dtype),
        C.c_int64(sl), C.c_int64(sh), C.c_int64(st), C.c_int32(token_offset), _ptr(dev_flags), _stream(stream))
    _check(rc, "stom_oqm_dequant_gather")


def stom_oqm_retrieve_workspace_bytes(cfg: Config, layer_count: int, n_groups: int, k: int) -> int:
    return int(lib().stom_oqm_retrieve_workspace_bytes(C.byref(cfg), C.c_int32(layer_count), C.c_int32(n_groups),
                                                       C.c_int32(k)))


def stom_oqm_retrieve(cfg: Config, store: Store, layer_begin, layer_count, n_groups, Q, T_q, q_strides, k,
                      scores, idx, k_active, v_active, out_dtype, strides, token_offset, workspace,
                      dev_flags=None, stream=None):
    ql, qh, qt = q_strides
    sl, sh, st = strides
    rc = lib().stom_oqm_retrieve(
        C.byref(cfg), C.byref(store.desc), C.c_int32(layer_begin), C.c_int32(layer_count), C.c_int32(n_groups),
        _ptr(Q), C.c_int32(T_q), C.c_int64(ql), C.c_int64(qh), C.c_int64(qt), C.c_int32(k), _ptr(scores),
        _ptr(idx), _ptr(k_active), _ptr(v_active), C.c_int32(out_dtype), C.c_int64(sl), C.c_int64(sh),
        C.c_int64(st), C.c_int32(token_offset), _ptr(workspace),
        C.c_int64(0 if workspace is None else workspace.numel() * workspace.element_size()), _ptr(dev_flags),
        _stream(stream))
    _check(rc, "stom_oqm_retrieve")


def stom_oqm_attend_workspace_bytes(cfg: Config, layer_count: int, k: int, sys_len: int) -> int:
    return int(lib().stom_oqm_attend_workspace_bytes(C.byref(cfg), C.c_int32(layer_count), C.c_int32(k),
                                                     C.c_int32(sys_len)))


def stom_oqm_attend(cfg: Config, store: Store, layer_begin, layer_count, idx, k, n_groups, q_dec, q_strides,
                    k_sys, v_sys, cache_dtype, sys_strides, sys_len, softmax_scale, out, out_strides, workspace,
                    dev_flags=None, stream=None):
    """q_strides = (layer, head); sys_strides = (layer, head, token); out_strides = (layer, head), all in elements.
    `workspace` is not used by the call (it may be None); the argument remains for callers of the earlier form."""
    rc = lib().stom_oqm_attend(
        C.byref(cfg), C.byref(store.desc), C.c_int32(layer_begin), C.c_int32(layer_count), _ptr(idx), C.c_int32(k),
        C.c_int32(n_groups), _ptr(q_dec), C.c_int64(q_strides[0]), C.c_int64(q_strides[1]), _ptr(k_sys), _ptr(v_sys),
        C.c_int32(cache_dtype), C.c_int64(sys_strides[0]), C.c_int64(sys_strides[1]), C.c_int64(sys_strides[2]),
        C.c_int32(sys_len), C.c_float(softmax_scale), _ptr(out), C.c_int64(out_strides[0]), C.c_int64(out_strides[1]),
        _ptr(workspace), C.c_int64(0 if workspace is None else workspace.numel() * workspace.element_size()),
        _ptr(dev_flags), _stream(stream))
    _check(rc, "stom_oqm_attend")


# ---------------------------------------------------------------- host-buffer entry points

def _hptr(t):
    """Address of a HOST tensor (pinned or pageable)."""
    if t is None:
        return None
    assert not t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def stom_oqm_quantize_host_scratch_bytes(cfg: Config, layer_count: int, group_count: int) -> int:
    return int(lib().stom_oqm_quantize_host_scratch_bytes(C.byref(cfg), C.c_int32(layer_count), C.c_int32(group_count)))


def stom_oqm_quantize_frame_host(cfg: Config, store: Store, layer_begin, layer_count, group_begin, group_count,
                                 K_host, V_host, scratch, dev_flags=None, stream=None):
    rc = lib().stom_oqm_quantize_frame_host(
        C.byref(cfg), C.byref(store.desc), C.c_int32(layer_begin), C.c_int32(layer_count), C.c_int32(group_begin),
        C.c_int32(group_count), _hptr(K_host), _hptr(V_host), _ptr(scratch),
        C.c_int64(scratch.numel() * scratch.element_size()), _ptr(dev_flags), _stream(stream))
    _check(rc, "stom_oqm_quantize_frame_host")


def stom_oqm_retrieve_host_scratch_bytes(cfg: Config, layer_count, n_groups, T_q, k, out_dtype) -> int:
    return int(lib().stom_oqm_retrieve_host_scratch_bytes(
        C.byref(cfg), C.c_int32(layer_count), C.c_int32(n_groups), C.c_int32(T_q), C.c_int32(k), C.c_int32(out_dtype)))


def stom_oqm_retrieve_host(cfg: Config, store: Store, layer_begin, layer_count, n_groups, Q_host, T_q, k,
                           idx_host, k_active_host, v_active_host, out_dtype, scratch, dev_flags=None, stream=None):
    rc = lib().stom_oqm_retrieve_host(
        C.byref(cfg), C.byref(store.desc), C.c_int32(layer_begin), C.c_int32(layer_count), C.c_int32(n_groups),
        _hptr(Q_host), C.c_int32(T_q), C.c_int32(k), _hptr(idx_host), _hptr(k_active_host), _hptr(v_active_host),
        C.c_int32(out_dtype), _ptr(scratch), C.c_int64(scratch.numel() * scratch.element_size()), _ptr(dev_flags),
        _stream(stream))
    _check(rc, "stom_oqm_retrieve_host")


# ---------------------------------------------------------------- CTR (include/stom_ctr.h)

def stom_ctr_similarity(F, prev, T, N, D, strides, sim, stream=None):
    """F: device tensor of T x N x D features (strides = (frame, token) in elements); prev: [N][D] or None."""
    sf, st = strides
    _check(lib().stom_ctr_similarity(_ptr(F), _ptr(prev), C.c_int32(dtype_code(F.dtype)), C.c_int32(T), C.c_int32(N),
                                     C.c_int32(D), C.c_int64(sf), C.c_int64(st), _ptr(sim), _stream(stream)),
           "stom_ctr_similarity")


def stom_ctr_select(sim, alpha, T, N, G, tau_c, k_s, k_d, static_idx, dyn_idx, stream=None):
    _check(lib().stom_ctr_select(_ptr(sim), _ptr(alpha), C.c_int32(T), C.c_int32(N), C.c_int32(G), C.c_float(tau_c),
                                 _ptr(k_s), _ptr(k_d), _ptr(static_idx), _ptr(dyn_idx), _stream(stream)),
           "stom_ctr_select")


def stom_ctr_reduce(F, prev, T, N, D, strides, alpha, G, tau_c, sim, k_s, k_d, static_idx, dyn_idx, stream=None):
    sf, st = strides
    _check(lib().stom_ctr_reduce(_ptr(F), _ptr(prev), C.c_int32(dtype_code(F.dtype)), C.c_int32(T), C.c_int32(N),
                                 C.c_int32(D), C.c_int64(sf), C.c_int64(st), _ptr(alpha), C.c_int32(G),
                                 C.c_float(tau_c), _ptr(sim), _ptr(k_s), _ptr(k_d), _ptr(static_idx), _ptr(dyn_idx),
                                 _stream(stream)), "stom_ctr_reduce")


def stom_ctr_merge(F, T, N, D, strides, k_s, k_d, static_idx, dyn_idx, G, knn, retained, retained_pos, centre=None,
                   assign=None, dev_flags=None, stream=None):
    """Merge_{k_s} of the static tokens and the retained group [T][G][D] (see include/stom_ctr.h for the rule)."""
    sf, st = strides
    _check(lib().stom_ctr_merge(_ptr(F), C.c_int32(dtype_code(F.dtype)), C.c_int32(T), C.c_int32(N), C.c_int32(D),
                                C.c_int64(sf), C.c_int64(st), _ptr(k_s), _ptr(k_d), _ptr(static_idx), _ptr(dyn_idx),
                                C.c_int32(G), C.c_int32(knn), _ptr(retained), _ptr(retained_pos), _ptr(centre),
                                _ptr(assign), _ptr(dev_flags), _stream(stream)), "stom_ctr_merge")


def stom_ctr_reduce_tokens(F, prev, T, N, D, strides, alpha, G, tau_c, knn, sim, k_s, k_d, static_idx, dyn_idx, retained,
                           retained_pos, dev_flags=None, stream=None):
    sf, st = strides
    _check(lib().stom_ctr_reduce_tokens(_ptr(F), _ptr(prev), C.c_int32(dtype_code(F.dtype)), C.c_int32(T), C.c_int32(N),
                                        C.c_int32(D), C.c_int64(sf), C.c_int64(st), _ptr(alpha), C.c_int32(G),
                                        C.c_float(tau_c), C.c_int32(knn), _ptr(sim), _ptr(k_s), _ptr(k_d),
                                        _ptr(static_idx), _ptr(dyn_idx), _ptr(retained), _ptr(retained_pos),
                                        _ptr(dev_flags), _stream(stream)), "stom_ctr_reduce_tokens")
