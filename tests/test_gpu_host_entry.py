"""GPU parity of the entry points that take HOST buffers (`stom_oqm_quantize_frame_host`,
`stom_oqm_retrieve_host`): the path a caller drives from host memory, and the one the end-to-end figure of the
benchmark runs through.

A stream is quantized through the host call in several chunks of unequal length (each chunk a compact host array, as
the call wants it), then one question goes through the host retrieval call.  The bank, the indices that come back in
host memory and the reconstructed K/V cache that comes back in host memory are compared with the CPU oracle under
the rules of tests/_parity.py (codes and scales bit-exact, selections identical up to score ties, reconstructed
groups bit-identical).  Also covered: the variant that leaves the cache on the device (NULL cache pointers), a bank
with fewer groups than asked for (unused slots -1, their tokens zero), and scratch that is missing or too small
(STOM_ERR_WORKSPACE, nothing launched)."""
import numpy as np
import pytest
import torch

import _parity as P
from paper_2510_18269_b200 import synth

pytestmark = pytest.mark.gpu


def _aligned(nbytes, fill=None):
    t = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda") if fill is None else \
        torch.full((nbytes + 256,), fill, dtype=torch.uint8, device="cuda")
    return t[(-t.data_ptr()) % 256:][:nbytes]


def _quantize_in_chunks(oqm, cfg, st, sh, K, V, chunks, flags):
    """K, V: host tensors [L][T][H_k][G][d]; every chunk is sent as its own compact pinned array."""
    f0 = 0
    for n in chunks:
        Kh = K[:, f0:f0 + n].contiguous().pin_memory()
        Vh = V[:, f0:f0 + n].contiguous().pin_memory()
        scr = _aligned(oqm.stom_oqm_quantize_host_scratch_bytes(cfg, sh.L, n))
        oqm.stom_oqm_quantize_frame_host(cfg, st, 0, sh.L, f0, n, Kh, Vh, scr, dev_flags=flags)
        torch.cuda.synchronize()      # the pinned chunk and its scratch go out of scope below
        f0 += n
    assert f0 == sh.T


@pytest.mark.parametrize("name,L,T,T_q,k,chunks", [
    ("C2-shaped", 1, 1024, 8, 32, (400, 1, 333, 290)),     # the 7B single layer, 51 200 tokens
    ("C3-shaped-short", 28, 96, 16, 64, (64, 31, 1)),      # all 28 layers of the 7B stack, a short stream
])
def test_host_entry_points_match_oracle(orc, name, L, T, T_q, k, chunks):
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    sh = synth.Shape(name, L=L, H_q=28, H_k=4, d=128, G=50, T=T, T_q=T_q, k=k, seed=321)
    K, V = synth.kv_stream(sh)
    Q = synth.queries(sh)
    gcfg, ocfg = P.gpu_cfg(oqm, sh), P.oracle_cfg(orc, sh)
    gst, ost = oqm.Store(gcfg), orc.Store(ocfg)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    _quantize_in_chunks(oqm, gcfg, gst, sh, K, V, chunks, flags)

    kn, vn = P.as_np16(K), P.as_np16(V)
    assert orc.quantize_frame(ocfg, ost, 0, L, 0, T, kn, vn, P.contiguous_strides(sh, sh.G)) == 0
    P.compare_store(gst, ost, P.f32_of(orc, kn, sh.dtype))

    # one question through the host call: Q up, indices and the reconstructed cache down
    S = k * sh.G
    Qh = Q.contiguous().pin_memory()
    idx_h = torch.full((L, k), -9, dtype=torch.int32).pin_memory()
    ka_h = torch.full((L, sh.H_k, S, sh.d), 3.0, dtype=torch.bfloat16).pin_memory()
    va_h = torch.full((L, sh.H_k, S, sh.d), 3.0, dtype=torch.bfloat16).pin_memory()
    scr = _aligned(oqm.stom_oqm_retrieve_host_scratch_bytes(gcfg, L, T, T_q, k, oqm.BF16), fill=0xAB)
    oqm.stom_oqm_retrieve_host(gcfg, gst, 0, L, T, Qh, T_q, k, idx_h, ka_h, va_h, oqm.BF16, scr, dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0

    o_scores = orc.score_groups(ocfg, ost, 0, L, T, P.as_np16(Q), T_q, P.q_strides(sh))
    o_idx, _, _ = orc.topk(o_scores.reshape(L, T), k)
    P.compare_topk(idx_h, o_idx, o_scores.reshape(L, T), k)
    oka = np.zeros((L, sh.H_k, S, sh.d), np.uint16)
    ova = np.zeros_like(oka)
    assert orc.dequant_gather(ocfg, ost, 0, L, o_idx, k, T, oka, ova, orc.BF16, P.active_strides(sh, S), 0) == 0
    g_idx = idx_h.numpy()
    P.compare_active(P.as_np16(ka_h), oka, g_idx, o_idx, 0, sh.G)
    P.compare_active(P.as_np16(va_h), ova, g_idx, o_idx, 0, sh.G)

    # the same question through the device-pointer call gives the same indices and the same cache, bit for bit
    scores = torch.empty(L, T, dtype=torch.float32, device="cuda")
    idx = torch.empty(L, k, dtype=torch.int32, device="cuda")
    ka = torch.zeros(L, sh.H_k, S, sh.d, dtype=torch.bfloat16, device="cuda")
    va = torch.zeros_like(ka)
    ws = _aligned(oqm.stom_oqm_retrieve_workspace_bytes(gcfg, L, T, k))
    oqm.stom_oqm_retrieve(gcfg, gst, 0, L, T, Q.cuda(), T_q, P.q_strides(sh), k, scores, idx, ka, va, oqm.BF16,
                          P.active_strides(sh, S), 0, ws, dev_flags=flags)
    torch.cuda.synchronize()
    assert torch.equal(idx.cpu(), idx_h)
    assert torch.equal(ka.cpu().view(torch.int16), ka_h.view(torch.int16))
    assert torch.equal(va.cpu().view(torch.int16), va_h.view(torch.int16))

    # NULL cache pointers: the cache stays on the device, only the indices come back
    idx_only = torch.full((L, k), -9, dtype=torch.int32).pin_memory()
    oqm.stom_oqm_retrieve_host(gcfg, gst, 0, L, T, Qh, T_q, k, idx_only, None, None, oqm.BF16, scr, dev_flags=flags)
    torch.cuda.synchronize()
    assert torch.equal(idx_only, idx_h)


def test_host_retrieve_with_fewer_groups_than_k_returns_unused_slots_as_minus_one_and_zero_tokens(orc):
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    sh = synth.Shape("few", L=2, H_q=8, H_k=4, d=128, G=50, T=5, T_q=3, k=8, seed=11)
    K, V = synth.kv_stream(sh)
    Q = synth.queries(sh)
    gcfg, ocfg = P.gpu_cfg(oqm, sh), P.oracle_cfg(orc, sh)
    gst, ost = oqm.Store(gcfg), orc.Store(ocfg)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    _quantize_in_chunks(oqm, gcfg, gst, sh, K, V, (2, 3), flags)
    assert orc.quantize_frame(ocfg, ost, 0, sh.L, 0, sh.T, P.as_np16(K), P.as_np16(V),
                              P.contiguous_strides(sh, sh.G)) == 0
    S = sh.k * sh.G
    idx_h = torch.full((sh.L, sh.k), -9, dtype=torch.int32).pin_memory()
    ka_h = torch.full((sh.L, sh.H_k, S, sh.d), 3.0, dtype=torch.bfloat16).pin_memory()
    va_h = torch.full((sh.L, sh.H_k, S, sh.d), 3.0, dtype=torch.bfloat16).pin_memory()
    scr = _aligned(oqm.stom_oqm_retrieve_host_scratch_bytes(gcfg, sh.L, sh.T, sh.T_q, sh.k, oqm.BF16), fill=0xAB)
    oqm.stom_oqm_retrieve_host(gcfg, gst, 0, sh.L, sh.T, Q.pin_memory(), sh.T_q, sh.k, idx_h, ka_h, va_h, oqm.BF16, scr,
                               dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    want = np.tile(np.concatenate([np.arange(sh.T), -np.ones(sh.k - sh.T)]).astype(np.int32), (sh.L, 1))
    assert np.array_equal(idx_h.numpy(), want)
    oka = np.zeros((sh.L, sh.H_k, S, sh.d), np.uint16)
    ova = np.zeros_like(oka)
    assert orc.dequant_gather(ocfg, ost, 0, sh.L, want, sh.k, sh.T, oka, ova, orc.BF16, P.active_strides(sh, S), 0) == 0
    assert np.array_equal(P.as_np16(ka_h), oka) and np.array_equal(P.as_np16(va_h), ova)   # zeros behind the 5 groups


def test_host_entry_points_reject_missing_or_small_scratch():
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    sh = synth.Shape("ws", L=2, H_q=8, H_k=4, d=128, G=50, T=6, T_q=3, k=4, seed=3)
    cfg = P.gpu_cfg(oqm, sh)
    st = oqm.Store(cfg)
    K, V = synth.kv_stream(sh)
    Kh, Vh = K.pin_memory(), V.pin_memory()
    before = {n: getattr(st, n).clone() for n in ("codes_k", "scale_k", "rep_key")}
    need = oqm.stom_oqm_quantize_host_scratch_bytes(cfg, sh.L, sh.T)
    with pytest.raises(oqm.StomError) as ei:
        oqm.stom_oqm_quantize_frame_host(cfg, st, 0, sh.L, 0, sh.T, Kh, Vh, _aligned(need - 256))
    assert ei.value.code == -8
    S = sh.k * sh.G
    idx_h = torch.full((sh.L, sh.k), -9, dtype=torch.int32).pin_memory()
    ka_h = torch.full((sh.L, sh.H_k, S, sh.d), 3.0, dtype=torch.bfloat16).pin_memory()
    va_h = ka_h.clone().pin_memory()
    need = oqm.stom_oqm_retrieve_host_scratch_bytes(cfg, sh.L, sh.T, sh.T_q, sh.k, oqm.BF16)
    Qh = synth.queries(sh).pin_memory()
    with pytest.raises(oqm.StomError) as ei:
        oqm.stom_oqm_retrieve_host(cfg, st, 0, sh.L, sh.T, Qh, sh.T_q, sh.k, idx_h, ka_h, va_h, oqm.BF16,
                                   _aligned(need - 256))
    assert ei.value.code == -8
    with pytest.raises(oqm.StomError) as ei:      # one cache pointer without the other
        oqm.stom_oqm_retrieve_host(cfg, st, 0, sh.L, sh.T, Qh, sh.T_q, sh.k, idx_h, ka_h, None, oqm.BF16, _aligned(need))
    assert ei.value.code == -1
    torch.cuda.synchronize()
    for n, t in before.items():
        assert torch.equal(getattr(st, n), t), "a rejected call must not touch the bank"
    assert torch.all(idx_h == -9) and torch.all(ka_h == 3.0)
