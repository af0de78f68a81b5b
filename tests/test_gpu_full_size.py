"""Parity at the sizes and in the launch configuration the benchmark times: the 7B-shaped 2-hour stream (28 layers,
7 200 frames of 50 tokens, 4 kv heads, d = 128; 20.6 GB of bf16 K/V) and the 72B-shaped stream (80 layers, 3 600
frames, 8 kv heads, 64 query heads, 32 question tokens; 59 GB of bf16 K/V), each quantized in ONE call over all
layers, then one question through the fused retrieval call.

The oracle cannot redo 20 GB in a test, so it redoes one whole layer (every frame of it: codes, scales, offsets,
representative keys, then that layer's 7 200 scores, its selection and its reconstructed cache) and a sample of
(layer, frame) units spread over the other layers, all from the SAME input bytes, copied from the device.  On top of
that, properties that hold at any size are checked on every layer: selections ascending and in range, and every
selected score at least as large as every score left out."""
import dataclasses

import numpy as np
import pytest
import torch

import _parity as P
from paper_2510_18269_b200 import synth

pytestmark = pytest.mark.gpu


def test_c3_full_stream_one_layer_in_full_and_samples_elsewhere(orc):
    _full_stream(orc, synth.C3, lf=13, need_gib=40)


def test_c5_full_stream_one_layer_in_full_and_samples_elsewhere(orc):
    _full_stream(orc, synth.C5, lf=47, need_gib=100)


def _full_stream(orc, sh, lf, need_gib):
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < need_gib * 2 ** 30:
        pytest.skip(f"needs {need_gib} GB of free device memory")
    dev = torch.device("cuda")
    gcfg = P.gpu_cfg(oqm, sh)
    gst = oqm.Store(gcfg, device=dev, zero=False)
    K, V = synth.kv_stream(sh, dev)
    Q = synth.queries(sh, dev)
    strides = P.contiguous_strides(sh, sh.G)
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    oqm.stom_oqm_quantize_frame(gcfg, gst, 0, sh.L, 0, sh.T, K, V, strides, dev_flags=flags)
    sys_len = 0
    S = sh.k * sh.G
    scores = torch.empty(sh.L, sh.T, dtype=torch.float32, device=dev)
    idx = torch.empty(sh.L, sh.k, dtype=torch.int32, device=dev)
    ka = torch.empty(sh.L, sh.H_k, S, sh.d, dtype=torch.bfloat16, device=dev)
    va = torch.empty_like(ka)
    ws = torch.empty(oqm.stom_oqm_retrieve_workspace_bytes(gcfg, sh.L, sh.T, sh.k), dtype=torch.uint8, device=dev)
    oqm.stom_oqm_retrieve(gcfg, gst, 0, sh.L, sh.T, Q, sh.T_q, P.q_strides(sh), sh.k, scores, idx, ka, va, oqm.BF16,
                          P.active_strides(sh, S), sys_len, ws, dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0

    # ---- properties on every layer
    sc_all = scores.cpu().numpy()
    ix_all = idx.cpu().numpy()
    for l in range(sh.L):
        sel = ix_all[l]
        assert np.all((sel >= 0) & (sel < sh.T)) and np.all(np.diff(sel) > 0)
        rest = np.ones(sh.T, bool)
        rest[sel] = False
        assert sc_all[l, sel].min() >= sc_all[l, rest].max(), f"layer {l}: a left-out group outscores a selected one"

    # ---- one layer in full
    one = dataclasses.replace(sh, L=1)
    ocfg = P.oracle_cfg(orc, one)
    ost = orc.Store(ocfg)
    kn, vn = P.as_np16(K[lf:lf + 1]), P.as_np16(V[lf:lf + 1])
    assert orc.quantize_frame(ocfg, ost, 0, 1, 0, sh.T, kn, vn, P.contiguous_strides(one, sh.G)) == 0
    for name in ("codes_k", "codes_v"):
        assert np.array_equal(getattr(gst, name)[lf].cpu().numpy(), getattr(ost, name)[0]), f"{name}: packed bytes differ"
    for name in ("scale_k", "scale_v"):
        assert np.array_equal(getattr(gst, name)[lf].cpu().numpy().view(np.uint32), getattr(ost, name)[0].view(np.uint32))
    for name in ("zero_k", "zero_v"):
        assert np.array_equal(getattr(gst, name)[lf].cpu().numpy(), getattr(ost, name)[0])
    kf = orc.to_f32(kn, P.dt_code(sh.dtype))[0]                                    # [T][H][G][d]
    tol = 2.0 ** -24 * np.abs(kf).astype(np.float64).sum(axis=-2) + 2.0 ** -23 * np.abs(ost.rep_key[0]) + 1e-30
    assert np.all(np.abs(gst.rep_key[lf].cpu().numpy().astype(np.float64) - ost.rep_key[0]) <= tol)
    o_scores = orc.score_groups(ocfg, ost, 0, 1, sh.T, P.as_np16(Q[lf:lf + 1]), sh.T_q, P.q_strides(sh))
    P.compare_scores(scores[lf], o_scores.reshape(-1))
    o_idx, _, _ = orc.topk(o_scores.reshape(1, sh.T), sh.k)
    P.compare_topk(idx[lf:lf + 1], o_idx, o_scores.reshape(1, sh.T), sh.k)
    oka = np.zeros((1, sh.H_k, S, sh.d), np.uint16)
    ova = np.zeros_like(oka)
    assert orc.dequant_gather(ocfg, ost, 0, 1, o_idx, sh.k, sh.T, oka, ova, orc.BF16, P.active_strides(sh, S), 0) == 0
    P.compare_active(P.as_np16(ka[lf])[None], oka, ix_all[lf:lf + 1], o_idx, 0, sh.G)
    P.compare_active(P.as_np16(va[lf])[None], ova, ix_all[lf:lf + 1], o_idx, 0, sh.G)

    # ---- sampled (layer, frame) units of the other layers, first and last frames included
    rng = np.random.default_rng(0)
    units = [(0, 0), (0, sh.T - 1), (sh.L - 1, 0), (sh.L - 1, sh.T - 1)]
    units += [(int(rng.integers(sh.L)), int(rng.integers(sh.T))) for _ in range(60)]
    tiny = dataclasses.replace(sh, L=1, T=1)
    tcfg = P.oracle_cfg(orc, tiny)
    for l, f in units:
        tst = orc.Store(tcfg)
        kk, vv = P.as_np16(K[l, f][None, None]), P.as_np16(V[l, f][None, None])
        assert orc.quantize_frame(tcfg, tst, 0, 1, 0, 1, kk, vv, P.contiguous_strides(tiny, sh.G)) == 0
        for name in ("codes_k", "codes_v", "zero_k", "zero_v"):
            assert np.array_equal(getattr(gst, name)[l, f].cpu().numpy(), getattr(tst, name)[0, 0]), f"{name} at {(l, f)}"
        for name in ("scale_k", "scale_v"):
            assert np.array_equal(getattr(gst, name)[l, f].cpu().numpy().view(np.uint32),
                                  getattr(tst, name)[0, 0].view(np.uint32)), f"{name} at {(l, f)}"
        assert np.allclose(gst.rep_key[l, f].cpu().numpy(), tst.rep_key[0, 0], rtol=0, atol=1e-5)
        assert np.allclose(gst.rep_norm2[l, f].cpu().numpy(), tst.rep_norm2[0, 0], rtol=1e-5, atol=1e-30)
