"""The streaming interleave end to end (at a small geometry, and at the 7B stack's own: 28 layers, 240 frames), CUDA
library against the oracle driven by the same call sequence: frames of
196 tokens arrive one at a time, 50 of them are kept by a seeded mask, quantized and appended; every few frames a
question is scored against what has been stored so far, the top groups are selected and reconstructed behind the
system tokens, and one decode step attends over the result.  Checked at every question: scores, selection, the
reconstructed cache (bit for bit), the size of the active cache (system tokens + K*G with K = min(k, stored groups),
whatever the stream length), and the attention output; at the end: the whole bank."""
import dataclasses

import numpy as np
import torch

import pytest

import _parity as P
from paper_2510_18269_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,geom,every,sys_len", [
    ("C4-small", dict(L=2, H_q=8, H_k=4, T=40, T_q=5, k=8), 6, 11),
    # the 7B stack as it streams: all 28 layers, 240 frames, a question every 60 frames, 64 groups + 32 system tokens
    ("C4-7B-240-frames", dict(L=28, H_q=28, H_k=4, T=240, T_q=16, k=64), 60, 32),
])
def test_streaming_interleave_matches_oracle(orc, name, geom, every, sys_len):
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    sh = dataclasses.replace(synth.C4, name=name, **geom)
    need = 2 * sh.L * sh.T * sh.H_k * sh.N_in * sh.d * 2 * 1.5
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip("not enough free device memory for this stream")
    K, V = synth.kv_stream(sh)                                       # [L][T][H_k][196][d]
    keep = synth.keep_mask(sh, 0, sh.T)                              # [T][50]
    ocfg, gcfg = P.oracle_cfg(orc, sh), P.gpu_cfg(oqm, sh)
    ost, gst = orc.Store(ocfg), oqm.Store(gcfg)
    Kd, Vd, keep_d = K.cuda(), V.cuda(), keep.cuda()
    kn, vn = P.as_np16(K), P.as_np16(V)
    strides = P.contiguous_strides(sh, sh.N_in)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    S = sys_len + sh.k * sh.G
    gen = torch.Generator().manual_seed(8)
    sys_k = torch.randn(sh.L, sh.H_k, sys_len, sh.d, generator=gen).to(torch.bfloat16)
    sys_v = torch.randn(sh.L, sh.H_k, sys_len, sh.d, generator=gen).to(torch.bfloat16)
    ws = torch.empty(oqm.stom_oqm_retrieve_workspace_bytes(gcfg, sh.L, sh.T, sh.k), dtype=torch.uint8, device="cuda")
    aws = torch.zeros(oqm.stom_oqm_attend_workspace_bytes(gcfg, sh.L, sh.k, sys_len) + 256, dtype=torch.uint8, device="cuda")
    aws = aws[(-aws.data_ptr()) % 256:]
    n_questions = 0
    for f in range(sh.T):
        # ---- ingest one frame (all layers in one call)
        off = f * strides[1]
        oqm.stom_oqm_quantize_frame(gcfg, gst, 0, sh.L, f, 1, Kd.view(-1)[off:], Vd.view(-1)[off:], strides,
                                    token_idx=keep_d[f:f + 1], tokens_per_frame_in=sh.N_in, dev_flags=flags)
        assert orc.quantize_frame(ocfg, ost, 0, sh.L, f, 1, kn.reshape(-1)[off:], vn.reshape(-1)[off:], strides,
                                  token_idx=keep[f:f + 1].numpy(), tokens_per_frame_in=sh.N_in) == 0
        if (f + 1) % every:
            continue
        # ---- a question over the f + 1 groups stored so far
        n_questions += 1
        n = f + 1
        qsh = dataclasses.replace(sh, seed=sh.seed + n)
        Q = synth.queries(qsh)
        o_scores = orc.score_groups(ocfg, ost, 0, sh.L, n, P.as_np16(Q), sh.T_q, P.q_strides(sh))
        o_idx, _, o_nsel = orc.topk(o_scores.reshape(sh.L, n), sh.k)
        ka = torch.zeros(sh.L, sh.H_k, S, sh.d, dtype=torch.bfloat16)
        va = torch.zeros_like(ka)
        ka[:, :, :sys_len], va[:, :, :sys_len] = sys_k, sys_v
        oka, ova = P.as_np16(ka).copy(), P.as_np16(va).copy()
        ka, va = ka.cuda(), va.cuda()
        scores = torch.empty(sh.L, n, dtype=torch.float32, device="cuda")
        idx = torch.empty(sh.L, sh.k, dtype=torch.int32, device="cuda")
        oqm.stom_oqm_retrieve(gcfg, gst, 0, sh.L, n, Q.cuda(), sh.T_q, P.q_strides(sh), sh.k, scores, idx, ka, va,
                              oqm.BF16, P.active_strides(sh, S), sys_len, ws, dev_flags=flags)
        torch.cuda.synchronize()
        P.compare_scores(scores, o_scores)
        P.compare_topk(idx, o_idx, o_scores.reshape(sh.L, n), sh.k)
        K_sel = min(sh.k, n)
        assert np.all(o_nsel == K_sel)
        g_idx = idx.cpu().numpy()
        assert np.all(g_idx[:, :K_sel] >= 0) and np.all(g_idx[:, K_sel:] == -1)
        assert orc.dequant_gather(ocfg, ost, 0, sh.L, o_idx, sh.k, n, oka, ova, orc.BF16, P.active_strides(sh, S),
                                  sys_len) == 0
        same_k = P.compare_active(P.as_np16(ka), oka, g_idx, o_idx, sys_len, sh.G)
        same_v = P.compare_active(P.as_np16(va), ova, g_idx, o_idx, sys_len, sh.G)
        assert np.array_equal(same_k, same_v) and same_k.any()
        # the active cache never exceeds the system tokens plus K groups, however long the stream is
        n_active = sys_len + K_sel * sh.G
        assert n_active <= S and torch.all(ka[:, :, n_active:] == 0)
        # ---- one decode step over [system tokens || selected groups]
        q_dec = torch.randn(sh.L, sh.H_q, sh.d, generator=gen).to(torch.bfloat16)
        out = torch.zeros(sh.L, sh.H_q, sh.d, dtype=torch.bfloat16, device="cuda")
        scale = 1.0 / np.sqrt(sh.d)
        oqm.stom_oqm_attend(gcfg, gst, 0, sh.L, idx, sh.k, n, q_dec.cuda(), (sh.H_q * sh.d, sh.d), ka, va, oqm.BF16,
                            P.active_strides(sh, S), sys_len, float(scale), out, (sh.H_q * sh.d, sh.d), aws,
                            dev_flags=flags)
        torch.cuda.synchronize()
        qn = P.as_np16(q_dec)
        want = np.stack([orc.to_f32(orc.attend(sh.H_q, sh.H_k, sh.d, qn[l], orc.BF16, oka[l], ova[l], orc.BF16,
                                               S * sh.d, sh.d, n_active, scale, out_dtype=orc.BF16), orc.BF16)
                         for l in range(sh.L)])
        got = orc.to_f32(P.as_np16(out), orc.BF16)
        # layers whose selection matches the oracle's slot for slot (all of them unless the K-th score is tied)
        assert np.all(np.abs(got - want)[same_k] <= np.maximum(2e-2, 2.0 ** -7 * np.abs(want))[same_k])
    assert n_questions == sh.T // every and int(flags.item()) == 0
    Kkept = orc.to_f32(kn, P.dt_code(sh.dtype)).transpose(0, 1, 2, 3, 4)
    Kkept = np.stack([Kkept[:, f][:, :, keep[f].numpy()] for f in range(sh.T)], axis=1)      # [L][T][H][G][d]
    P.compare_store(gst, ost, Kkept)


def test_question_sequence_replays_from_a_cuda_graph(orc):
    """The per-question sequence (fused retrieval, gather, one decode-attention step) captured once into a CUDA graph
    and replayed: same selection, same reconstructed cache, same attention output as the direct calls, also after
    the bank has grown and the question changed between replays (the graph reads the same buffers)."""
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    sh = synth.Shape("graph", L=3, H_q=8, H_k=4, d=128, G=50, T=120, T_q=4, k=8, seed=77)
    ocfg, gcfg, ost, gst, _ = P.random_bank(orc, oqm, sh, 0, seed=5)
    sys_len = 6
    S = sys_len + sh.k * sh.G
    dev = "cuda"
    Q = synth.queries(sh).cuda()
    q_dec = torch.randn(sh.L, sh.H_q, sh.d, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16).cuda()
    scores = torch.zeros(sh.L, sh.T, dtype=torch.float32, device=dev)
    idx = torch.zeros(sh.L, sh.k, dtype=torch.int32, device=dev)
    ka = torch.randn(sh.L, sh.H_k, S, sh.d, generator=torch.Generator().manual_seed(4)).to(torch.bfloat16).cuda()
    va = ka.clone()
    out = torch.zeros(sh.L, sh.H_q, sh.d, dtype=torch.bfloat16, device=dev)
    ws = torch.empty(oqm.stom_oqm_retrieve_workspace_bytes(gcfg, sh.L, sh.T, sh.k), dtype=torch.uint8, device=dev)
    aws = torch.zeros(oqm.stom_oqm_attend_workspace_bytes(gcfg, sh.L, sh.k, sys_len) + 256, dtype=torch.uint8, device=dev)
    aws = aws[(-aws.data_ptr()) % 256:]
    flags = torch.zeros(1, dtype=torch.int32, device=dev)

    def question():
        oqm.stom_oqm_retrieve(gcfg, gst, 0, sh.L, sh.T, Q, sh.T_q, P.q_strides(sh), sh.k, scores, idx, ka, va, oqm.BF16,
                              P.active_strides(sh, S), sys_len, ws, dev_flags=flags)
        oqm.stom_oqm_attend(gcfg, gst, 0, sh.L, idx, sh.k, sh.T, q_dec, (sh.H_q * sh.d, sh.d), ka, va, oqm.BF16,
                            P.active_strides(sh, S), sys_len, float(sh.d) ** -0.5, out, (sh.H_q * sh.d, sh.d), aws,
                            dev_flags=flags)

    # warm up on a side stream (first use of each kernel), then capture
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        question()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        question()
    for trial in range(2):
        if trial == 1:   # another question against a changed bank, through the same buffers
            Q.copy_(synth.queries(dataclasses.replace(sh, seed=78)).cuda())
            gst.rep_key[:, 5:9].mul_(-1.0)
            ost.rep_key[:, 5:9] *= -1.0
        idx.fill_(-7); out.zero_(); scores.zero_()
        graph.replay()
        torch.cuda.synchronize()
        got = (scores.clone(), idx.clone(), ka.clone(), va.clone(), out.clone())
        idx.fill_(-7); out.zero_(); scores.zero_()
        question()
        torch.cuda.synchronize()
        for a, b in zip(got, (scores, idx, ka, va, out)):
            assert torch.equal(a, b)
        # and the replayed result is the oracle's
        o_scores = orc.score_groups(ocfg, ost, 0, sh.L, sh.T, P.as_np16(Q.cpu()), sh.T_q, P.q_strides(sh))
        o_idx, _, _ = orc.topk(o_scores.reshape(sh.L, sh.T), sh.k)
        P.compare_scores(got[0], o_scores)
        P.compare_topk(got[1], o_idx, o_scores.reshape(sh.L, sh.T), sh.k)
    assert int(flags.item()) == 0
