"""GPU parity of the fused retrieval call (question embedding + scores + top-K in one launch, then the
reconstruction) against the CPU oracle, at row lengths that exercise each way the selecting block holds its keys
(registers, shared memory, global memory), in both scoring modes and for every input type.

The bank is filled with seeded random arrays on both sides (representative keys with their norms, codes, scales,
offsets), so that long rows do not need a long quantization on the CPU first; the quantizer has its own tests.
Tolerances are those of tests/_parity.py."""
import numpy as np
import pytest
import torch

import _parity as P
from paper_2510_18269_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("L,H_q,H_k,d,G,T,T_q,k,mode,dtype", [
    (2, 28, 4, 128, 4, 7200, 16, 64, 0, "bf16"),   # 7B geometry, keys of the selecting block in shared memory
    (2, 16, 8, 128, 4, 3600, 5, 64, 0, "bf16"),    # 72B geometry (8 kv heads)
    (1, 4, 2, 64, 4, 11000, 3, 300, 0, "fp16"),    # row longer than the shared-memory key array
    (3, 8, 4, 128, 4, 1500, 4, 32, 1, "bf16"),     # one selection per kv head; keys in registers
    (2, 6, 2, 128, 2, 2500, 2, 2500, 0, "fp32"),   # every stored group selected
    (1, 2, 1, 256, 4, 40, 1, 64, 0, "bf16"),       # fewer groups stored than asked for
    (2, 6, 3, 128, 4, 333, 7, 16, 0, "bf16"),      # a head count the pipelined scorer does not cover
    (2, 6, 3, 128, 4, 333, 7, 16, 1, "fp16"),
])
@pytest.mark.parametrize("two_level_ws", [False, True])
def test_fused_retrieve_matches_oracle(orc, L, H_q, H_k, d, G, T, T_q, k, mode, dtype, two_level_ws):
    _check_fused(orc, L, H_q, H_k, d, G, T, T_q, k, mode, dtype, two_level_ws, {})


@pytest.mark.parametrize("L,H_q,H_k,d,G,T,T_q,k,mode,dtype,meta,bits", [
    (2, 28, 4, 128, 4, 7200, 16, 64, 0, "bf16", "bf16", 4),   # 7B geometry: two 16-byte vectors of k-bar per lane
    (2, 28, 4, 128, 4, 3000, 3, 64, 0, "bf16", "fp16", 4),
    (2, 16, 8, 128, 4, 3600, 5, 64, 0, "bf16", "fp16", 2),    # 72B geometry, 2-bit codes
    (1, 4, 2, 128, 4, 900, 3, 30, 0, "fp16", "fp16", 4),      # H*d = 256: one vector per lane
    (1, 2, 1, 128, 4, 500, 2, 20, 0, "bf16", "bf16", 4),      # H*d = 128: the general loop
    (2, 6, 3, 128, 4, 333, 7, 16, 1, "fp32", "bf16", 4),      # one selection per kv head
    (1, 4, 2, 64, 2, 700, 2, 9, 0, "fp32", "fp16", 4),
])
@pytest.mark.parametrize("two_level_ws", [False, True])
def test_fused_retrieve_sixteen_bit_metadata(orc, L, H_q, H_k, d, G, T, T_q, k, mode, dtype, meta, bits, two_level_ws):
    """s, m and k-bar stored in 16 bits: the same bank on both sides (values representable in the storage type)."""
    _check_fused(orc, L, H_q, H_k, d, G, T, T_q, k, mode, dtype, two_level_ws, {"meta": meta, "bits": bits})


def _check_fused(orc, L, H_q, H_k, d, G, T, T_q, k, mode, dtype, two_level_ws, extra):
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    sh = synth.Shape("fused", L=L, H_q=H_q, H_k=H_k, d=d, G=G, T=T, T_q=T_q, k=k, dtype=dtype, seed=5, extra=extra)
    ocfg, gcfg, ost, gst, u = P.random_bank(orc, oqm, sh, mode, seed=T + k)
    rows = L * (H_k if mode else 1)
    rep = H_q // H_k
    g = torch.Generator().manual_seed(99)
    base = torch.from_numpy(u[:, 0]).repeat_interleave(rep, dim=1)[:, :, None, :]
    Q = (base + 0.5 * torch.randn(L, H_q, T_q, d, generator=g)).to(synth.DTYPES[dtype]).contiguous()

    o_scores = orc.score_groups(ocfg, ost, 0, L, T, P.as_np16(Q), T_q, P.q_strides(sh))
    o_idx, _, _ = orc.topk(o_scores.reshape(rows, T), k)

    sys_len = 3
    S = sys_len + k * G + 1
    ka_flat, ka = P.out_buffers(sh, L, S, torch.bfloat16, "cuda", 3.0)
    va_flat, va = P.out_buffers(sh, L, S, torch.bfloat16, "cuda", 3.0)
    scores = torch.full((rows * T + P.GUARD,), -7.0, dtype=torch.float32, device="cuda")
    idx = torch.full((rows * k + P.GUARD,), -9, dtype=torch.int32, device="cuda")
    # the small workspace keeps the selection in the completing block; the large one lets every block pre-select
    nbytes = oqm.stom_oqm_retrieve_workspace_bytes(gcfg, L, T, k) if two_level_ws else oqm.stom_oqm_score_workspace_bytes(gcfg, L)
    ws = torch.full((nbytes + 256,), 0xAB, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(2):   # twice: the second call finds the layer counters as the first one left them
        oqm.stom_oqm_retrieve(gcfg, gst, 0, L, T, Q.cuda(), T_q, P.q_strides(sh), k, scores, idx, ka, va, oqm.BF16,
                              P.active_strides(sh, S), sys_len, ws, dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    assert torch.all(scores[rows * T:] == -7.0) and torch.all(idx[rows * k:] == -9), "guard band overwritten"
    P.compare_scores(scores[:rows * T], o_scores)
    P.compare_topk(idx[:rows * k], o_idx, o_scores.reshape(rows, T), k)

    # reconstruction: the oracle gathers ITS selection; slots where the library selected the same group are compared
    g_idx = idx[:rows * k].view(rows, k).cpu().numpy()
    sent = P.as_np16(torch.tensor([3.0], dtype=torch.bfloat16))[0]
    oka = np.full((L, H_k, S, d), sent, np.uint16)
    ova = np.full((L, H_k, S, d), sent, np.uint16)
    assert orc.dequant_gather(ocfg, ost, 0, L, o_idx, k, T, oka, ova, orc.BF16, P.active_strides(sh, S), sys_len) == 0
    n_el = L * H_k * S * d
    for flat, o16 in ((ka_flat, oka), (va_flat, ova)):
        assert torch.all(flat[n_el:] == 3.0), "guard band overwritten"
        P.compare_active(P.as_np16(flat[:n_el]).reshape(o16.shape), o16, g_idx, o_idx, sys_len, G, per_head=bool(mode))


def test_fused_retrieve_on_an_empty_bank_marks_every_slot_unused(orc):
    from paper_2510_18269_b200 import oqm
    sh = synth.Shape("empty", L=2, H_q=4, H_k=2, d=128, G=4, T=8, T_q=2, k=4, seed=1)
    gcfg = P.gpu_cfg(oqm, sh)
    gst = oqm.Store(gcfg)
    Q = synth.queries(sh).cuda()
    S = sh.k * sh.G
    _, ka = P.out_buffers(sh, sh.L, S, torch.bfloat16, "cuda", 3.0)
    _, va = P.out_buffers(sh, sh.L, S, torch.bfloat16, "cuda", 3.0)
    scores = torch.zeros(sh.L * sh.T, dtype=torch.float32, device="cuda")
    idx = torch.zeros(sh.L * sh.k, dtype=torch.int32, device="cuda")
    ws = torch.empty(oqm.stom_oqm_score_workspace_bytes(gcfg, sh.L), dtype=torch.uint8, device="cuda")
    oqm.stom_oqm_retrieve(gcfg, gst, 0, sh.L, 0, Q, sh.T_q, P.q_strides(sh), sh.k, scores, idx, ka, va, oqm.BF16,
                          P.active_strides(sh, S), 0, ws)
    torch.cuda.synchronize()
    assert torch.all(idx == -1) and torch.all(ka == 3.0) and torch.all(va == 3.0)


@pytest.mark.parametrize("copies", [3, 40, 200, "all"])
def test_fused_retrieve_equal_scores_go_to_the_lower_index(orc, copies):
    """Stored groups with identical representative keys score identically; which of them make the top-K is then
    decided by index alone (the lower one wins), although the candidates reach the completing block from several
    blocks' pre-selections.  Cases: a few copies of the group ranked around K, many, and a bank of identical groups.
    Expected: the stable ordering (score descending, index ascending) of the scores the call itself wrote, cut at
    K, ascending; the scores are checked against the oracle as everywhere else."""
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    L, H_q, H_k, d, G, T, T_q, k = 2, 28, 4, 128, 4, 2400, 4, 64
    sh = synth.Shape("ties", L=L, H_q=H_q, H_k=H_k, d=d, G=G, T=T, T_q=T_q, k=k, dtype="bf16", seed=5, extra={})
    ocfg, gcfg, ost, gst, u = P.random_bank(orc, oqm, sh, 0, seed=77)
    g = torch.Generator().manual_seed(3)
    base = torch.from_numpy(u[:, 0]).repeat_interleave(H_q // H_k, dim=1)[:, :, None, :]
    Q = (base + 0.5 * torch.randn(L, H_q, T_q, d, generator=g)).to(torch.bfloat16).contiguous()
    # the group the oracle ranks K-th in layer 0 is copied over other slots, spread over the bank
    o_scores = orc.score_groups(ocfg, ost, 0, L, T, P.as_np16(Q), T_q, P.q_strides(sh))
    kth = int(np.argsort(-o_scores[0], kind="stable")[k - 1])
    rng = np.random.default_rng(11)
    where = np.arange(T) if copies == "all" else rng.choice(T, size=copies, replace=False)
    for l in range(L):
        ost.rep_key[l, where] = ost.rep_key[l, kth]
        ost.rep_norm2[l, where] = ost.rep_norm2[l, kth]
    gst.rep_key.copy_(torch.from_numpy(ost.rep_key))
    gst.rep_norm2.copy_(torch.from_numpy(ost.rep_norm2))
    o_scores = orc.score_groups(ocfg, ost, 0, L, T, P.as_np16(Q), T_q, P.q_strides(sh))

    S = k * G
    _, ka = P.out_buffers(sh, L, S, torch.bfloat16, "cuda", 3.0)
    _, va = P.out_buffers(sh, L, S, torch.bfloat16, "cuda", 3.0)
    scores = torch.empty(L * T, dtype=torch.float32, device="cuda")
    idx = torch.full((L * k,), -9, dtype=torch.int32, device="cuda")
    ws = torch.full((oqm.stom_oqm_retrieve_workspace_bytes(gcfg, L, T, k) + 256,), 0xAB, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    oqm.stom_oqm_retrieve(gcfg, gst, 0, L, T, Q.cuda(), T_q, P.q_strides(sh), k, scores, idx, ka, va, oqm.BF16,
                          P.active_strides(sh, S), 0, ws)
    torch.cuda.synchronize()
    P.compare_scores(scores, o_scores)
    got_scores = scores.view(L, T).cpu().numpy()
    got = idx.view(L, k).cpu().numpy()
    for l in range(L):
        same = got_scores[l, where]
        assert np.all(same == same[0]), "identical groups must score identically"
        order = np.lexsort((np.arange(T), -got_scores[l].astype(np.float64)))  # score descending, then index ascending
        assert np.array_equal(got[l], np.sort(order[:k])), f"layer {l}"
