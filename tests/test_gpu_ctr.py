"""GPU parity of the CTR steps the library implements (temporal similarity, static / dynamic split, budget,
saliency selection of the dynamic tokens; paper Sec. 3.3) against the CPU oracle.

Tolerances: similarity 1e-5 absolute (binary32 accumulation over D channels against binary64); every integer output
of stom_ctr_select bit-exact when both sides are given the same similarities (the oracle's, uploaded).  For the
chained call the library's own similarities decide the split, so a frame is compared exactly unless one of its
tokens has an oracle similarity within 1e-5 of tau_c, where either side of the threshold is a correct answer."""
import numpy as np
import pytest
import torch

import _parity as P
from paper_2510_18269_b200 import synth

pytestmark = pytest.mark.gpu
TAU = 0.9


def _lib():
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    return oqm


def _select_outputs(T, N, G):
    dev = "cuda"
    return (torch.full((T + P.GUARD,), -9, dtype=torch.int32, device=dev), torch.full((T + P.GUARD,), -9, dtype=torch.int32, device=dev),
            torch.full((T * N + P.GUARD,), -9, dtype=torch.int32, device=dev), torch.full((T * G + P.GUARD,), -9, dtype=torch.int32, device=dev))


@pytest.mark.parametrize("T,N,D,dtype", [
    (70, 196, 1152, "bf16"),    # the 7B model's encoder: 196 tokens of 1152 channels; two runs of frames and a tail
    (33, 49, 1024, "fp16"),     # one frame more than a run
    (5, 196, 4104, None),       # wider than the kernels cover: must be refused (see below)
    (9, 60, 3584, "bf16"),      # the language model's width (features after the projector)
    (4, 7, 4096, "fp16"),       # the widest 16-bit row
    (12, 64, 72, "fp16"),       # a row narrower than one warp pass
    (40, 100, 1024, "fp32"),
    (1, 196, 1152, "bf16"),     # a single frame
])
def test_similarity_matches_oracle(orc, T, N, D, dtype):
    oqm = _lib()
    if dtype is None:
        F = torch.zeros(T, N, D, dtype=torch.bfloat16, device="cuda")
        sim = torch.zeros(T, N, dtype=torch.float32, device="cuda")
        with pytest.raises(oqm.StomError) as e:
            oqm.stom_ctr_similarity(F, None, T, N, D, (N * D, D), sim)
        assert e.value.code == -2
        return
    F, _ = synth.ctr_stream(T, N, D, seed=T + N, dtype=dtype)
    prev, _ = synth.ctr_stream(1, N, D, seed=T + N + 1, dtype=dtype)
    Fn = P.as_np16(F)
    for with_prev in (False, True):
        sim = torch.full((T * N + P.GUARD,), -7.0, dtype=torch.float32, device="cuda")
        oqm.stom_ctr_similarity(F.cuda(), prev[0].cuda() if with_prev else None, T, N, D, (N * D, D), sim)
        torch.cuda.synchronize()
        assert torch.all(sim[T * N:] == -7.0), "guard band overwritten"
        got = sim[:T * N].view(T, N).cpu().numpy()
        want = orc.ctr_similarity(Fn, P.dt_code(dtype), prev=P.as_np16(prev[0]) if with_prev else None)
        if not with_prev:
            assert np.all(np.isneginf(got[0])) and np.all(np.isneginf(want[0]))
            got, want = got[1:], want[1:]
        assert np.abs(got.astype(np.float64) - want).max(initial=0.0) <= 1e-5


def test_similarity_strided_rows_and_zero_vectors(orc):
    oqm = _lib()
    T, N, D, pad = 6, 10, 64, 16
    F, _ = synth.ctr_stream(T, N, D, seed=3, dtype="bf16")
    F[2, 4] = 0          # zero vectors: similarity 0 on both frames that see them
    buf = torch.full((T, N, D + pad), 7.0, dtype=torch.bfloat16)
    buf[:, :, :D] = F
    sim = torch.zeros(T, N, dtype=torch.float32, device="cuda")
    oqm.stom_ctr_similarity(buf.cuda(), None, T, N, D, (N * (D + pad), D + pad), sim)
    want = orc.ctr_similarity(P.as_np16(F), orc.BF16)
    got = sim.cpu().numpy()
    assert got[2, 4] == 0.0 and got[3, 4] == 0.0 and want[2, 4] == 0.0
    assert np.abs(got[1:].astype(np.float64) - want[1:]).max() <= 1e-5


@pytest.mark.parametrize("T,N,G", [(64, 196, 50), (7, 1024, 300), (5, 9, 9), (3, 33, 1), (20, 256, 64)])
def test_select_is_bit_exact_on_the_same_similarities(orc, T, N, G):
    oqm = _lib()
    rng = np.random.default_rng(T * N + G)
    sim = rng.uniform(0.6, 1.0, (T, N)).astype(np.float32)
    sim[0] = -np.inf
    if T > 2:
        sim[1] = 0.99
        sim[2, : N // 2] = np.float32(TAU)           # exactly on the threshold: dynamic
    alpha = rng.uniform(0, 1, (T, N)).astype(np.float32)
    alpha[-1, ::2] = 0.25                            # equal saliencies: ties to the lower index
    ks, kd, sidx, didx = orc.ctr_select(sim, alpha, G, TAU)
    g_ks, g_kd, g_s, g_d = _select_outputs(T, N, G)
    oqm.stom_ctr_select(torch.from_numpy(sim).cuda(), torch.from_numpy(alpha).cuda(), T, N, G, TAU, g_ks, g_kd, g_s, g_d)
    torch.cuda.synchronize()
    for t, n in ((g_ks, T), (g_kd, T), (g_s, T * N), (g_d, T * G)):
        assert torch.all(t[n:] == -9), "guard band overwritten"
    assert np.array_equal(g_ks[:T].cpu().numpy(), ks) and np.array_equal(g_kd[:T].cpu().numpy(), kd)
    assert np.array_equal(g_s[:T * N].view(T, N).cpu().numpy(), sidx)
    assert np.array_equal(g_d[:T * G].view(T, G).cpu().numpy(), didx)


def test_reduce_chain_matches_oracle_frame_by_frame(orc):
    oqm = _lib()
    T, N, D, G = 150, 196, 1152, 50
    F, alpha = synth.ctr_stream(T, N, D, seed=11, dtype="bf16")
    o_sim = orc.ctr_similarity(P.as_np16(F), orc.BF16)
    ks, kd, sidx, didx = orc.ctr_select(o_sim, alpha.numpy(), G, TAU)
    sim = torch.zeros(T, N, dtype=torch.float32, device="cuda")
    g_ks, g_kd, g_s, g_d = _select_outputs(T, N, G)
    oqm.stom_ctr_reduce(F.cuda(), None, T, N, D, (N * D, D), alpha.cuda(), G, TAU, sim, g_ks, g_kd, g_s, g_d)
    torch.cuda.synchronize()
    got = sim.cpu().numpy()
    assert np.abs(got[1:].astype(np.float64) - o_sim[1:]).max() <= 1e-5
    clear = np.all(np.abs(o_sim - TAU) > 1e-5, axis=1)              # frames without a token on the threshold
    assert clear.mean() > 0.9
    assert np.array_equal(g_ks[:T].cpu().numpy()[clear], ks[clear]) and np.array_equal(g_kd[:T].cpu().numpy()[clear], kd[clear])
    assert np.array_equal(g_s[:T * N].view(T, N).cpu().numpy()[clear], sidx[clear])
    assert np.array_equal(g_d[:T * G].view(T, G).cpu().numpy()[clear], didx[clear])
    # the synthetic stream exercises both paths: some frames static-heavy, every frame with dynamic tokens
    assert ks[1:].min() >= 1 and kd.min() >= 1 and 0 < (o_sim[1:] > TAU).mean() < 1
