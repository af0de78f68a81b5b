"""The scoring entry point for hosts that cannot allocate device memory.

`stom_oqm_score_groups_noalloc` is meant for callers that have no way to hand the library
a scratch buffer: a process whose memory pool already owns the whole GPU, or code that is
not allowed to call the CUDA allocator because doing so would stall every stream of the
process.  It must return what `stom_oqm_score_groups` returns.  The array it keeps its
intermediate question embeddings in is shared by all calls and is never cleared, so the
check is made on two calls in a row with different questions and different layer ranges:
stale contents of the first call must not leak into the second.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import dataclasses

import pytest
import torch

import _parity as P
from paper_2510_18269_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5   # the absolute tolerance every score comparison of this suite uses


def _bank_on_both_sides(oqm, orc, sh):
    """The same stream quantized by the library (device bank) and by the oracle (host bank)."""
    K, V = synth.kv_stream(sh)
    cfg, ocfg = P.gpu_cfg(oqm, sh), P.oracle_cfg(orc, sh)
    st, ost = oqm.Store(cfg), orc.Store(ocfg)
    oqm.stom_oqm_quantize_frame(cfg, st, 0, sh.L, 0, sh.T, K.cuda(), V.cuda(), P.contiguous_strides(sh, sh.G))
    assert orc.quantize_frame(ocfg, ost, 0, sh.L, 0, sh.T, P.as_np16(K), P.as_np16(V),
                              P.contiguous_strides(sh, sh.G)) == 0
    torch.cuda.synchronize()
    return cfg, st, ocfg, ost


def test_noalloc_scores_equal_the_scratch_taking_entry_point_twice_in_a_row(orc):
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    assert torch.cuda.is_available()
    sh = synth.Shape("noalloc", L=3, H_q=28, H_k=4, d=128, G=50, T=333, T_q=8, k=8, seed=77)
    cfg, st, ocfg, ost = _bank_on_both_sides(oqm, orc, sh)
    ws = torch.empty(oqm.stom_oqm_score_workspace_bytes(cfg, sh.L), dtype=torch.uint8, device="cuda")

    # call 1: all layers, question A;  call 2: layers 1..2 only, question B (other seed, other length)
    sh_b = dataclasses.replace(sh, seed=78, T_q=5)
    cases = [(sh, 0, sh.L), (sh_b, 1, 2)]
    for call, (shq, l0, lc) in enumerate(cases):
        Q = synth.queries(shq)
        Ql = Q[l0:l0 + lc].contiguous().cuda()
        want = torch.full((lc * sh.T + P.GUARD,), -7.0, dtype=torch.float32, device="cuda")
        got = torch.full((lc * sh.T + P.GUARD,), -7.0, dtype=torch.float32, device="cuda")
        oqm.stom_oqm_score_groups(cfg, st, l0, lc, sh.T, Ql, shq.T_q, P.q_strides(shq), want, ws)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        oqm.stom_oqm_score_groups_noalloc(cfg, st, l0, lc, sh.T, Ql, shq.T_q, P.q_strides(shq), got)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if call > 0:   # the first call on a GPU may make the driver load the array's module; later ones take nothing
            assert free_after == free_before, "the call changed the amount of free device memory"
        assert torch.all(got[lc * sh.T:] == -7.0), "guard band overwritten"
        # same kernels on the same inputs: the sibling call's scores, bit for bit, and within the suite's
        # tolerance of the sibling (the check asked of this entry point)
        err = (got[:lc * sh.T] - want[:lc * sh.T]).abs().max().item()
        assert err <= TOL, f"layers [{l0}, {l0 + lc}): scores differ by {err}"
        assert torch.equal(got[:lc * sh.T], want[:lc * sh.T]), "scores are not bit-identical to the sibling call's"
        # and the oracle's scores for these layers, computed from the oracle's own bank
        o_scores = orc.score_groups(ocfg, ost, l0, lc, sh.T, P.as_np16(Q[l0:l0 + lc].contiguous()), shq.T_q,
                                    P.q_strides(shq))
        P.compare_scores(got[:lc * sh.T], o_scores)


def test_noalloc_rejects_a_layer_range_that_does_not_fit():
    from paper_2510_18269_b200 import oqm
    # 1 100 layers x 8 heads x 129 floats = 4.5 MB of embeddings: far beyond the built-in array
    cfg = oqm.make_config(1100, 64, 8, 128, 50, 4)
    assert oqm.stom_oqm_score_workspace_bytes(cfg, 1100) > oqm.NOALLOC_SCRATCH_BYTES
    st = oqm.Store(cfg)
    Q = torch.zeros(1100, 64, 1, 128, dtype=torch.bfloat16, device="cuda")
    scores = torch.full((1100 * 4,), -7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(oqm.StomError) as ei:
        oqm.stom_oqm_score_groups_noalloc(cfg, st, 0, 1100, 4, Q, 1, (64 * 128, 128, 128), scores)
    assert ei.value.code == -9
    torch.cuda.synchronize()
    assert torch.all(scores == -7.0), "a rejected call must not launch anything"
    # a range that fits goes through
    oqm.stom_oqm_score_groups_noalloc(cfg, st, 0, 100, 4, Q, 1, (64 * 128, 128, 128), scores)
    torch.cuda.synchronize()
