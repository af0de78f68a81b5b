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


def _bank(oqm, sh):
    K, V = synth.kv_stream(sh)
    cfg = P.gpu_cfg(oqm, sh)
    st = oqm.Store(cfg)
    oqm.stom_oqm_quantize_frame(cfg, st, 0, sh.L, 0, sh.T, K.cuda(), V.cuda(), P.contiguous_strides(sh, sh.G))
    torch.cuda.synchronize()
    return cfg, st


def test_noalloc_scores_equal_the_scratch_taking_entry_point_twice_in_a_row():
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    assert torch.cuda.is_available()
    sh = synth.Shape("noalloc", L=3, H_q=28, H_k=4, d=128, G=50, T=333, T_q=8, k=8, seed=77)
    cfg, st = _bank(oqm, sh)
    ws = torch.empty(oqm.stom_oqm_score_workspace_bytes(cfg, sh.L), dtype=torch.uint8, device="cuda")

    # call 1: all layers, question A;  call 2: layers 1..2 only, question B (other seed, other length)
    sh_b = dataclasses.replace(sh, seed=78, T_q=5)
    cases = [(sh, 0, sh.L), (sh_b, 1, 2)]
    for shq, l0, lc in cases:
        Q = synth.queries(shq).cuda()
        Ql = Q[l0:l0 + lc].contiguous()
        want = torch.full((lc * sh.T + P.GUARD,), -7.0, dtype=torch.float32, device="cuda")
        got = torch.full((lc * sh.T + P.GUARD,), -7.0, dtype=torch.float32, device="cuda")
        oqm.stom_oqm_score_groups(cfg, st, l0, lc, sh.T, Ql, shq.T_q, P.q_strides(shq), want, ws)
        oqm.stom_oqm_score_groups_noalloc(cfg, st, l0, lc, sh.T, Ql, shq.T_q, P.q_strides(shq), got)
        torch.cuda.synchronize()
        assert torch.all(got[lc * sh.T:] == -7.0), "guard band overwritten"
        err = (got[:lc * sh.T] - want[:lc * sh.T]).abs().max().item()
        assert err <= TOL, f"layers [{l0}, {l0 + lc}): scores differ by {err}"
        assert torch.isfinite(got[:lc * sh.T]).all() and got[:lc * sh.T].abs().max().item() <= 1.0 + TOL


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
