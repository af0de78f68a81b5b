"""GPU parity of the decode attention that dequantizes the selected groups on the fly (stom_oqm_attend) against the
CPU oracle: the oracle reconstructs the active cache (system tokens followed by the selected groups, rounded to
bf16 as a materialised cache holds them) and runs plain softmax attention over it in binary64.

Tolerance: 2e-2 absolute on the 16-bit output (the benchmark definition's figure for attention outputs), widened to
one unit in the last place of bfloat16 (2^-7 relative) where an output exceeds 2 in magnitude: there the spacing of
the output type itself is above 2e-2, and two correctly rounded results of nearby sums may land one step apart.
The kernel works from the unrounded reconstruction fmaf(code, s, m) and accumulates in binary32."""
import numpy as np
import pytest
import torch

import _parity as P
from paper_2510_18269_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _selection(rng, rows, T, k, n_sel):
    """[rows][k] ascending group ids, the last k - n_sel slots unused (-1), as the top-K call leaves them."""
    idx = np.full((rows, k), -1, np.int32)
    for r in range(rows):
        idx[r, :n_sel] = np.sort(rng.choice(T, size=n_sel, replace=False))
    return idx


@pytest.mark.parametrize("L,H_q,H_k,d,G,T,k,n_sel,sys_len,mode,dtype,cache", [
    (2, 28, 4, 128, 50, 200, 64, 64, 37, 0, "bf16", "bf16"),   # 7B geometry
    (1, 16, 2, 128, 50, 90, 24, 24, 5, 0, "bf16", "bf16"),     # 8 query heads per kv head (72B ratio)
    (2, 8, 4, 64, 16, 70, 9, 9, 130, 0, "fp16", "fp16"),       # three runs of system tokens, d = 64
    (1, 4, 2, 256, 64, 30, 10, 10, 3, 0, "bf16", "bf16"),      # d = 256, full 64-token groups
    (2, 8, 4, 128, 50, 120, 16, 16, 20, 1, "bf16", "bf16"),    # one selection per kv head
    (1, 8, 4, 128, 50, 60, 20, 13, 8, 0, "bf16", "bf16"),      # fewer groups stored than slots: trailing -1
    (1, 12, 1, 128, 7, 40, 11, 11, 0, 0, "fp32", "bf16"),      # 12 query heads on one kv head; no system tokens
    (1, 4, 4, 128, 50, 10, 8, 0, 70, 0, "bf16", "bf16"),       # nothing selected: system tokens only
])
def test_attend_matches_oracle(orc, L, H_q, H_k, d, G, T, k, n_sel, sys_len, mode, dtype, cache):
    _check_attend(orc, L, H_q, H_k, d, G, T, k, n_sel, sys_len, mode, dtype, cache, bits=4)


@pytest.mark.parametrize("L,H_q,H_k,d,G,T,k,n_sel,sys_len,mode,dtype,cache", [
    (2, 28, 4, 128, 50, 100, 16, 16, 9, 0, "bf16", "bf16"),
    (1, 4, 2, 64, 16, 40, 5, 4, 70, 1, "fp16", "fp16"),
    (1, 8, 1, 256, 8, 20, 6, 6, 0, 0, "bf16", "bf16"),
])
def test_attend_two_bit_codes(orc, L, H_q, H_k, d, G, T, k, n_sel, sys_len, mode, dtype, cache):
    _check_attend(orc, L, H_q, H_k, d, G, T, k, n_sel, sys_len, mode, dtype, cache, bits=2)


@pytest.mark.parametrize("L,H_q,H_k,d,G,T,k,n_sel,sys_len,mode,dtype,cache,meta,bits", [
    (2, 28, 4, 128, 50, 100, 16, 16, 9, 0, "bf16", "bf16", "bf16", 4),
    (2, 28, 4, 128, 50, 100, 16, 16, 9, 0, "bf16", "bf16", "fp16", 4),
    (1, 4, 2, 64, 16, 40, 5, 4, 70, 1, "fp16", "fp16", "fp16", 2),
    (1, 8, 1, 256, 8, 20, 6, 6, 0, 0, "fp32", "bf16", "bf16", 4),
])
def test_attend_sixteen_bit_metadata(orc, L, H_q, H_k, d, G, T, k, n_sel, sys_len, mode, dtype, cache, meta, bits):
    _check_attend(orc, L, H_q, H_k, d, G, T, k, n_sel, sys_len, mode, dtype, cache, bits=bits, meta=meta)


def _check_attend(orc, L, H_q, H_k, d, G, T, k, n_sel, sys_len, mode, dtype, cache, bits, meta="fp32"):
    from paper_2510_18269_b200 import oqm
    oqm.lib()
    sh = synth.Shape("attend", L=L, H_q=H_q, H_k=H_k, d=d, G=G, T=T, T_q=1, k=k, dtype=dtype, seed=3,
                     extra={"bits": bits, "meta": meta})
    ocfg, gcfg, ost, gst, _ = P.random_bank(orc, oqm, sh, mode, seed=17 * k + sys_len)
    rng = np.random.default_rng(5 + k)
    rows = L * (H_k if mode else 1)
    idx = _selection(rng, rows, T, k, n_sel)

    cdt = torch.bfloat16 if cache == "bf16" else torch.float16
    ccode = P.dt_code(cache)
    g = torch.Generator().manual_seed(21)
    q = torch.randn(L, H_q, d, generator=g).to(synth.DTYPES[dtype]).contiguous()
    S = sys_len + k * G
    k_act = torch.randn(L, H_k, S, d, generator=g).to(cdt).contiguous()     # system tokens in front, rest overwritten
    v_act = torch.randn(L, H_k, S, d, generator=g).to(cdt).contiguous()

    # oracle: materialise the cache, then plain attention over its first sys_len + n_sel*G tokens
    oka, ova = P.as_np16(k_act).copy(), P.as_np16(v_act).copy()
    assert orc.dequant_gather(ocfg, ost, 0, L, idx, k, T, oka, ova, ccode, P.active_strides(sh, S), sys_len) == 0
    n_tok = sys_len + n_sel * G
    scale = 1.0 / np.sqrt(d)
    qn = P.as_np16(q)
    want = np.stack([orc.to_f32(orc.attend(H_q, H_k, d, qn[l], P.dt_code(dtype), oka[l], ova[l], ccode, S * d, d,
                                           n_tok, scale, out_dtype=ccode), ccode) for l in range(L)])

    ws = torch.zeros(oqm.stom_oqm_attend_workspace_bytes(gcfg, L, k, sys_len) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    out_flat = torch.full((L * H_q * d + P.GUARD,), 3.0, dtype=cdt, device="cuda")
    out = out_flat[:L * H_q * d].view(L, H_q, d)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    ks, vs = k_act.cuda(), v_act.cuda()
    for _ in range(2):   # twice: the second call finds the counters as the first one left them
        oqm.stom_oqm_attend(gcfg, gst, 0, L, torch.from_numpy(idx).cuda(), k, T, q.cuda(), (H_q * d, d), ks, vs, ccode,
                            P.active_strides(sh, S), sys_len, float(scale), out, (H_q * d, d), ws, dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    assert torch.all(out_flat[L * H_q * d:] == 3.0), "guard band overwritten"
    got = orc.to_f32(P.as_np16(out), ccode)
    err = np.abs(got - want)
    tol = np.maximum(TOL, 2.0 ** -7 * np.abs(want))
    assert np.isfinite(got).all() and np.all(err <= tol), f"attention output differs by {err.max()}"
    assert err.mean() <= 0.2 * TOL, f"mean error {err.mean()} is too close to the tolerance to be rounding noise"
    assert np.abs(want).max() > 0.05, "degenerate case: outputs too small to mean anything"


def test_attend_flags_bad_indices_and_skips_them(orc):
    from paper_2510_18269_b200 import oqm
    sh = synth.Shape("attend-bad", L=1, H_q=4, H_k=2, d=128, G=8, T=12, T_q=1, k=4, seed=3)
    ocfg, gcfg, ost, gst, _ = P.random_bank(orc, oqm, sh, 0, seed=9)
    q = torch.randn(1, 4, 128).to(torch.bfloat16).cuda()
    ws = torch.zeros(oqm.stom_oqm_attend_workspace_bytes(gcfg, 1, 4, 0) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    outs = []
    for idx in ([1, 5, 99, -1], [1, 5, -1, -1]):   # 99 is out of range: skipped and flagged
        out = torch.zeros(1, 4, 128, dtype=torch.bfloat16, device="cuda")
        flags = torch.zeros(1, dtype=torch.int32, device="cuda")
        oqm.stom_oqm_attend(gcfg, gst, 0, 1, torch.tensor([idx], dtype=torch.int32).cuda(), 4, 12, q, (512, 128), None,
                            None, oqm.BF16, (0, 0, 128), 0, 0.088, out, (512, 128), ws, dev_flags=flags)
        torch.cuda.synchronize()
        outs.append((out.clone(), int(flags.item())))
    assert outs[0][1] == oqm.FLAG_BAD_INDEX and outs[1][1] == 0
    assert torch.equal(outs[0][0], outs[1][0])


def test_calls_over_any_layer_range_give_the_same_rows(orc):
    """A call over all layers, calls layer by layer and a call over a sub-range follow each other and give the same
    rows: the call keeps nothing between launches, whatever the workspace argument holds."""
    from paper_2510_18269_b200 import oqm
    sh = synth.Shape("attend-ws", L=5, H_q=14, H_k=2, d=128, G=50, T=40, T_q=1, k=6, seed=3)
    ocfg, gcfg, ost, gst, _ = P.random_bank(orc, oqm, sh, 0, seed=23)
    L, Hq, d, k, sys_len = sh.L, sh.H_q, sh.d, sh.k, 9
    rng = np.random.default_rng(2)
    idx = torch.from_numpy(_selection(rng, L, sh.T, k, k)).cuda()
    g = torch.Generator().manual_seed(8)
    q = torch.randn(L, Hq, d, generator=g).to(torch.bfloat16).cuda()
    S = sys_len + k * sh.G
    ks = torch.randn(L, sh.H_k, S, d, generator=g).to(torch.bfloat16).cuda()
    vs = torch.randn(L, sh.H_k, S, d, generator=g).to(torch.bfloat16).cuda()
    ws = torch.zeros(oqm.stom_oqm_attend_workspace_bytes(gcfg, L, k, sys_len) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    act = P.active_strides(sh, S)

    def run(l0, n):
        out = torch.zeros(n, Hq, d, dtype=torch.bfloat16, device="cuda")
        oqm.stom_oqm_attend(gcfg, gst, l0, n, idx[l0:], k, sh.T, q[l0:], (Hq * d, d), ks[l0:], vs[l0:], oqm.BF16, act, sys_len,
                            d ** -0.5, out, (Hq * d, d), ws)
        torch.cuda.synchronize()
        return out

    whole = run(0, L)
    assert float(whole.float().abs().max()) > 0.05
    for l in range(L):
        assert torch.equal(run(l, 1)[0], whole[l])
    assert torch.equal(run(1, 3), whole[1:4])
    ws.fill_(0xAB)           # the workspace argument is not read: its contents do not matter
    assert torch.equal(run(0, L), whole)


def test_system_tokens_with_a_padded_token_stride_and_many_units_per_warp(orc):
    """System tokens whose rows are not adjacent in memory (token stride above d: one copy per row), more units than
    one pass of the warps of a cluster takes (several units per warp, both ring stages in use), and k far above
    what one batch of prefetched indices holds."""
    from paper_2510_18269_b200 import oqm
    sh = synth.Shape("attend-many", L=1, H_q=8, H_k=1, d=128, G=16, T=3000, T_q=1, k=2300, seed=3)
    ocfg, gcfg, ost, gst, _ = P.random_bank(orc, oqm, sh, 0, seed=41)
    L, Hq, d, k, sys_len, T = sh.L, sh.H_q, sh.d, sh.k, 75, sh.T
    rng = np.random.default_rng(6)
    idx = _selection(rng, L, T, k, k - 5)
    g = torch.Generator().manual_seed(12)
    q = torch.randn(L, Hq, d, generator=g).to(torch.bfloat16)
    S = sys_len + k * sh.G
    pitch = d + 64                                             # padded rows of the system-token cache
    k_sys = torch.randn(L, 1, sys_len, pitch, generator=g).to(torch.bfloat16)
    v_sys = torch.randn(L, 1, sys_len, pitch, generator=g).to(torch.bfloat16)
    k_act = torch.zeros(L, 1, S, d, dtype=torch.bfloat16)
    v_act = torch.zeros(L, 1, S, d, dtype=torch.bfloat16)
    k_act[:, :, :sys_len] = k_sys[..., :d]
    v_act[:, :, :sys_len] = v_sys[..., :d]
    oka, ova = P.as_np16(k_act).copy(), P.as_np16(v_act).copy()
    assert orc.dequant_gather(ocfg, ost, 0, L, idx, k, T, oka, ova, orc.BF16, P.active_strides(sh, S), sys_len) == 0
    scale = 1.0 / np.sqrt(d)
    n_tok = sys_len + (k - 5) * sh.G
    want = np.stack([orc.to_f32(orc.attend(Hq, 1, d, P.as_np16(q)[l], orc.BF16, oka[l], ova[l], orc.BF16, S * d, d, n_tok,
                                           scale, out_dtype=orc.BF16), orc.BF16) for l in range(L)])
    out = torch.zeros(L, Hq, d, dtype=torch.bfloat16, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.zeros(512, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    oqm.stom_oqm_attend(gcfg, gst, 0, L, torch.from_numpy(idx).cuda(), k, T, q.cuda(), (Hq * d, d), k_sys.cuda(), v_sys.cuda(),
                        oqm.BF16, (sys_len * pitch, sys_len * pitch, pitch), sys_len, float(scale), out, (Hq * d, d), ws,
                        dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    got = orc.to_f32(P.as_np16(out), orc.BF16)
    err = np.abs(got - want)
    assert np.all(err <= np.maximum(TOL, 2.0 ** -7 * np.abs(want))), f"attention output differs by {err.max()}"
