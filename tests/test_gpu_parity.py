"""GPU parity: the C-ABI CUDA library against the CPU oracle, element by element,
on the same seeded inputs.  Tolerances are those listed in tests/_parity.py."""
import dataclasses

import numpy as np
import pytest
import torch

import _parity as P
from paper_2510_18269_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def oqm():
    from paper_2510_18269_b200 import oqm as m
    m.lib()  # fails loudly if the CUDA library is missing
    assert torch.cuda.is_available()
    return m


def _quantize_both(orc, oqm, sh, K, V, mode=0, token_idx=None, K_summary=None, strides=None, frames_per_call=None):
    """Returns (gpu store, oracle store, float32 keys the representative key comes from)."""
    tokens = K.shape[3] if strides is None else None
    strides = strides or P.contiguous_strides(sh, tokens)
    ocfg, gcfg = P.oracle_cfg(orc, sh, mode), P.gpu_cfg(oqm, sh, mode)
    ost, gst = orc.Store(ocfg), oqm.Store(gcfg)
    kn, vn = P.as_np16(K), P.as_np16(V)
    ksn = None if K_summary is None else P.as_np16(K_summary)
    tin = None if token_idx is None else token_idx.numpy()
    n_in = sh.N_in if token_idx is not None else 0
    assert orc.quantize_frame(ocfg, ost, 0, sh.L, 0, sh.T, kn, vn, strides, K_summary=ksn, token_idx=tin,
                              tokens_per_frame_in=n_in) == 0
    Kd, Vd = K.cuda(), V.cuda()
    Ksd = None if K_summary is None else K_summary.cuda()
    tid = None if token_idx is None else token_idx.cuda()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    step = frames_per_call or sh.T
    for f0 in range(0, sh.T, step):
        n = min(step, sh.T - f0)
        off = f0 * strides[1]
        oqm.stom_oqm_quantize_frame(
            gcfg, gst, 0, sh.L, f0, n, Kd.view(-1)[off:], Vd.view(-1)[off:], strides,
            K_summary=None if Ksd is None else Ksd.view(-1)[off:],
            token_idx=None if tid is None else tid[f0:], tokens_per_frame_in=n_in, dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    return gst, ost, gcfg, ocfg


def _keys_f32(orc, sh, Ksrc, token_idx=None, layout="LTHGd"):
    a = P.f32_of(orc, P.as_np16(Ksrc), sh.dtype)
    if layout == "LTNHd":                       # token-major input -> [L][T][H][N][d]
        a = a.transpose(0, 1, 3, 2, 4)
    if token_idx is not None:
        ti = token_idx.numpy()
        a = np.stack([a[:, f][:, :, ti[f]] for f in range(a.shape[1])], axis=1)
    return a


def _retrieve_both(orc, oqm, sh, gst, ost, gcfg, ocfg, Q, n_groups, mode=0, sys_len=3, out="bf16"):
    """Score, select and gather on both sides; compare every stage."""
    rows = sh.L * (sh.H_k if mode else 1)
    qn = P.as_np16(Q)
    o_scores = orc.score_groups(ocfg, ost, 0, sh.L, n_groups, qn, sh.T_q, P.q_strides(sh))
    o_idx, o_sel, o_nsel = orc.topk(o_scores.reshape(rows, n_groups), sh.k)

    Qd = Q.cuda()
    ws = torch.empty(oqm.stom_oqm_score_workspace_bytes(gcfg, sh.L), dtype=torch.uint8, device="cuda")
    g_scores = torch.full((rows * n_groups + P.GUARD,), -7.0, dtype=torch.float32, device="cuda")
    oqm.stom_oqm_score_groups(gcfg, gst, 0, sh.L, n_groups, Qd, sh.T_q, P.q_strides(sh), g_scores, ws)
    g_idx = torch.full((rows * sh.k + P.GUARD,), -9, dtype=torch.int32, device="cuda")
    g_sel = torch.full((rows * sh.k + P.GUARD,), -7.0, dtype=torch.float32, device="cuda")
    g_nsel = torch.full((rows + P.GUARD,), -9, dtype=torch.int32, device="cuda")
    oqm.stom_oqm_topk(g_scores, rows, n_groups, n_groups, sh.k, g_idx, g_sel, g_nsel)
    torch.cuda.synchronize()
    assert torch.all(g_scores[rows * n_groups:] == -7.0) and torch.all(g_idx[rows * sh.k:] == -9)
    assert torch.all(g_sel[rows * sh.k:] == -7.0) and torch.all(g_nsel[rows:] == -9)
    P.compare_scores(g_scores[:rows * n_groups], o_scores)
    P.compare_topk(g_idx[:rows * sh.k], o_idx, o_scores.reshape(rows, n_groups), sh.k)
    assert np.array_equal(g_nsel[:rows].cpu().numpy(), o_nsel)
    # selected scores follow the GPU's own selection
    gi = g_idx[:rows * sh.k].view(rows, sh.k).cpu().numpy()
    gs = g_sel[:rows * sh.k].view(rows, sh.k).cpu().numpy()
    gsc = g_scores[:rows * n_groups].view(rows, n_groups).cpu().numpy()
    for r in range(rows):
        ks = int(o_nsel[r])
        assert np.array_equal(gs[r, :ks], gsc[r, gi[r, :ks]]) and np.all(gs[r, ks:] == 0.0)

    # gather with the ORACLE's indices on both sides, so that the same groups are compared
    S = sys_len + sh.k * sh.G + 2
    tdt = torch.bfloat16 if out == "bf16" else torch.float16
    ka_flat, ka = P.out_buffers(sh, sh.L, S, tdt, "cuda", 3.0)
    va_flat, va = P.out_buffers(sh, sh.L, S, tdt, "cuda", 3.0)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    idx_d = torch.from_numpy(o_idx).cuda().contiguous()
    oqm.stom_oqm_dequant_gather(gcfg, gst, 0, sh.L, idx_d, sh.k, n_groups, ka, va, P.dt_code(out),
                                P.active_strides(sh, S), sys_len, dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    sent = P.as_np16(torch.tensor([3.0], dtype=tdt))[0]
    oka = np.full((sh.L, sh.H_k, S, sh.d), sent, np.uint16)
    ova = np.full((sh.L, sh.H_k, S, sh.d), sent, np.uint16)
    assert orc.dequant_gather(ocfg, ost, 0, sh.L, o_idx, sh.k, n_groups, oka, ova, P.dt_code(out),
                              P.active_strides(sh, S), sys_len) == 0
    n_el = sh.L * sh.H_k * S * sh.d
    for flat, o16, s_arr in ((ka_flat, oka, ost.scale_k), (va_flat, ova, ost.scale_v)):
        assert torch.all(flat[n_el:] == 3.0), "guard band overwritten"
        g16 = P.as_np16(flat[:n_el]).reshape(o16.shape)
        gf, of = orc.to_f32(g16, P.dt_code(out)), orc.to_f32(o16, P.dt_code(out))
        smax = float(s_arr.max())
        assert np.all(np.abs(gf - of) <= 1e-3 * np.maximum(np.abs(of), smax)), "dequantized values out of tolerance"
        assert int((gf != of).sum()) == 0, "dequantized values expected bit-identical"
    return o_idx, o_scores


def _full_path(orc, oqm, sh, mode=0, out="bf16", frames_per_call=None, n_groups=None):
    K, V = synth.kv_stream(sh)
    Q = synth.queries(sh)
    gst, ost, gcfg, ocfg = _quantize_both(orc, oqm, sh, K, V, mode, frames_per_call=frames_per_call)
    P.compare_store(gst, ost, _keys_f32(orc, sh, K))
    if P.meta_of(sh) != "fp32":
        # a 16-bit k-bar may sit one step from the oracle's in a few entries (binary32 against binary64 mean at a
        # rounding boundary); scoring is compared on the oracle's bank, uploaded, so that its 1e-5 bound stays meaningful
        gst.rep_key.copy_(torch.from_numpy(ost.rep_key).to(gst.rep_key.dtype))
        gst.rep_norm2.copy_(torch.from_numpy(ost.rep_norm2))
    return _retrieve_both(orc, oqm, sh, gst, ost, gcfg, ocfg, Q, n_groups or sh.T, mode, out=out)


# ------------------------------------------------------------------ the benchmark definition's small workloads

def test_c1_tiny_workload(orc, oqm):
    o_idx, _ = _full_path(orc, oqm, synth.C1)
    assert np.array_equal(o_idx[0], synth.planted_groups(synth.C1)[0].numpy())


def test_c2_7b_single_layer(orc, oqm):
    sh = synth.C2
    o_idx, _ = _full_path(orc, oqm, sh, frames_per_call=32)
    planted = set(synth.planted_groups(sh)[0].tolist())
    assert planted <= set(o_idx[0].tolist())                      # strong matches are always retrieved


def test_c2_per_head_mode(orc, oqm):
    sh = dataclasses.replace(synth.C2, T=200, k=16)
    _full_path(orc, oqm, sh, mode=1)


# ------------------------------------------------------------------ shape sweep (several tiles, ragged tails)

@pytest.mark.parametrize("G", [1, 16, 49, 50, 51, 64])
@pytest.mark.parametrize("d,H_k,H_q", [(128, 4, 28), (64, 1, 2), (256, 8, 8)])
def test_shape_sweep_bf16(orc, oqm, G, d, H_k, H_q):
    sh = synth.Shape("sweep", L=2, H_q=H_q, H_k=H_k, d=d, G=G, T=37, T_q=3, k=5, seed=100 + G + d)
    _full_path(orc, oqm, sh)


@pytest.mark.parametrize("G,d,H_k,H_q,dtype", [
    (50, 128, 4, 28, "bf16"), (16, 64, 1, 2, "bf16"), (49, 64, 2, 4, "fp16"), (7, 256, 8, 8, "bf16"),
    (64, 128, 2, 6, "fp32"), (1, 64, 1, 1, "bf16"), (51, 256, 1, 3, "fp16")])
def test_two_bit_codes(orc, oqm, G, d, H_k, H_q, dtype):
    """The 2-bit variant of the paper's ablation: three levels above the offset, four codes per byte."""
    sh = synth.Shape("two-bit", L=2, H_q=H_q, H_k=H_k, d=d, G=G, T=29, T_q=2, k=6, dtype=dtype, seed=300 + G + d,
                     extra={"bits": 2})
    _full_path(orc, oqm, sh)


@pytest.mark.parametrize("G,d,H_k,H_q,dtype,meta,bits", [
    (50, 128, 4, 28, "bf16", "bf16", 4), (50, 128, 4, 28, "bf16", "fp16", 4), (50, 128, 4, 28, "fp16", "fp16", 4),
    (49, 64, 2, 4, "fp16", "bf16", 4), (16, 64, 1, 2, "bf16", "fp16", 4), (7, 256, 8, 8, "bf16", "bf16", 4),
    (64, 128, 2, 6, "fp32", "fp16", 4), (33, 256, 4, 4, "fp32", "bf16", 4), (1, 64, 1, 1, "bf16", "bf16", 4),
    (50, 128, 4, 28, "bf16", "bf16", 2), (51, 256, 1, 3, "fp16", "fp16", 2), (50, 128, 8, 32, "bf16", "fp16", 4)])
def test_sixteen_bit_metadata(orc, oqm, G, d, H_k, H_q, dtype, meta, bits):
    """s, m and k-bar stored in fp16 or bf16: offset rounded down, scale rounded up from the stored offset, codes
    against the stored pair -- codes, s and m stay bit-exact against the oracle's reading."""
    sh = synth.Shape("meta16", L=2, H_q=H_q, H_k=H_k, d=d, G=G, T=31, T_q=2, k=6, dtype=dtype, seed=500 + G + d,
                     extra={"bits": bits, "meta": meta})
    _full_path(orc, oqm, sh, out="fp16" if dtype == "fp16" else "bf16")
    _full_path(orc, oqm, sh, mode=1, out="bf16")


@pytest.mark.parametrize("dtype,G", [("fp32", 16), ("fp32", 50), ("fp16", 50), ("fp16", 7)])
def test_input_dtypes(orc, oqm, dtype, G):
    sh = synth.Shape("dtype", L=2, H_q=8, H_k=4, d=128, G=G, T=21, T_q=2, k=4, dtype=dtype, seed=7)
    _full_path(orc, oqm, sh, out="fp16" if dtype == "fp16" else "bf16")


@pytest.mark.parametrize("n,k", [(1, 4), (3, 4), (4, 4), (5, 4), (63, 64), (64, 64), (65, 64), (300, 300)])
def test_k_and_stored_groups_edges(orc, oqm, n, k):
    sh = synth.Shape("edge", L=3, H_q=4, H_k=2, d=128, G=8, T=n, T_q=2, k=k, seed=n * 1000 + k)
    _full_path(orc, oqm, sh)


def test_partial_bank_and_layer_ranges(orc, oqm):
    """Only the first n groups are scored; layer sub-ranges address the right slices."""
    sh = synth.Shape("partial", L=4, H_q=4, H_k=2, d=128, G=10, T=40, T_q=2, k=6, seed=5)
    K, V = synth.kv_stream(sh)
    Q = synth.queries(sh)
    gst, ost, gcfg, ocfg = _quantize_both(orc, oqm, sh, K, V)
    _retrieve_both(orc, oqm, sh, gst, ost, gcfg, ocfg, Q, n_groups=17)
    # layers [1,3) only
    ws = torch.empty(oqm.stom_oqm_score_workspace_bytes(gcfg, 2), dtype=torch.uint8, device="cuda")
    sc = torch.zeros(2 * sh.T, dtype=torch.float32, device="cuda")
    Qd = Q.cuda()
    oqm.stom_oqm_score_groups(gcfg, gst, 1, 2, sh.T, Qd[1:], sh.T_q, P.q_strides(sh), sc, ws)
    o_sc = orc.score_groups(ocfg, ost, 1, 2, sh.T, P.as_np16(Q[1:].contiguous()), sh.T_q, P.q_strides(sh))
    P.compare_scores(sc, o_sc)
    # quantize layers [2,4) of frames [5,9) into a fresh bank: other slots stay zero
    g2 = oqm.Store(gcfg)
    st = P.contiguous_strides(sh, sh.G)
    Kd, Vd = K.cuda(), V.cuda()
    oqm.stom_oqm_quantize_frame(gcfg, g2, 2, 2, 5, 4, Kd[2:, 5:], Vd[2:, 5:], st)
    torch.cuda.synchronize()
    assert torch.equal(g2.codes_k[2:, 5:9], gst.codes_k[2:, 5:9]) and torch.equal(g2.scale_v[2:, 5:9], gst.scale_v[2:, 5:9])
    assert int(g2.codes_k[:2].sum()) == 0 and int(g2.codes_k[2:, :5].sum()) == 0 and int(g2.codes_k[2:, 9:].sum()) == 0
    assert float(g2.rep_key[:2].abs().sum()) == 0.0 and float(g2.rep_key[2:, 9:].abs().sum()) == 0.0


# ------------------------------------------------------------------ quantizer corner cases

def test_exact_ties_constant_and_tiny_channels(orc, oqm):
    """Data built so that (x-m)/s hits .5 exactly on many elements, plus constant, denormal-range and huge-range
    channels (the slow path of the kernel)."""
    sh = synth.Shape("ties", L=1, H_q=2, H_k=2, d=128, G=31, T=6, T_q=1, k=2, dtype="fp32", seed=3)
    g = torch.Generator().manual_seed(3)
    K = torch.randint(0, 31, (1, sh.T, sh.H_k, sh.G, sh.d), generator=g).float()
    K[:, :, :, 0, :] = 0.0
    K[:, :, :, 1, :] = 30.0                                  # range 30 -> s = 2: odd values are exact ties
    V = torch.randint(0, 16, (1, sh.T, sh.H_k, sh.G, sh.d), generator=g).float() * 0.5
    V[:, :, :, 0, :] = 0.0
    V[:, :, :, 1, :] = 7.5                                   # s = 0.5: every x.25 / x.75... and halves are ties
    V[:, 1, :, :, 5] = 1.25                                  # constant channel
    V[:, 2, :, :, 6] = torch.tensor([0.0, 1e-45] * 15 + [0.0])   # range underflows: s == 0
    V[:, 3, :, :, 7] *= 1e-30                                # scale below the fast-path window
    V[:, 4, :, :, 8] *= 1e30                                 # scale above the fast-path window
    V[:, 5, :, :, 9] = torch.linspace(-1e38, 1e38, sh.G)     # huge but finite range (values only: the key mean
                                                             # is accumulated in binary32 and would overflow)
    gst, ost, gcfg, ocfg = _quantize_both(orc, oqm, sh, K, V)
    P.compare_store(gst, ost, K.numpy())
    ties = (K[0, 0, 0, :, 0] % 2 == 1).sum()
    assert ties > 0


def test_bf16_structured_data_has_no_code_mismatch(orc, oqm):
    """bf16 inputs on a coarse grid make near-ties frequent; codes must still be bit-exact."""
    sh = synth.Shape("grid", L=2, H_q=4, H_k=4, d=128, G=50, T=64, T_q=1, k=2, seed=11)
    g = torch.Generator().manual_seed(11)
    K = (torch.randint(-64, 64, (sh.L, sh.T, sh.H_k, sh.G, sh.d), generator=g).float() / 16).to(torch.bfloat16)
    V = (torch.randint(-8, 8, (sh.L, sh.T, sh.H_k, sh.G, sh.d), generator=g).float() / 4).to(torch.bfloat16)
    gst, ost, _, _ = _quantize_both(orc, oqm, sh, K, V)
    P.compare_store(gst, ost, K.float().numpy())


@pytest.mark.parametrize("bits", [4, 2])
def test_quotients_one_float_away_from_a_rounding_boundary(orc, oqm, bits):
    """binary32 inputs placed 0, 1, 2 and 3 floats to either side of m + (k + 1/2) s for every level k and many
    random (m, s): the codes flip exactly where the true division says, so a quotient that is only nearly correctly
    rounded (one correction too few, a reciprocal that is off by an ulp) shows up here as a mismatch."""
    levels = (1 << bits) - 1
    sh = synth.Shape("boundary", L=1, H_q=2, H_k=2, d=128, G=64, T=40, T_q=1, k=2, dtype="fp32", seed=5,
                     extra={"bits": bits})
    rng = np.random.default_rng(17 + bits)
    shape = (1, sh.T, sh.H_k, sh.d)
    lo = rng.uniform(-4, 4, shape).astype(np.float32)
    span = (rng.uniform(0.05, 8.0, shape) * 2.0 ** rng.integers(-6, 7, shape)).astype(np.float32)
    hi = (lo + span).astype(np.float32)
    s = ((hi - lo).astype(np.float32) / np.float32(levels)).astype(np.float32)      # what both sides will compute
    X = np.empty((1, sh.T, sh.H_k, sh.G, sh.d), np.float32)
    X[:, :, :, 0] = lo
    X[:, :, :, 1] = hi
    for g in range(2, sh.G):
        k = (g - 2) % levels
        off = ((g - 2) // levels) % 7 - 3                                              # -3 .. 3 floats
        mid = (lo.astype(np.float64) + (k + 0.5) * s.astype(np.float64)).astype(np.float32)
        x = mid.copy()
        for _ in range(abs(off)):
            x = np.nextafter(x, np.float32(np.inf if off > 0 else -np.inf), dtype=np.float32)
        X[:, :, :, g] = np.clip(x, lo, hi)                                             # the range stays (lo, hi)
    K = torch.from_numpy(X)
    V = torch.from_numpy(X[:, ::-1].copy())
    gst, ost, gcfg, ocfg = _quantize_both(orc, oqm, sh, K, V)
    P.compare_store(gst, ost, X)
    # the construction does what it says: a good share of the elements sits within 2^-20 of a boundary
    q = (X - lo[:, :, :, None]) / s[:, :, :, None]
    near = np.abs(q - np.floor(q) - 0.5) < 2.0 ** -20
    assert near.mean() > 0.3


# ------------------------------------------------------------------ keep-mask, summary keys, strided inputs

def test_keep_mask_summary_keys_and_token_major_layout(orc, oqm):
    sh = synth.Shape("mask", L=2, H_q=28, H_k=4, d=128, G=50, T=9, T_q=4, k=3, N_in=196, seed=21)
    K, V = synth.kv_stream(sh)                                 # [L][T][H][196][d]
    Ks = (K.float() * 0.5 + 1.0).to(torch.bfloat16)            # stands in for the pre-rotary keys
    tok = synth.keep_mask(sh, 0, sh.T)
    # token-major copies: [L][T][N][H][d]
    Kt, Vt, Kst = (x.permute(0, 1, 3, 2, 4).contiguous() for x in (K, V, Ks))
    N, H, d = sh.N_in, sh.H_k, sh.d
    strides = (sh.T * N * H * d, N * H * d, d, H * d)
    gst, ost, gcfg, ocfg = _quantize_both(orc, oqm, sh, Kt, Vt, token_idx=tok, K_summary=Kst, strides=strides)
    P.compare_store(gst, ost, _keys_f32(orc, sh, Kst, tok, layout="LTNHd"))
    _retrieve_both(orc, oqm, sh, gst, ost, gcfg, ocfg, synth.queries(sh), sh.T)


def test_bad_indices_are_flagged_not_followed(orc, oqm):
    sh = synth.Shape("bad", L=1, H_q=2, H_k=2, d=128, G=4, T=5, T_q=1, k=3, N_in=6, seed=2)
    K, V = synth.kv_stream(sh)
    gcfg = P.gpu_cfg(oqm, sh)
    gst = oqm.Store(gcfg)
    tok = synth.keep_mask(sh, 0, sh.T).cuda()
    tok[2, 1] = 99                                             # outside [0, 6): clamped, flagged
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    oqm.stom_oqm_quantize_frame(gcfg, gst, 0, 1, 0, sh.T, K.cuda(), V.cuda(), P.contiguous_strides(sh, sh.N_in),
                                token_idx=tok, tokens_per_frame_in=sh.N_in, dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) & oqm.FLAG_BAD_INDEX
    S = sh.k * sh.G
    ka_flat, ka = P.out_buffers(sh, 1, S, torch.bfloat16, "cuda", 3.0)
    va_flat, va = P.out_buffers(sh, 1, S, torch.bfloat16, "cuda", 3.0)
    flags.zero_()
    idx = torch.tensor([[0, 7, -1]], dtype=torch.int32, device="cuda")      # 7 >= n_groups: skipped + flagged
    oqm.stom_oqm_dequant_gather(gcfg, gst, 0, 1, idx, sh.k, sh.T, ka, va, oqm.BF16, P.active_strides(sh, S), 0,
                                dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) & oqm.FLAG_BAD_INDEX
    assert torch.all(ka[:, :, sh.G:] == 3.0) and torch.all(va[:, :, sh.G:] == 3.0)   # slots 1, 2 untouched
    assert not torch.any(ka[:, :, :sh.G] == 3.0)


# ------------------------------------------------------------------ top-K alone, long rows

@pytest.mark.parametrize("n,k", [(7200, 64), (7200, 251), (49152, 64), (60000, 64), (5000, 5000)])
def test_topk_long_rows(orc, oqm, n, k):
    rng = np.random.default_rng(n + k)
    sc = rng.standard_normal((4, n)).astype(np.float32)
    sc[1] = np.round(sc[1] * 4) / 4                             # heavy exact ties
    sc[2] = 0.25                                                # all equal: lowest indices win
    sc[3, ::3] = -0.0
    sc[3, 1::3] = 0.0                                           # signed zeros are one value
    o_idx, o_sel, o_nsel = orc.topk(sc, k)
    g_idx = torch.empty(4 * k, dtype=torch.int32, device="cuda")
    g_sel = torch.empty(4 * k, dtype=torch.float32, device="cuda")
    oqm.stom_oqm_topk(torch.from_numpy(sc).cuda(), 4, n, n, k, g_idx, g_sel, None)
    torch.cuda.synchronize()
    assert np.array_equal(g_idx.cpu().numpy().reshape(4, k), o_idx)       # exact, ties included
    assert np.array_equal(g_sel.cpu().numpy().reshape(4, k), o_sel)


def test_retrieve_convenience_call_matches_the_three_calls(orc, oqm):
    sh = synth.Shape("retr", L=3, H_q=8, H_k=4, d=128, G=50, T=90, T_q=4, k=8, seed=31)
    K, V = synth.kv_stream(sh)
    Q = synth.queries(sh).cuda()
    gst, ost, gcfg, ocfg = _quantize_both(orc, oqm, sh, K, V)
    S = 2 + sh.k * sh.G
    outs = []
    for fused in (False, True):
        _, ka = P.out_buffers(sh, sh.L, S, torch.bfloat16, "cuda", 3.0)
        _, va = P.out_buffers(sh, sh.L, S, torch.bfloat16, "cuda", 3.0)
        sc = torch.zeros(sh.L * sh.T, dtype=torch.float32, device="cuda")
        idx = torch.zeros(sh.L * sh.k, dtype=torch.int32, device="cuda")
        ws = torch.empty(oqm.stom_oqm_score_workspace_bytes(gcfg, sh.L), dtype=torch.uint8, device="cuda")
        if fused:
            oqm.stom_oqm_retrieve(gcfg, gst, 0, sh.L, sh.T, Q, sh.T_q, P.q_strides(sh), sh.k, sc, idx, ka, va,
                                  oqm.BF16, P.active_strides(sh, S), 2, ws)
        else:
            oqm.stom_oqm_score_groups(gcfg, gst, 0, sh.L, sh.T, Q, sh.T_q, P.q_strides(sh), sc, ws)
            oqm.stom_oqm_topk(sc, sh.L, sh.T, sh.T, sh.k, idx)
            oqm.stom_oqm_dequant_gather(gcfg, gst, 0, sh.L, idx, sh.k, sh.T, ka, va, oqm.BF16,
                                        P.active_strides(sh, S), 2)
        torch.cuda.synchronize()
        outs.append((sc.clone(), idx.clone(), ka.clone(), va.clone()))
    # the fused kernel adds the question tokens up in another order: scores agree to the score tolerance (each
    # side is within 1e-5 of the oracle), the selection up to ties, and the reconstruction exactly for equal indices
    (sc_a, idx_a, ka_a, va_a), (sc_b, idx_b, ka_b, va_b) = outs
    assert (sc_a - sc_b).abs().max().item() <= 2e-5
    P.compare_topk(idx_b, idx_a.view(sh.L, sh.k).cpu().numpy(), sc_a.view(sh.L, sh.T).cpu().numpy(), sh.k)
    if torch.equal(idx_a, idx_b):
        assert torch.equal(ka_a, ka_b) and torch.equal(va_a, va_b)


@pytest.mark.parametrize("G,d,H_k,T,dtype", [(8, 64, 2, 3000, "bf16"), (25, 128, 4, 900, "bf16"), (3, 128, 1, 5000, "fp16")])
def test_many_small_tiles_wrap_the_ring_many_times(orc, oqm, G, d, H_k, T, dtype):
    """Small groups make the consumers fast and the producer the slow side, and every block's ring of shared-memory
    slots is refilled dozens of times: the bank must equal the oracle's for the whole stream, must not depend on how
    the stream is cut into calls (another tile -> slot mapping), and must come out the same twice."""
    sh = synth.Shape("ring", L=2, H_q=2 * H_k, H_k=H_k, d=d, G=G, T=T, T_q=1, k=4, dtype=dtype, seed=900 + G)
    K, V = synth.kv_stream(sh)
    gst, ost, gcfg, ocfg = _quantize_both(orc, oqm, sh, K, V)
    P.compare_store(gst, ost, _keys_f32(orc, sh, K))
    again, _, _, _ = _quantize_both(orc, oqm, sh, K, V, frames_per_call=997)
    for name in ("codes_k", "codes_v", "scale_k", "zero_k", "scale_v", "zero_v", "rep_key", "rep_norm2"):
        assert torch.equal(getattr(gst, name), getattr(again, name)), f"{name} depends on how the stream was cut"
    twice = oqm.Store(gcfg)
    Kd, Vd = K.cuda(), V.cuda()
    oqm.stom_oqm_quantize_frame(gcfg, twice, 0, sh.L, 0, sh.T, Kd, Vd, P.contiguous_strides(sh, sh.G))
    torch.cuda.synchronize()
    assert torch.equal(twice.codes_k, gst.codes_k) and torch.equal(twice.codes_v, gst.codes_v)
