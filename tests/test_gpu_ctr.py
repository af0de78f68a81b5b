"""GPU parity of the CTR steps the library implements (temporal similarity, static / dynamic split, budget,
saliency selection of the dynamic tokens, Merge of the static tokens and the retained group; paper Sec. 3.3) against
the CPU oracle.

Tolerances: similarity 1e-5 absolute (binary32 accumulation over D channels against binary64); every integer output
of stom_ctr_select bit-exact when both sides are given the same similarities (the oracle's, uploaded).  For the
chained call the library's own similarities decide the split, so a frame is compared exactly unless one of its
tokens has an oracle similarity within 1e-5 of tau_c, where either side of the threshold is a correct answer.
Merge: the library takes its decisions (which tokens are centres, which centre a token joins) from binary32 distances,
the oracle from binary64 ones.  Every frame is checked for a VALID result (k_s centres among the static tokens, a
partition, dynamic rows copied bit for bit, positions ascending); the decisions themselves are compared wherever the
oracle's own margin (relative gap to the alternative) exceeds 1e-4, and the merged rows of clusters with the same
members on both sides must be within one step of the feature type, all but 0.2 % of the values identical."""
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


# ------------------------------------------------------------------ Merge_{k_s} and the retained group

MARGIN = 1e-4   # relative gap below which a centre choice or a nearest-centre assignment may fall either way in binary32


def _oracle_frame(orc, Fn, dt, sidx_t, didx_t, ks_t, kd_t, G, knn):
    S = sidx_t[sidx_t >= 0]
    r = orc.ctr_merge(Fn, dt, S, int(ks_t), knn)
    ret, pos = orc.ctr_retain(Fn, dt, didx_t[:kd_t], r["centre"], r["merged"], G)
    return r, ret, pos


def _check_merge(orc, oqm, F, alpha, G, knn, dtype, o_sim=None, min_clear=0.3):
    T, N, D = F.shape
    dt = P.dt_code(dtype)
    Fn = P.as_np16(F)
    if o_sim is None:
        o_sim = orc.ctr_similarity(Fn, dt)
    ks, kd, sidx, didx = orc.ctr_select(o_sim, alpha, G, TAU)
    tdt = synth.DTYPES[dtype]
    ret_flat = torch.full((T * G * D + P.GUARD,), 3.0, dtype=tdt, device="cuda")
    pos = torch.full((T * G + P.GUARD,), -9, dtype=torch.int32, device="cuda")
    cen = torch.full((T * G + P.GUARD,), -9, dtype=torch.int32, device="cuda")
    asg = torch.full((T * N + P.GUARD,), -9, dtype=torch.int32, device="cuda")
    up = lambda a: torch.from_numpy(a).cuda()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    oqm.stom_ctr_merge(F.cuda(), T, N, D, (N * D, D), up(ks), up(kd), up(sidx), up(didx), G, knn, ret_flat, pos, cen, asg,
                       dev_flags=flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    torch.cuda.synchronize()
    assert torch.all(ret_flat[T * G * D:] == 3.0) and torch.all(pos[T * G:] == -9), "guard band overwritten"
    assert torch.all(cen[T * G:] == -9) and torch.all(asg[T * N:] == -9), "guard band overwritten"
    g_ret = P.as_np16(ret_flat[:T * G * D]).reshape(T, G, D)
    g_pos, g_cen = pos[:T * G].view(T, G).cpu().numpy(), cen[:T * G].view(T, G).cpu().numpy()
    g_asg = asg[:T * N].view(T, N).cpu().numpy()
    step = 2.0 ** -7 if dtype == "bf16" else 2.0 ** -10
    clear, differing, merged_elems = 0, 0, 0
    for t in range(T):
        r, o_ret, o_pos = _oracle_frame(orc, Fn[t], dt, sidx[t], didx[t], ks[t], kd[t], G, knn)
        n_s = int((sidx[t] >= 0).sum())
        # whatever the clustering decided, the result is a valid one: k_s centres among the static tokens, ascending,
        # every static token in a cluster, the dynamic rows copied bit for bit, unused rows zero
        c = g_cen[t, :ks[t]]
        assert np.all(g_cen[t, ks[t]:] == -1) and np.all(np.diff(c) > 0) and np.all(np.isin(c, sidx[t, :n_s]))
        a = g_asg[t, :n_s]
        assert np.all(g_asg[t, n_s:] == -1)
        if ks[t] > 0:
            assert a.min() >= 0 and a.max() < ks[t] and len(np.unique(a)) == ks[t]
            assert np.array_equal(a[np.searchsorted(sidx[t, :n_s], c)], np.arange(ks[t])), "a centre left its cluster"
        want_pos = np.sort(np.concatenate([didx[t, :kd[t]], c]))
        assert np.array_equal(g_pos[t, :kd[t] + ks[t]], want_pos) and np.all(g_pos[t, kd[t] + ks[t]:] == -1)
        assert not g_ret[t, kd[t] + ks[t]:].any()
        for w, tok in enumerate(want_pos):
            if tok in didx[t, :kd[t]]:
                assert np.array_equal(g_ret[t, w], Fn[t, tok]), f"frame {t}: dynamic row {tok} was not copied unchanged"
        if r["margin_centres"] <= MARGIN:
            continue                                    # the centre choice of this frame sits on the fence: either side is right
        clear += 1
        assert np.array_equal(c, r["centre"]), f"frame {t}: centres differ"
        sure = r["margin_assign"] > MARGIN              # tokens whose nearest centre is not a close call
        assert np.array_equal(a[sure], r["assign"][sure]), f"frame {t}: assignments differ"
        assert np.array_equal(g_pos[t], o_pos)
        # merged rows of the clusters that have the same members on both sides
        for j in range(ks[t]):
            if not np.array_equal(a == j, r["assign"] == j):
                continue
            w_ = int(np.nonzero(o_pos == c[j])[0][0])
            got, want = orc.to_f32(g_ret[t, w_], dt).astype(np.float64), orc.to_f32(o_ret[w_], dt).astype(np.float64)
            assert np.all(np.abs(got - want) <= step * np.abs(want) + 1e-30), f"frame {t}: a merged value is more than one step off"
            differing += int((g_ret[t, w_] != o_ret[w_]).sum())
            merged_elems += D
    assert clear >= min_clear * T, f"only {clear} of {T} frames had a clear-cut centre choice"
    assert differing <= 2e-3 * max(merged_elems, 1), f"{differing} of {merged_elems} merged values differ from the oracle's"
    return ks, kd


def _blob_stream(T, N, D, n_blobs, seed, dtype):
    """Features with an unmistakable cluster structure: every position belongs to one of n_blobs blobs (tight around the
    blob's centre, later positions a little looser), and a moving block of positions is redrawn every frame."""
    g = torch.Generator().manual_seed(seed)
    blob = torch.randint(0, n_blobs, (N,), generator=g)
    mu = 3.0 * torch.randn(n_blobs, D, generator=g)
    F = torch.empty(T, N, D)
    alpha = torch.rand(T, N, generator=g)
    for t in range(T):
        x = mu[blob] + 0.15 * torch.randn(N, D, generator=g) * torch.linspace(0.2, 1.0, N)[:, None]
        lo = (7 * t) % max(1, N - N // 5)
        x[lo:lo + N // 5] = 2.0 * torch.randn(N // 5, D, generator=g)
        F[t] = x
    return F.to(synth.DTYPES[dtype]).contiguous(), alpha.numpy().astype(np.float32)


@pytest.mark.parametrize("T,N,D,G,knn,dtype,n_blobs", [
    (24, 196, 1152, 50, 5, "bf16", 60),     # the 7B encoder's frame
    (10, 50, 128, 20, 3, "fp16", 12),       # a token count that is no multiple of 16; two slabs of channels
    (6, 224, 256, 224, 5, "bf16", 40),      # the largest frame; G = N
    (8, 33, 64, 9, 0, "bf16", 6),           # no neighbours in the density: rho = 1, delta alone decides
    (8, 64, 192, 16, 8, "fp16", 10),        # the most neighbours
    (6, 128, 128, 32, 5, "bf16", 16),       # exactly one 128-row tile of the Gram product
    (6, 144, 320, 40, 5, "fp16", 20),       # two tiles that overlap in all but 16 rows; five slabs through a ring of three
])
def test_merge_matches_oracle_on_clustered_features(orc, T, N, D, G, knn, dtype, n_blobs):
    oqm = _lib()
    F, alpha = _blob_stream(T, N, D, n_blobs, seed=T + N, dtype=dtype)
    ks, kd = _check_merge(orc, oqm, F, alpha, G, knn, dtype, min_clear=0.5)
    assert ks[0] == 0 and ks[1:].max() >= 1          # the first frame has no static tokens; later ones do


def test_merge_matches_oracle_on_the_synthetic_encoder_stream(orc):
    """The stream the benchmark uses: static tokens here are one noisy copy each of unrelated base vectors, so the
    clustering has little to hold on to and many decisions are close; decisions on the fence are checked for validity
    only, the others exactly."""
    oqm = _lib()
    T, N, D, G = 40, 196, 1152, 50
    F, alpha = synth.ctr_stream(T, N, D, seed=21, dtype="bf16")
    _check_merge(orc, oqm, F, alpha.numpy(), G, 5, "bf16", min_clear=0.2)


def test_merge_all_static_and_all_dynamic_frames(orc):
    oqm = _lib()
    T, N, D, G = 4, 48, 128, 12
    F, alpha = _blob_stream(T, N, D, 8, seed=5, dtype="bf16")
    sim = np.full((T, N), 0.99, np.float32)          # every token static: k_s = G, k_d = 0
    sim[2] = 0.1                                     # frame 2: every token dynamic: k_s = 0, k_d = G
    ks, kd = _check_merge(orc, oqm, F, alpha, G, 5, "bf16", o_sim=sim, min_clear=0.5)
    assert ks.tolist() == [12, 12, 0, 12] and kd.tolist() == [0, 0, 12, 0]


def test_merge_rejects_what_the_kernel_does_not_cover():
    oqm = _lib()
    z = lambda *s: torch.zeros(*s, dtype=torch.int32, device="cuda")

    def call(N=32, D=128, G=8, knn=5, dtype=torch.bfloat16):
        F = torch.zeros(2, N, D, dtype=dtype, device="cuda")
        ret = torch.zeros(2, G, D, dtype=dtype, device="cuda")
        oqm.stom_ctr_merge(F, 2, N, D, (N * D, D), z(2), z(2), z(2, N), z(2, G), G, knn, ret, z(2, G))
    call()
    for kw, code in ((dict(N=240), -2), (dict(D=96), -2), (dict(knn=9), -2), (dict(G=40), -2), (dict(dtype=torch.float32), -6)):
        with pytest.raises(oqm.StomError) as e:
            call(**kw)
        assert e.value.code == code


def test_ctr_output_feeds_the_quantizer(orc):
    """CTR end to end, then A1: the retained tokens [T][G][D] come out of stom_ctr_reduce_tokens and are handed to
    stom_oqm_quantize_frame as they lie in memory (D = 9 x 128 read as 9 heads of 128 channels through the strides; in
    the method the language model sits between the two and produces K and V of these tokens -- here the tokens
    themselves stand in for both).  Frames whose retained group equals the oracle's bit for bit must give the oracle's
    bank entries."""
    oqm = _lib()
    T, N, D, G, knn = 12, 196, 1152, 50, 5
    F, alpha = _blob_stream(T, N, D, 20, seed=77, dtype="bf16")   # fewer blobs than centres: every blob gets one
    Fn = P.as_np16(F)
    sim = torch.zeros(T, N, dtype=torch.float32, device="cuda")
    g_ks, g_kd, g_s, g_d = _select_outputs(T, N, G)
    ret = torch.zeros(T, G, D, dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros(T, G, dtype=torch.int32, device="cuda")
    oqm.stom_ctr_reduce_tokens(F.cuda(), None, T, N, D, (N * D, D), torch.from_numpy(alpha).cuda(), G, TAU, knn, sim, g_ks,
                               g_kd, g_s, g_d, ret, pos)
    H = D // 128
    cfg = oqm.make_config(1, H, H, 128, G, T)
    st = oqm.Store(cfg)
    oqm.stom_oqm_quantize_frame(cfg, st, 0, 1, 0, T, ret, ret, (T * G * D, G * D, 128, D))
    torch.cuda.synchronize()
    # the oracle's own chain
    o_sim = orc.ctr_similarity(Fn, orc.BF16)
    ks, kd, sidx, didx = orc.ctr_select(o_sim, alpha, G, TAU)
    o_ret = np.zeros((T, G, D), np.uint16)
    for t in range(T):
        _, o_ret[t], _ = _oracle_frame(orc, Fn[t], orc.BF16, sidx[t], didx[t], ks[t], kd[t], G, knn)
    g_ret = P.as_np16(ret)
    same = np.array([np.array_equal(g_ret[t], o_ret[t]) for t in range(T)])
    assert same.sum() >= T // 3, "too few frames whose retained group equals the oracle's"
    ocfg = orc.make_config(1, H, H, 128, G, T)
    ost = orc.Store(ocfg)
    assert orc.quantize_frame(ocfg, ost, 0, 1, 0, T, o_ret, o_ret, (T * G * D, G * D, 128, D)) == 0
    frames = np.nonzero(same)[0]
    for name in ("codes_k", "codes_v", "scale_k", "zero_k", "scale_v", "zero_v"):
        g = getattr(st, name)[0].cpu().numpy()
        o = getattr(ost, name)[0]
        assert np.array_equal(g[frames].view(np.uint8), o[frames].view(np.uint8)), f"{name} differs from the oracle's"
