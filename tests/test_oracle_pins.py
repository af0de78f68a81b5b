"""Pins for the CPU oracle: every check here compares the oracle with something
that is NOT the oracle -- a value the paper prints, a closed form, an
invariant, a library routine, or brute force on a tiny input -- so that a
plausible mistake in it (dropped term, wrong axis, wrong sign, transposed
operand) fails at least one test.  CPU only."""
from pathlib import Path

import numpy as np
import pytest
import torch

GOLD = Path(__file__).parent / "golden" / "paper_values.txt"


def golden():
    out = {}
    for line in GOLD.read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, rest = line.split("=", 1)
        val, tol, _cite = [x.strip() for x in rest.split("|", 2)]
        out[name.strip()] = (float(val), float(tol))
    return out


# ------------------------------------------------------------------ formats

def test_bf16_to_f32_all_patterns_match_torch(orc):
    bits = np.arange(65536, dtype=np.uint16)
    ours = orc.to_f32(bits, orc.BF16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(ours.view(np.uint32), ref.view(np.uint32))


def test_f16_to_f32_all_patterns_match_numpy(orc):
    bits = np.arange(65536, dtype=np.uint16)
    ours = orc.to_f32(bits, orc.FP16)
    ref = bits.view(np.float16).astype(np.float32)
    ok = (ours.view(np.uint32) == ref.view(np.uint32)) | (np.isnan(ours) & np.isnan(ref))
    assert ok.all()


def _interesting_floats(rng, n):
    a = rng.standard_normal(n).astype(np.float32) * np.float32(10.0) ** rng.integers(-9, 6, n).astype(np.float32)
    # exact ties and their neighbours for both 16-bit formats
    base = rng.integers(0, 1 << 16, n // 4).astype(np.uint32) << 16
    ties = (base | 0x8000).view(np.float32)
    near = ((base | 0x8000) + rng.integers(-1, 2, n // 4).astype(np.uint32)).view(np.float32)
    h = rng.integers(0, 0x7c00, n // 4).astype(np.uint16).view(np.float16).astype(np.float32)
    hn = np.nextafter(h, np.float32(np.inf))
    half_ties = ((h.astype(np.float64) + hn.astype(np.float64)) / 2).astype(np.float32)
    special = np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 65536.0, 1e-8, 5.96e-8, 2.98e-8, 6.1e-5,
                        6.103515625e-05, np.inf, -np.inf, 3.0e38, -3.0e38], np.float32)
    return np.concatenate([a, ties, near, half_ties, -half_ties, special])


def test_f32_to_bf16_matches_torch(orc):
    x = _interesting_floats(np.random.default_rng(1), 200_000)
    x = x[np.isfinite(x)]
    ours = orc.from_f32(x, orc.BF16)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(ours, ref)


def test_f32_to_f16_matches_numpy(orc):
    x = _interesting_floats(np.random.default_rng(2), 200_000)
    x = x[~np.isnan(x)]                                     # NaN payloads are not part of the contract
    ours = orc.from_f32(x, orc.FP16)
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    np.testing.assert_array_equal(ours, ref)


# ------------------------------------------------------------------ O1 quantizer

def _group(rng, H=2, G=16, d=32, outliers=True):
    X = rng.standard_normal((H, G, d)).astype(np.float32)
    if outliers:
        X[:, :, :4] *= 10
    return X


@pytest.mark.parametrize("bits", [4, 2])
@pytest.mark.parametrize("G", [1, 2, 16, 50])
def test_quantizer_invariants(orc, bits, G):
    rng = np.random.default_rng(10 + G)
    X = _group(rng, H=3, G=G, d=64)
    codes, s, m = orc.quantize_group(X, bits)
    nlev = (1 << bits) - 1
    assert codes.min() >= 0 and codes.max() <= nlev
    mn, mx = X.min(axis=1), X.max(axis=1)           # statistics are over the G tokens (axis 1)
    np.testing.assert_array_equal(m, mn)             # offset is the channel minimum, exactly
    # scale: nlev * s equals the range up to binary32 rounding of the division
    rng_ = (mx.astype(np.float64) - mn.astype(np.float64))
    assert np.all(np.abs(s.astype(np.float64) * nlev - rng_) <= 2.0 ** -22 * np.abs(rng_) + 1e-45)
    # reconstruction error bound |x - (m + c*s)| <= s/2 (+ rounding slack), every element
    xhat = m[:, None, :].astype(np.float64) + codes.astype(np.float64) * s[:, None, :].astype(np.float64)
    err = np.abs(X.astype(np.float64) - xhat)
    bound = s[:, None, :].astype(np.float64) * (0.5 + 2.0 ** -18) + 2.0 ** -22 * np.abs(X)
    assert np.all(err <= bound)
    # channel minimum -> code 0, channel maximum -> top code (when the channel is not constant)
    amin, amax = X.argmin(axis=1), X.argmax(axis=1)
    h_i, c_i = np.meshgrid(np.arange(X.shape[0]), np.arange(X.shape[2]), indexing="ij")
    assert np.all(codes[h_i, amin, c_i] == 0)
    nonconst = mx > mn
    assert np.all(codes[h_i, amax, c_i][nonconst] == nlev)


def test_quantizer_codes_are_nearest_level_bruteforce(orc):
    """Each code must be an argmin over the 16 levels of |x - (m + c s)| (float64; exact ties either way)."""
    rng = np.random.default_rng(3)
    X = _group(rng, H=2, G=7, d=16)
    codes, s, m = orc.quantize_group(X, 4)
    lv = np.arange(16, dtype=np.float64)
    for h in range(2):
        for c in range(16):
            levels = float(m[h, c]) + lv * float(s[h, c])
            for g in range(7):
                dist = np.abs(float(X[h, g, c]) - levels)
                best = dist.min()
                assert dist[codes[h, g, c]] <= best + 2.0 ** -20 * max(1.0, abs(float(X[h, g, c])))


def test_quantizer_statistics_axis_and_indexing(orc):
    """A tensor whose min/max per (head, channel) is known in closed form; a wrong reduction axis fails."""
    H, G, d = 3, 5, 8
    h, g, c = np.meshgrid(np.arange(H), np.arange(G), np.arange(d), indexing="ij")
    X = (100.0 * h + c + 0.25 * g).astype(np.float32)
    codes, s, m = orc.quantize_group(X, 4)
    hh, cc = np.meshgrid(np.arange(H), np.arange(d), indexing="ij")
    np.testing.assert_array_equal(m, (100.0 * hh + cc).astype(np.float32))
    np.testing.assert_allclose(s, np.full((H, d), 1.0 / 15.0, np.float32), rtol=1e-6)
    # tokens are at 0, .25, .5, .75, 1.0 of the range -> levels 0, 3.75, 7.5, 11.25, 15
    # 7.5 is an exact tie only in exact arithmetic; in binary32 (0.5)/(1/15 rounded) decides it.
    expect = np.array([0, 4, None, 11, 15], dtype=object)
    for gi in (0, 1, 3, 4):
        assert np.all(codes[:, gi, :] == expect[gi])
    assert set(np.unique(codes[:, 2, :])) <= {7, 8}


def test_quantizer_round_half_to_even_on_exact_ties(orc):
    """Range 30 -> s = 2 exactly; odd offsets are exact .5 ties and must go to the even code."""
    G = 31
    col = np.arange(G, dtype=np.float32)          # 0..30 -> (x-m)/s = 0, .5, 1, 1.5, ...
    X = col.reshape(1, G, 1).copy()
    codes, s, m = orc.quantize_group(X, 4)
    assert s[0, 0] == 2.0 and m[0, 0] == 0.0
    t = col / 2.0
    expect = np.array([int(round(v)) for v in t])  # Python's round is half-to-even
    np.testing.assert_array_equal(codes[0, :, 0], expect)
    assert codes[0, 1, 0] == 0 and codes[0, 3, 0] == 2 and codes[0, 5, 0] == 2 and codes[0, 7, 0] == 4


def test_quantizer_constant_and_underflowing_channel(orc):
    X = np.zeros((1, 4, 3), np.float32)
    X[0, :, 0] = 3.25                                  # constant
    X[0, :, 1] = [0.0, 1e-45, 0.0, 1e-45]              # range/15 underflows to 0
    X[0, :, 2] = [-1.0, 0.0, 1.0, 2.0]
    codes, s, m = orc.quantize_group(X, 4)
    assert s[0, 0] == 0.0 and m[0, 0] == 3.25 and np.all(codes[0, :, 0] == 0)
    assert s[0, 1] == 0.0 and np.all(codes[0, :, 1] == 0)
    assert orc.dequant_value(0, float(s[0, 0]), float(m[0, 0])) == 3.25
    np.testing.assert_array_equal(codes[0, :, 2], [0, 5, 10, 15])


def test_pack_unpack_identity_and_layout(orc):
    # unpack(pack(.)) is the identity over every byte value
    for b in range(256):
        lo, hi = b & 15, b >> 4
        packed = orc.pack_row(np.array([lo, hi], np.uint8), 4)
        assert packed[0] == b                          # even channel in the low nibble (layout is a build decision)
        np.testing.assert_array_equal(orc.unpack_row(packed, 2, 4), [lo, hi])
    rng = np.random.default_rng(4)
    c4 = rng.integers(0, 16, 128).astype(np.uint8)
    np.testing.assert_array_equal(orc.unpack_row(orc.pack_row(c4, 4), 128, 4), c4)
    c2 = rng.integers(0, 4, 128).astype(np.uint8)
    p2 = orc.pack_row(c2, 2)
    assert p2.size == 32
    np.testing.assert_array_equal(orc.unpack_row(p2, 128, 2), c2)
    assert orc.pack_row(np.array([1, 2, 3, 0], np.uint8), 2)[0] == 1 | (2 << 2) | (3 << 4)


def test_dequant_is_affine_and_exact_at_code_zero(orc):
    rng = np.random.default_rng(5)
    for _ in range(200):
        s, m = np.float32(abs(rng.standard_normal())), np.float32(rng.standard_normal() * 10)
        assert orc.dequant_value(0, s, m) == m
        for code in (1, 7, 15):
            exact = float(m) + code * float(s)         # exact in binary64
            assert orc.dequant_value(code, s, m) == np.float32(exact)  # one rounding only


# ------------------------------------------------------------------ O2 representative key

def test_rep_key_is_numpy_mean_over_tokens(orc):
    rng = np.random.default_rng(6)
    K = _group(rng, H=4, G=50, d=128)
    rep, n2 = orc.rep_key(K)
    ref = K.astype(np.float64).mean(axis=1)
    np.testing.assert_allclose(rep, ref, rtol=0, atol=1e-6)
    np.testing.assert_allclose(n2, (rep.astype(np.float64) ** 2).sum(axis=1), rtol=1e-6)
    const = np.broadcast_to(np.arange(8, dtype=np.float32), (2, 5, 8)).copy()
    rep, n2 = orc.rep_key(const)
    np.testing.assert_array_equal(rep, const[:, 0, :])
    np.testing.assert_allclose(n2, [140.0, 140.0])


# ------------------------------------------------------------------ 16-bit metadata (storage reading of s, m, k-bar)

def _values16(dtype_name):
    """Every finite value of a 16-bit format, ascending, as float64 (built from bit patterns with torch, not with
    the oracle)."""
    bits = torch.arange(65536, dtype=torch.int32).to(torch.int16)
    t = bits.view(torch.float16 if dtype_name == "fp16" else torch.bfloat16).to(torch.float64)
    v = t[torch.isfinite(t)].numpy()
    return np.unique(v)  # sorted; +0 and -0 collapse


@pytest.mark.parametrize("dtype_name", ["fp16", "bf16"])
def test_directed_rounding_brackets_every_input(orc, dtype_name):
    """round_down(x) is the largest representable value <= x and round_up(x) the smallest >= x: checked against the
    sorted table of all values of the format (searchsorted), at representable points, midpoints and random points."""
    dt = orc.FP16 if dtype_name == "fp16" else orc.BF16
    table = _values16(dtype_name)
    rng = np.random.default_rng(41)
    lim = 6.0e4 if dtype_name == "fp16" else 1.0e30
    pts = np.concatenate([
        rng.choice(table[np.abs(table) < lim], 300),                                      # representable
        rng.standard_normal(300) * 3.0, rng.standard_normal(200) * 1e-3, rng.standard_normal(100) * 1e3,
        rng.standard_normal(100) * 1e-7,                                                  # fp16 subnormal range
        np.array([0.0, 1e-30, -1e-30, 1.0, -1.0, 0.1, -0.1]),
    ]).astype(np.float32)
    mids = ((table[1:] + table[:-1]) / 2.0)
    mids = mids[np.abs(mids) < lim]
    pts = np.concatenate([pts, rng.choice(mids, 300).astype(np.float32)])
    for x in pts:
        x = float(x)
        lo = table[np.searchsorted(table, x, side="right") - 1]
        hi = table[np.searchsorted(table, x, side="left")]
        assert orc.round_down(x, dt) == lo, x
        assert orc.round_up(x, dt) == hi, x
        assert orc.round_down(x, orc.FP32) == x and orc.round_up(x, orc.FP32) == x
    # nearest-even agrees with torch's conversion
    t = torch.from_numpy(pts)
    want = t.to(torch.float16 if dtype_name == "fp16" else torch.bfloat16).to(torch.float32).numpy()
    got = np.array([orc.round_nearest(float(x), dt) for x in pts], np.float32)
    np.testing.assert_array_equal(got, want)


@pytest.mark.parametrize("dtype_name", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", [4, 2])
def test_quantizer_with_16bit_metadata_keeps_codes_in_range_and_the_error_bound(orc, dtype_name, bits):
    dt = orc.FP16 if dtype_name == "fp16" else orc.BF16
    tdt = torch.float16 if dtype_name == "fp16" else torch.bfloat16
    table = _values16(dtype_name)
    rng = np.random.default_rng(43)
    X = _group(rng, H=3, G=50, d=64)
    X[1, :, 5] = 0.375           # a constant channel
    X[2, :, 7] += 100.0          # a channel whose offset is far from zero: m loses bits in 16-bit storage
    codes, s, m = orc.quantize_group(X, bits, dt)
    nlev = (1 << bits) - 1
    # stored values are representable
    for a in (s, m):
        np.testing.assert_array_equal(torch.from_numpy(a).to(tdt).to(torch.float32).numpy(), a)
    mn, mx = X.min(axis=1).astype(np.float64), X.max(axis=1).astype(np.float64)
    m64, s64 = m.astype(np.float64), s.astype(np.float64)
    # m is the largest representable value <= min
    assert np.all(m64 <= mn)
    nxt = table[np.searchsorted(table, m64.ravel(), side="right")].reshape(m.shape)
    assert np.all(nxt > mn)
    # s covers the range from the STORED offset (so the top code never overshoots) and is minimal up to one step
    assert np.all(m64 + nlev * s64 >= mx * (1 - 2.0 ** -23) - 1e-30)
    prev = table[np.maximum(np.searchsorted(table, s64.ravel(), side="left") - 1, 0)].reshape(s.shape)
    need = ((mx - m64) / nlev)
    assert np.all((prev < need * (1 + 2.0 ** -22)) | (s64 == 0))
    assert s[1, 5] == 0 and np.all(codes[1, :, 5] == 0) and m[1, 5] == np.float32(0.375)
    # codes in range, nearest level of the stored (s, m), error <= s/2
    assert codes.max() <= nlev
    xhat = m64[:, None, :] + codes.astype(np.float64) * s64[:, None, :]
    err = np.abs(X.astype(np.float64) - xhat)
    assert np.all(err <= s64[:, None, :] * (0.5 + 2.0 ** -18) + 2.0 ** -22 * np.abs(X))
    lv = np.arange(nlev + 1, dtype=np.float64)
    dist = np.abs(X.astype(np.float64)[..., None] - (m64[:, None, :, None] + lv * s64[:, None, :, None]))
    chosen = np.take_along_axis(dist, codes[..., None].astype(np.int64), axis=-1)[..., 0]
    assert np.all(chosen <= dist.min(axis=-1) + 2.0 ** -20 * np.maximum(1.0, np.abs(X)))
    # inputs that are already 16-bit values of the same type keep their minimum exactly
    X16 = torch.from_numpy(X).to(tdt).to(torch.float32).numpy()
    _, _, m16 = orc.quantize_group(X16, bits, dt)
    np.testing.assert_array_equal(m16, X16.min(axis=1))


@pytest.mark.parametrize("dtype_name", ["fp16", "bf16"])
def test_rep_key_with_16bit_metadata_is_the_rounded_mean(orc, dtype_name):
    dt = orc.FP16 if dtype_name == "fp16" else orc.BF16
    tdt = torch.float16 if dtype_name == "fp16" else torch.bfloat16
    rng = np.random.default_rng(47)
    K = _group(rng, H=4, G=50, d=128)
    rep, n2 = orc.rep_key(K, dt)
    mean = torch.from_numpy(K.astype(np.float64).mean(axis=1))
    lo = mean.to(torch.float32).to(tdt).to(torch.float64).numpy()
    # the mean passes through binary32 first; allow the neighbouring 16-bit value only where that matters
    step = np.abs(lo) * (2.0 ** -10 if dtype_name == "fp16" else 2.0 ** -7) + 1e-12
    assert np.all(np.abs(rep.astype(np.float64) - lo) <= step)
    assert np.mean(rep.astype(np.float64) == lo) > 0.999
    np.testing.assert_array_equal(torch.from_numpy(rep).to(tdt).to(torch.float32).numpy(), rep)   # representable
    np.testing.assert_allclose(n2, (rep.astype(np.float64) ** 2).sum(axis=1), rtol=1e-6)           # norm of the STORED key


def test_store_bytes_with_16bit_metadata(orc):
    """Per (group, kv head) at G = 50, d = 128: 6400 bytes of codes, 5 x 128 metadata values, one norm."""
    for dt, eb in ((orc.FP32, 4), (orc.FP16, 2), (orc.BF16, 2)):
        cfg = orc.make_config(1, 1, 1, 128, 50, 1, meta_dtype=dt)
        assert orc.store_bytes(cfg, 1, True) == 6400 + 5 * 128 * eb + 4
        assert orc.store_bytes(cfg, 1, False) == 6400
    full = 2 * 50 * 128 * 2  # the same group in 16-bit K and V
    assert abs(full / (orc.store_bytes(orc.make_config(1, 1, 1, 128, 50, 1, meta_dtype=orc.FP16), 1, True) - 4) - 10 / 3) < 1e-9


def test_quantize_frame_with_16bit_metadata_matches_the_group_functions(orc):
    """The frame-level call applies the same reading to every (layer, group, head) and to the representative key."""
    rng = np.random.default_rng(53)
    L, T, H, G, d = 2, 3, 2, 5, 32
    cfg = orc.make_config(L, 4, H, d, G, T, kv_dtype=orc.FP32, meta_dtype=orc.BF16)
    st = orc.Store(cfg)
    K = rng.standard_normal((L, T, H, G, d)).astype(np.float32)
    V = rng.standard_normal((L, T, H, G, d)).astype(np.float32)
    assert orc.quantize_frame(cfg, st, 0, L, 0, T, K, V, (T * H * G * d, H * G * d, G * d, d)) == 0
    for l in range(L):
        for t in range(T):
            _, s, m = orc.quantize_group(V[l, t], 4, orc.BF16)
            np.testing.assert_array_equal(st.scale_v[l, t], s)
            np.testing.assert_array_equal(st.zero_v[l, t], m)
            rep, n2 = orc.rep_key(K[l, t], orc.BF16)
            np.testing.assert_array_equal(st.rep_key[l, t], rep)
            np.testing.assert_array_equal(st.rep_norm2[l, t], n2)
    f32 = orc.Store(orc.make_config(L, 4, H, d, G, T, kv_dtype=orc.FP32))
    orc.quantize_frame(f32.cfg, f32, 0, L, 0, T, K, V, (T * H * G * d, H * G * d, G * d, d))
    assert np.all(st.zero_v <= f32.zero_v) and np.all(st.scale_v >= f32.scale_v)


# ------------------------------------------------------------------ O3 / O4 query embedding, scores

def test_query_embedding_gqa_blocks_and_token_mean(orc):
    cfg = orc.make_config(1, 6, 2, 4, 5, 8, kv_dtype=orc.FP32)
    Hq, Tq, d = 6, 3, 4
    hq, j, c = np.meshgrid(np.arange(Hq), np.arange(Tq), np.arange(d), indexing="ij")
    Q = (10.0 * hq + j + 0.125 * c).astype(np.float32)
    q = orc.query_embedding(cfg, Q, orc.FP32)
    # kv head 0 <- q heads 0,1,2 (mean 10), kv head 1 <- q heads 3,4,5 (mean 40); token mean 1
    expect = np.array([[10 + 1 + 0.125 * cc for cc in range(d)], [40 + 1 + 0.125 * cc for cc in range(d)]])
    np.testing.assert_allclose(q, expect, rtol=0, atol=1e-12)
    rng = np.random.default_rng(7)
    Q = rng.standard_normal((6, 3, 4)).astype(np.float32)
    q = orc.query_embedding(cfg, Q, orc.FP32)
    np.testing.assert_allclose(q, Q.astype(np.float64).reshape(2, 3, 3, 4).mean(axis=(1, 2)), atol=1e-12)


def _score_setup(orc, mode, H=4, Hq=8, d=16, T=12, Tq=3, seed=8):
    rng = np.random.default_rng(seed)
    cfg = orc.make_config(2, Hq, H, d, 5, T, kv_dtype=orc.FP32, score_mode=mode)
    st = orc.Store(cfg)
    st.rep_key[:] = rng.standard_normal(st.rep_key.shape).astype(np.float32)
    Q = rng.standard_normal((2, Hq, Tq, d)).astype(np.float32)
    return cfg, st, Q


def test_scores_match_numpy_normalised_dot(orc):
    for mode in (orc.PER_LAYER, orc.PER_HEAD):
        cfg, st, Q = _score_setup(orc, mode)
        Hq, Tq, d, H, T = 8, 3, 16, 4, 12
        sc = orc.score_groups(cfg, st, 0, 2, T, Q, Tq, (Hq * Tq * d, Tq * d, d))
        q = Q.astype(np.float64).reshape(2, H, Hq // H, Tq, d).mean(axis=(2, 3))      # [L][H][d]
        kb = st.rep_key.astype(np.float64)                                            # [L][T][H][d]
        if mode == orc.PER_LAYER:
            qf = q.reshape(2, -1)
            kf = kb.reshape(2, T, -1)
            ref = np.einsum("li,lti->lt", qf, kf) / (np.linalg.norm(qf, axis=1)[:, None] * np.linalg.norm(kf, axis=2))
        else:
            ref = np.einsum("lhc,lthc->lht", q, kb) / (
                np.linalg.norm(q, axis=2)[:, :, None] * np.linalg.norm(kb, axis=3).transpose(0, 2, 1))
        np.testing.assert_allclose(sc, ref, atol=1e-6)
        assert np.all(np.abs(sc) <= 1.0 + 1e-6)


def test_scores_special_cases(orc):
    cfg, st, Q = _score_setup(orc, 0)
    Hq, Tq, d, H, T = 8, 3, 16, 4, 12
    strides = (Hq * Tq * d, Tq * d, d)
    q = Q.astype(np.float64).reshape(2, H, Hq // H, Tq, d).mean(axis=(2, 3))
    st.rep_key[0, 3] = (2.5 * q[0]).astype(np.float32)       # parallel   -> +1
    st.rep_key[0, 4] = (-0.5 * q[0]).astype(np.float32)      # antiparallel -> -1
    st.rep_key[0, 5] = 0.0                                   # zero key  -> 0 (norm clamp)
    sc = orc.score_groups(cfg, st, 0, 2, T, Q, Tq, strides)
    assert abs(sc[0, 3] - 1.0) < 1e-6 and abs(sc[0, 4] + 1.0) < 1e-6 and sc[0, 5] == 0.0
    sc2 = orc.score_groups(cfg, st, 0, 2, T, (Q * 8).astype(np.float32), Tq, strides)   # scale invariance in Q
    np.testing.assert_allclose(sc, sc2, atol=1e-6)
    zero = orc.score_groups(cfg, st, 0, 2, T, np.zeros_like(Q), Tq, strides)
    assert np.all(zero == 0.0)
    # layer offset: scoring layer 1 alone gives row 1
    only1 = orc.score_groups(cfg, st, 1, 1, T, Q[1:], Tq, strides)
    np.testing.assert_array_equal(only1[0], sc[1])


def test_per_layer_equals_per_head_when_one_kv_head(orc):
    rng = np.random.default_rng(9)
    out = []
    for mode in (0, 1):
        cfg = orc.make_config(1, 4, 1, 16, 5, 9, kv_dtype=orc.FP32, score_mode=mode)
        st = orc.Store(cfg)
        st.rep_key[:] = np.random.default_rng(9).standard_normal(st.rep_key.shape).astype(np.float32)
        Q = np.random.default_rng(10).standard_normal((1, 4, 2, 16)).astype(np.float32)
        out.append(orc.score_groups(cfg, st, 0, 1, 9, Q, 2, (4 * 2 * 16, 2 * 16, 16)).reshape(-1))
    np.testing.assert_array_equal(out[0], out[1])


# ------------------------------------------------------------------ O5 top-K

def _brute_topk(row, k):
    order = sorted(range(len(row)), key=lambda i: (-float(row[i]), i))[:min(k, len(row))]
    return sorted(order)


@pytest.mark.parametrize("n,k", [(1, 1), (5, 8), (8, 8), (9, 8), (64, 4), (300, 64), (7, 1)])
def test_topk_bruteforce(orc, n, k):
    rng = np.random.default_rng(n * 100 + k)
    sc = rng.standard_normal((3, n)).astype(np.float32)
    sc[1] = np.round(sc[1] * 2) / 2                           # many exact ties
    idx, sel, nsel = orc.topk(sc, k)
    for r in range(3):
        want = _brute_topk(sc[r], k)
        assert nsel[r] == min(k, n)
        np.testing.assert_array_equal(idx[r, :len(want)], want)
        assert np.all(idx[r, len(want):] == -1)
        np.testing.assert_array_equal(sel[r, :len(want)], sc[r, want])
        assert np.all(np.diff(idx[r, :len(want)]) > 0)        # ascending, chronological order


def test_topk_ties_prefer_lower_index(orc):
    sc = np.array([[0.5, 0.9, 0.5, 0.5, 0.1]], np.float32)
    idx, _, _ = orc.topk(sc, 3)
    np.testing.assert_array_equal(idx[0], [0, 1, 2])


def test_budget_to_k(orc):
    g = golden()
    B = int(g["budget_tokens"][0])
    assert orc.budget_to_k(B, 50, 10_000) == int(g["budget_groups_G50"][0])
    assert orc.budget_to_k(B, 50, 100) == 100                 # fewer groups stored than the budget allows
    assert orc.budget_to_k(100, 50, 10) == 2 and orc.budget_to_k(101, 50, 10) == 3


# ------------------------------------------------------------------ O6 dequant-gather

def test_dequant_gather_places_groups_and_respects_bound(orc):
    rng = np.random.default_rng(11)
    L, H, G, d, T, k, sys_len = 2, 2, 5, 8, 6, 3, 4
    cfg = orc.make_config(L, 4, H, d, G, T, kv_dtype=orc.FP32)
    st = orc.Store(cfg)
    K = rng.standard_normal((L, T, H, G, d)).astype(np.float32)
    V = rng.standard_normal((L, T, H, G, d)).astype(np.float32)
    assert orc.quantize_frame(cfg, st, 0, L, 0, T, K, V, (T * H * G * d, H * G * d, G * d, d)) == 0
    S_act = sys_len + k * G
    ka = np.full((L, H, S_act + 2, d), 7.0, np.float32)       # 2 guard tokens past the bound
    va = np.full((L, H, S_act + 2, d), 7.0, np.float32)
    idx = np.array([[1, 3, 5], [0, 2, -1]], np.int32)
    strides = (H * (S_act + 2) * d, (S_act + 2) * d, d)
    assert orc.dequant_gather(cfg, st, 0, L, idx, k, T, ka, va, orc.FP32, strides, sys_len) == 0
    assert np.all(ka[:, :, :sys_len] == 7.0) and np.all(ka[:, :, S_act:] == 7.0)   # active size = sys + k*G, no more
    assert np.all(va[:, :, :sys_len] == 7.0) and np.all(va[:, :, S_act:] == 7.0)
    assert np.all(ka[1, :, sys_len + 2 * G:S_act] == 7.0)                           # -1 entry leaves its slot alone
    for l in range(L):
        for j in range(k):
            t = idx[l, j]
            if t < 0:
                continue
            for (src, out, s_, m_) in ((K, ka, st.scale_k, st.zero_k), (V, va, st.scale_v, st.zero_v)):
                got = out[l, :, sys_len + j * G: sys_len + (j + 1) * G]            # [H][G][d]
                want = src[l, t]                                                   # [H][G][d]
                s = s_[l, t][:, None, :]
                assert np.all(np.abs(got.astype(np.float64) - want) <= 0.5 * s * (1 + 2.0 ** -18) + 1e-6)
                # each output is one of the 16 levels of its channel
                q = (got.astype(np.float64) - m_[l, t][:, None, :]) / np.where(s == 0, 1, s)
                assert np.all(np.abs(q - np.round(q)) < 1e-4)


def test_dequant_gather_bf16_rounding_matches_torch(orc):
    rng = np.random.default_rng(12)
    L, H, G, d, T = 1, 1, 4, 16, 2
    cfg = orc.make_config(L, 1, H, d, G, T, kv_dtype=orc.FP32)
    st = orc.Store(cfg)
    K = (rng.standard_normal((L, T, H, G, d)) * 3).astype(np.float32)
    orc.quantize_frame(cfg, st, 0, 1, 0, T, K, K, (T * H * G * d, H * G * d, G * d, d))
    ka32 = np.zeros((L, H, 2 * G, d), np.float32)
    va32 = np.zeros_like(ka32)
    ka16 = np.zeros((L, H, 2 * G, d), np.uint16)
    va16 = np.zeros_like(ka16)
    idx = np.array([[0, 1]], np.int32)
    orc.dequant_gather(cfg, st, 0, 1, idx, 2, T, ka32, va32, orc.FP32, (H * 2 * G * d, 2 * G * d, d), 0)
    orc.dequant_gather(cfg, st, 0, 1, idx, 2, T, ka16, va16, orc.BF16, (H * 2 * G * d, 2 * G * d, d), 0)
    ref = torch.from_numpy(ka32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(ka16, ref)


def test_quantize_frame_layout_strides_and_token_idx(orc):
    """The frame call must agree with the single-group routine under arbitrary strides and a keep-mask."""
    rng = np.random.default_rng(13)
    L, H, G, d, F, N = 2, 2, 3, 8, 3, 7
    cfg = orc.make_config(L, 2, H, d, G, 5, kv_dtype=orc.FP32)
    st = orc.Store(cfg)
    # token-major input: [L][F][N][H][d]  (head stride d, token stride H*d)
    K = rng.standard_normal((L, F, N, H, d)).astype(np.float32)
    V = rng.standard_normal((L, F, N, H, d)).astype(np.float32)
    Ks = rng.standard_normal((L, F, N, H, d)).astype(np.float32)
    tok = np.array([[0, 2, 6], [1, 3, 4], [2, 5, 6]], np.int32)
    strides = (F * N * H * d, N * H * d, d, H * d)
    assert orc.quantize_frame(cfg, st, 0, L, 1, F, K, V, strides, K_summary=Ks, token_idx=tok,
                              tokens_per_frame_in=N) == 0
    assert np.all(st.codes_k[:, 0] == 0) and np.all(st.codes_k[:, 4] == 0)        # slots outside [1,4) untouched
    for l in range(L):
        for f in range(F):
            Xk = K[l, f, tok[f]].transpose(1, 0, 2)                                # [H][G][d]
            Xv = V[l, f, tok[f]].transpose(1, 0, 2)
            ck, sk, mk = orc.quantize_group(Xk)
            cv, sv, mv = orc.quantize_group(Xv)
            np.testing.assert_array_equal(st.scale_k[l, 1 + f], sk)
            np.testing.assert_array_equal(st.zero_v[l, 1 + f], mv)
            for h in range(H):
                for g in range(G):
                    np.testing.assert_array_equal(orc.unpack_row(st.codes_k[l, 1 + f, h, g], d), ck[h, g])
                    np.testing.assert_array_equal(orc.unpack_row(st.codes_v[l, 1 + f, h, g], d), cv[h, g])
            ref = Ks[l, f, tok[f]].astype(np.float64).mean(axis=0)                 # [H][d] from the summary keys
            np.testing.assert_allclose(st.rep_key[l, 1 + f], ref, atol=1e-6)
    # out-of-range keep index is an argument error, not a crash
    bad = tok.copy()
    bad[0, 0] = N
    assert orc.quantize_frame(cfg, st, 0, L, 1, F, K, V, strides, token_idx=bad, tokens_per_frame_in=N) != 0


# ------------------------------------------------------------------ O7 attention

def test_attend_matches_torch_sdpa(orc):
    rng = np.random.default_rng(14)
    Hq, Hk, d, S = 6, 2, 16, 37
    q = rng.standard_normal((Hq, d)).astype(np.float32)
    k = rng.standard_normal((Hk, S, d)).astype(np.float32)
    v = rng.standard_normal((Hk, S, d)).astype(np.float32)
    out = orc.attend(Hq, Hk, d, q, orc.FP32, k, v, orc.FP32, S * d, d, S, 1.0 / np.sqrt(d), out_dtype=orc.FP32)
    tq = torch.from_numpy(q).double()[:, None, :]                                   # [Hq][1][d]
    tk = torch.from_numpy(k).double().repeat_interleave(Hq // Hk, dim=0)
    tv = torch.from_numpy(v).double().repeat_interleave(Hq // Hk, dim=0)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[:, 0, :].numpy()
    np.testing.assert_allclose(out, ref, atol=1e-6)


# ------------------------------------------------------------------ O8 accounting (values the paper prints)

def test_accounting_matches_paper(orc):
    g = golden()
    v, tol = g["combined_ratio_N196_G50"]
    assert abs(orc.paper_ratio(196, 50, 4) - v) <= tol
    v, tol = g["fp16_kv_one_hour_GiB"]
    full = orc.fp16_kv_bytes(28, 1800, 196, 4, 128, 2)
    assert abs(full / 2 ** 30 - v) <= tol
    v, tol = g["after_streamingtom_GiB"]
    assert abs(full / orc.paper_ratio(196, 50, 4) / 2 ** 30 - v) <= tol
    for G in (40, 50, 60):
        for bits in (4, 2):
            v, tol = g[f"ratio_pct_{G}_{bits}bit"]
            assert abs(orc.ratio_percent(196, G, bits) - v) <= tol + 1e-9
    # codes alone reproduce the paper's number; metadata makes the real footprint larger
    cfg = orc.make_config(28, 28, 4, 128, 50, 1800)
    codes_only = orc.store_bytes(cfg, 1800, False)
    assert abs(codes_only / 2 ** 30 - g["after_streamingtom_GiB"][0]) <= 0.05
    assert abs(full / codes_only - 15.68) < 1e-9
    per_head_real = orc.store_bytes(orc.make_config(1, 1, 1, 128, 50, 1), 1, True)
    assert per_head_real == 6400 + 2048 + 512 + 4


# ------------------------------------------------------------------ CTR: similarity, split, budget, dynamic selection

def test_ctr_similarity_closed_forms_and_library(orc):
    rng = np.random.default_rng(61)
    T, N, D = 5, 7, 24
    F = rng.standard_normal((T, N, D)).astype(np.float32)
    F[2] = F[1]                      # a frame that repeats its predecessor: similarity exactly 1
    F[3, :, :] = -2.5 * F[2]         # negated and rescaled: exactly -1, whatever the scale
    F[4, 0] = 0.0                    # a zero vector: 0 by the norm clamp
    F[4, 1, :12], F[4, 1, 12:] = F[3, 1, 12:], -F[3, 1, :12]   # (b, -a) against (a, b): orthogonal
    sim = orc.ctr_similarity(F, orc.FP32)
    assert np.all(np.isneginf(sim[0]))                        # no predecessor
    np.testing.assert_allclose(sim[2], 1.0, atol=1e-7)
    np.testing.assert_allclose(sim[3], -1.0, atol=1e-7)
    assert sim[4, 0] == 0.0 and abs(sim[4, 1]) < 1e-7
    # library routine, token by token
    want = torch.nn.functional.cosine_similarity(torch.from_numpy(F[1:]).double(), torch.from_numpy(F[:-1]).double(), dim=-1)
    np.testing.assert_allclose(sim[1], want[0].numpy(), atol=1e-6)
    assert abs(sim[4, 3] - float(want[3, 3])) < 1e-6
    # positions do not mix: changing token 5 of frame 1 moves s_1^(5) and s_2^(5) only
    F2 = F.copy()
    F2[1, 5] = rng.standard_normal(D)
    sim2 = orc.ctr_similarity(F2, orc.FP32)
    changed = sim2 != sim
    assert changed[1, 5] and changed[2, 5] and changed.sum() == 2
    # the carried state: scoring frames 2.. with frame 1 as `prev` equals the tail of the whole-stream result
    tail = orc.ctr_similarity(F[2:], orc.FP32, prev=F[1])
    np.testing.assert_array_equal(tail, sim[2:])
    # 16-bit inputs are read exactly
    Fb = torch.from_numpy(F).to(torch.bfloat16)
    sb = orc.ctr_similarity(Fb.view(torch.int16).numpy().view(np.uint16), orc.BF16)
    np.testing.assert_array_equal(sb, orc.ctr_similarity(Fb.to(torch.float32).numpy(), orc.FP32))


def test_ctr_select_split_budget_and_saliency_topk(orc):
    rng = np.random.default_rng(67)
    T, N, G, tau = 40, 196, 50, 0.9
    sim = rng.uniform(0.5, 1.0, (T, N)).astype(np.float32)
    sim[0] = -np.inf                     # first frame: everything dynamic
    sim[1] = 0.99                        # everything static
    sim[2, :98], sim[2, 98:] = 0.95, 0.2  # half and half: k_s = floor(50 * 98 / 196) = 25
    sim[3, :10] = np.float32(tau)        # exactly on the threshold: NOT static (strict inequality)
    sim[3, 10:] = 0.0
    alpha = rng.uniform(0, 1, (T, N)).astype(np.float32)
    alpha[4, ::2] = 0.5                  # many equal saliencies: ties go to the lower index
    ks, kd, sidx, didx = orc.ctr_select(sim, alpha, G, tau)
    assert ks[0] == 0 and kd[0] == G and ks[1] == G and kd[1] == 0 and ks[2] == 25 and kd[2] == 25 and ks[3] == 0
    for t in range(T):
        S = np.flatnonzero(sim[t] > np.float32(tau))
        Dm = np.setdiff1d(np.arange(N), S)
        assert np.array_equal(sidx[t, :len(S)], S) and np.all(sidx[t, len(S):] == -1)
        assert ks[t] == (G * len(S)) // N and ks[t] + kd[t] == G
        assert ks[t] <= len(S) and kd[t] <= max(len(Dm), 0) or len(Dm) == 0
        # brute force with a library sort: descending saliency, ascending index among equals
        order = Dm[np.lexsort((Dm, -alpha[t, Dm].astype(np.float64)))]
        want = np.sort(order[:kd[t]])
        assert np.array_equal(didx[t, :len(want)], want) and np.all(didx[t, len(want):] == -1)
        assert len(want) == kd[t]


# ------------------------------------------------------------------ CTR: Merge_{k_s} (this code's reading of Sec. 3.3)

def test_ctr_merge_points_on_a_line_worked_by_hand(orc):
    """Six one-channel tokens 0, 1, 2, 10, 11, 12 with two neighbours each and k_s = 2, worked out from the stated rule:
    the middle tokens 1 and 11 have their two neighbours at distance 1 (rho = exp(-1)), the four outer tokens at 1 and
    2 (rho = exp(-(1 + 4)/2)).  Token 1 and token 11 tie for the highest density and the earlier one ranks first: its
    delta is its largest distance, 11; token 11 then looks back to token 1, delta = 10; every outer token has its
    denser neighbour next to it, delta = 1.  gamma = rho * delta: 11/e, 10/e, and exp(-2.5) four times, so the centres
    are tokens 1 and 11, each outer token joins the centre one step away, and the merged tokens are the means 1 and 11."""
    F = np.array([[0], [1], [2], [10], [11], [12]], np.float32)
    r = orc.ctr_merge(F, orc.FP32, np.arange(6), 2, knn=2)
    assert r["centre"].tolist() == [1, 4] and r["assign"].tolist() == [0, 0, 0, 1, 1, 1]
    np.testing.assert_allclose(r["gamma"], [np.exp(-2.5), 11 / np.e, np.exp(-2.5), np.exp(-2.5), 10 / np.e, np.exp(-2.5)],
                               rtol=1e-14)
    np.testing.assert_array_equal(r["merged"], [[1.0], [11.0]])
    # the distances are normalised by the width: the same tokens written with each channel four times change nothing
    r4 = orc.ctr_merge(np.repeat(F, 4, axis=1), orc.FP32, np.arange(6), 2, knn=2)
    assert r4["centre"].tolist() == [1, 4] and r4["assign"].tolist() == [0, 0, 0, 1, 1, 1]
    np.testing.assert_allclose(r4["gamma"], r["gamma"], rtol=1e-14)
    # a subset as the static set: tokens 0, 2, 3, 5 -> neighbours change, the rule does not
    rs = orc.ctr_merge(F, orc.FP32, np.array([0, 2, 3, 5]), 2, knn=1)
    assert rs["centre"].tolist() in ([0, 3], [0, 5], [2, 3], [2, 5]) and rs["assign"].tolist() == [0, 0, 1, 1]
    np.testing.assert_array_equal(rs["merged"], [[1.0], [11.0]])


def test_ctr_merge_invariants(orc):
    """Whatever the clustering decides: k_s clusters, none empty, every static token in exactly one, a centre in its
    own cluster, each merged token the mean of its members (so a convex combination, channel by channel inside the
    members' range); k_s = |S| leaves the tokens as they are; relabelling the tokens permutes the result with them."""
    rng = np.random.default_rng(3)
    N, D = 40, 24
    F = rng.standard_normal((N, D)).astype(np.float32)
    S = np.sort(rng.choice(N, size=29, replace=False)).astype(np.int32)
    for k_s in (1, 2, 7, 28, 29):
        r = orc.ctr_merge(F, orc.FP32, S, k_s)
        c, a, m = r["centre"], r["assign"], r["merged"]
        assert len(c) == k_s and np.all(np.diff(c) > 0) and np.all(np.isin(c, S))
        assert a.min() == 0 and a.max() == k_s - 1 and len(np.unique(a)) == k_s
        for j in range(k_s):
            members = S[a == j]
            assert c[j] in members
            want = F[members].astype(np.float64).mean(axis=0)
            np.testing.assert_allclose(m[j], want, rtol=1e-6, atol=1e-7)
            assert np.all(m[j] <= F[members].max(axis=0) + 1e-6) and np.all(m[j] >= F[members].min(axis=0) - 1e-6)
        if k_s == len(S):
            np.testing.assert_array_equal(c, S)
            np.testing.assert_array_equal(m, F[S])
    # permutation: token i of the permuted frame is token perm[i] of the original
    k_s = 7
    base = orc.ctr_merge(F, orc.FP32, S, k_s)
    perm = rng.permutation(N)
    inv = np.argsort(perm)
    Sp = np.sort(inv[S]).astype(np.int32)
    rp = orc.ctr_merge(F[perm], orc.FP32, Sp, k_s)
    assert sorted(perm[rp["centre"]].tolist()) == base["centre"].tolist()
    clusters = lambda r, S_, back: sorted(sorted(back[S_[r["assign"] == j]].tolist()) for j in range(k_s))
    assert clusters(rp, Sp, perm) == clusters(base, S, np.arange(N))


def test_ctr_merge_separated_blobs_and_retained_group(orc):
    """Three tight, well separated blobs and k_s = 3: the clusters are the blobs and the merged tokens their means
    (numpy).  The retained group then interleaves the selected dynamic rows (bit for bit) with the merged rows rounded
    to the feature type (torch's nearest-even), in position order, a merged token at its centre's position."""
    import torch
    rng = np.random.default_rng(8)
    N, D, G = 30, 16, 9
    blob = rng.integers(0, 3, size=N)
    blob[:3] = [0, 1, 2]
    mu = 20.0 * rng.standard_normal((3, D))
    X = torch.from_numpy((mu[blob] + 0.05 * rng.standard_normal((N, D))).astype(np.float32)).to(torch.bfloat16)
    Xf = X.to(torch.float32).numpy().astype(np.float64)
    Xu = X.view(torch.int16).numpy().view(np.uint16)
    dyn = np.array([4, 11, 20, 27], np.int32)
    S = np.setdiff1d(np.arange(N), dyn).astype(np.int32)
    r = orc.ctr_merge(Xu, orc.BF16, S, 3)
    assert sorted(blob[r["centre"]].tolist()) == [0, 1, 2]
    for j in range(3):
        members = S[r["assign"] == j]
        b = blob[r["centre"][j]]
        assert np.array_equal(members, S[blob[S] == b])
        np.testing.assert_allclose(r["merged"][j], Xf[members].mean(axis=0), rtol=1e-6, atol=1e-6)
    assert r["margin_centres"] > 0.5 and r["margin_assign"].min() > 0.9     # nothing about these decisions is close
    ret, pos = orc.ctr_retain(Xu, orc.BF16, dyn, r["centre"], r["merged"], G)
    want_pos = np.sort(np.concatenate([dyn, r["centre"]]))
    assert np.array_equal(pos[:7], want_pos) and np.all(pos[7:] == -1) and not ret[7:].any()
    merged16 = torch.from_numpy(r["merged"]).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    for w, t in enumerate(want_pos):
        if t in dyn:
            assert np.array_equal(ret[w], Xu[t])
        else:
            assert np.array_equal(ret[w], merged16[list(r["centre"]).index(t)])


# ------------------------------------------------------------------ whole path on the tiny workload

def test_tiny_workload_retrieves_planted_groups_and_bounds_active_cache(orc):
    from paper_2510_18269_b200 import synth
    sh = synth.C1
    K, V = synth.kv_stream(sh)
    Q = synth.queries(sh)
    planted = synth.planted_groups(sh)
    cfg = orc.make_config(sh.L, sh.H_q, sh.H_k, sh.d, sh.G, sh.T, kv_dtype=orc.FP32)
    st = orc.Store(cfg)
    kn, vn, qn = synth.as_u16(K), synth.as_u16(V), synth.as_u16(Q)
    strides = (sh.T * sh.H_k * sh.G * sh.d, sh.H_k * sh.G * sh.d, sh.G * sh.d, sh.d)
    sys_len = 3
    for t in range(sh.T):                                      # frames arrive one by one
        assert orc.quantize_frame(cfg, st, 0, 1, t, 1, kn[:, t:], vn[:, t:], strides) == 0
        if t % 16 == 15 or t == 2:
            n = t + 1
            sc = orc.score_groups(cfg, st, 0, 1, n, qn, sh.T_q, (sh.H_q * sh.T_q * sh.d, sh.T_q * sh.d, sh.d))
            idx, _, nsel = orc.topk(sc, sh.k)
            ksel = min(sh.k, n)
            assert nsel[0] == ksel
            S = sys_len + sh.k * sh.G
            ka = np.full((1, 1, S + 1, sh.d), np.nan, np.float32)
            va = np.full((1, 1, S + 1, sh.d), np.nan, np.float32)
            assert orc.dequant_gather(cfg, st, 0, 1, idx, sh.k, n, ka, va, orc.FP32, ((S + 1) * sh.d, (S + 1) * sh.d, sh.d), sys_len) == 0
            written = ~np.isnan(ka[0, 0, :, 0])
            assert written.sum() == ksel * sh.G                # active size is K*G whatever the stream length
            assert not written[:sys_len].any() and not written[sys_len + ksel * sh.G:].any()
    np.testing.assert_array_equal(idx[0], planted[0].numpy())  # the planted groups are exactly the ones retrieved
    # and what was reconstructed is within s/2 of the original keys
    for j, t in enumerate(idx[0]):
        got = ka[0, 0, sys_len + j * sh.G: sys_len + (j + 1) * sh.G]
        assert np.all(np.abs(got - kn[0, t, 0]) <= 0.5 * st.scale_k[0, t, 0] * (1 + 2.0 ** -18) + 1e-6)
