"""CPU-only checks of the C-ABI library: it builds, loads, exports every symbol the
header declares, and its host-side logic (layout, K formula, argument validation)
behaves as documented; and an arithmetic identity one kernel relies on.  No kernel is launched here."""
import ctypes as C
import re
from pathlib import Path

import numpy as np
import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def oqm():
    from paper_2510_18269_b200 import build, oqm as m
    build.build()
    m.lib()
    return m


def declared_symbols():
    text = "".join(h.read_text() for h in sorted((ROOT / "include").glob("*.h")))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(stom_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(oqm):
    names = declared_symbols()
    assert "stom_oqm_quantize_frame" in names and "stom_oqm_dequant_gather" in names
    assert "stom_oqm_score_groups" in names and "stom_oqm_topk" in names
    assert "stom_ctr_similarity" in names and "stom_ctr_select" in names and "stom_ctr_reduce" in names
    for n in names:
        assert hasattr(oqm.lib(), n), f"{n} declared in the header but not exported"
    assert set(oqm.EXPORTS) <= set(names)


def test_store_layout_and_bind(oqm):
    cfg = oqm.make_config(28, 28, 4, 128, 50, 7200)
    lay = oqm.stom_oqm_store_layout(cfg)
    slots = 28 * 7200 * 4
    assert lay.bytes_codes == slots * 50 * 64 and lay.bytes_meta == slots * 128 * 4 and lay.bytes_norm2 == slots * 4
    offs = [lay.off_codes_k, lay.off_codes_v, lay.off_scale_k, lay.off_zero_k, lay.off_scale_v, lay.off_zero_v,
            lay.off_rep_key, lay.off_rep_norm2]
    assert offs == sorted(offs) and all(o % 256 == 0 for o in offs)
    assert lay.bytes_total >= 2 * lay.bytes_codes + 5 * lay.bytes_meta + lay.bytes_norm2
    desc = oqm.StoreDesc()
    base = 0x7f0000000000                                   # pointer arithmetic only; never dereferenced
    assert oqm.lib().stom_oqm_store_bind(C.byref(cfg), C.c_void_p(base), C.byref(desc)) == 0
    assert desc.codes_k == base and desc.rep_norm2 == base + lay.off_rep_norm2
    assert oqm.lib().stom_oqm_store_bind(C.byref(cfg), C.c_void_p(base + 8), C.byref(desc)) == -3   # alignment
    # 16-bit metadata halves the five metadata arrays and nothing else
    for meta in (oqm.FP16, oqm.BF16):
        lay16 = oqm.stom_oqm_store_layout(oqm.make_config(28, 28, 4, 128, 50, 7200, meta_dtype=meta))
        assert lay16.bytes_meta * 2 == lay.bytes_meta and lay16.bytes_codes == lay.bytes_codes
        assert lay16.bytes_norm2 == lay.bytes_norm2 and lay16.bytes_total < lay.bytes_total


def test_budget_to_k_matches_paper_example(oqm):
    assert oqm.stom_oqm_budget_to_k(64 * 196, 50, 10_000) == 251     # appendix: ceil(12544 / 50)
    assert oqm.stom_oqm_budget_to_k(64 * 196, 50, 100) == 100
    assert oqm.stom_oqm_budget_to_k(-1, 50, 100) < 0


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=96), -2), (dict(group_tokens=0), -2), (dict(group_tokens=65), -2), (dict(bits=3), -6),
    (dict(n_q_heads=7), -2), (dict(kv_dtype=5), -6), (dict(n_layers=0), -1), (dict(score_mode=3), -6),
    (dict(meta_dtype=3), -6), (dict(meta_dtype=-1), -6),
])
def test_config_validation(oqm, kw, code):
    args = dict(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=128, group_tokens=50, capacity_groups=10)
    args.update(kw)
    cfg = oqm.make_config(**args)
    lay = oqm.Layout()
    assert oqm.lib().stom_oqm_store_layout(C.byref(cfg), C.byref(lay)) == code
    assert oqm.lib().stom_status_string(code).decode() != "unknown status"


def test_entry_points_reject_bad_arguments_before_any_launch(oqm):
    L = oqm.lib()
    cfg = oqm.make_config(2, 8, 4, 128, 50, 10)
    desc = oqm.StoreDesc(*[0x7f0000000000 + 4096 * i for i in range(8)])
    p = C.c_void_p(0x7f1000000000)
    i64, i32 = C.c_int64, C.c_int32
    st = (i64(10 * 4 * 50 * 128), i64(4 * 50 * 128), i64(50 * 128), i64(128))

    def quant(**o):
        a = dict(lb=0, lc=2, gb=0, gc=10, K=p, V=p, st=st, tok=None, nin=0)
        a.update(o)
        return L.stom_oqm_quantize_frame(C.byref(cfg), C.byref(desc), i32(a["lb"]), i32(a["lc"]), i32(a["gb"]),
                                         i32(a["gc"]), a["K"], a["V"], *a["st"], None, a["tok"], i32(a["nin"]),
                                         None, None)
    assert quant(K=None) == -1
    assert quant(lc=3) == -1                                  # layers beyond n_layers
    assert quant(gb=5, gc=6) == -4                            # beyond capacity_groups
    assert quant(K=C.c_void_p(0x7f1000000002)) == -3          # misaligned base
    assert quant(st=(st[0], st[1], st[2], i64(100))) == -3    # token stride breaks 16-byte rows
    assert quant(tok=p, nin=0) == -1
    assert quant(gc=0) == 0                                   # empty call is a no-op
    null_desc = oqm.StoreDesc()
    assert L.stom_oqm_quantize_frame(C.byref(cfg), C.byref(null_desc), 0, 2, 0, 1, p, p, *st, None, None, 0, None, None) == -1

    def score(**o):
        a = dict(n=10, Q=p, Tq=4, sc=p, ws=p, wsb=1 << 20)
        a.update(o)
        return L.stom_oqm_score_groups(C.byref(cfg), C.byref(desc), 0, 2, i32(a["n"]), a["Q"], i32(a["Tq"]),
                                       i64(8 * 4 * 128), i64(4 * 128), i64(128), a["sc"], a["ws"], i64(a["wsb"]), None)
    assert score(Q=None) == -1 and score(Tq=0) == -1 and score(n=11) == -4
    assert score(ws=None) == -8 and score(wsb=16) == -8
    assert oqm.stom_oqm_score_workspace_bytes(cfg, 2) >= 2 * 4 * 129 * 4

    assert L.stom_oqm_topk(None, 1, 10, i64(10), 4, p, None, None, None) == -1
    assert L.stom_oqm_topk(p, 1, 10, i64(5), 4, p, None, None, None) == -1      # row stride shorter than the row
    assert L.stom_oqm_topk(p, 1, 10, i64(10), 0, p, None, None, None) == -1
    assert L.stom_oqm_topk(p, 0, 10, i64(10), 4, p, None, None, None) == 0

    def gather(**o):
        a = dict(idx=p, k=4, n=10, ka=p, va=p, od=0, st=(i64(4 * 300 * 128), i64(300 * 128), i64(128)), off=3)
        a.update(o)
        return L.stom_oqm_dequant_gather(C.byref(cfg), C.byref(desc), 0, 2, a["idx"], i32(a["k"]), i32(a["n"]),
                                         a["ka"], a["va"], i32(a["od"]), *a["st"], i32(a["off"]), None, None)
    assert gather(idx=None) == -1 and gather(k=0) == -1 and gather(n=11) == -4 and gather(od=2) == -6
    assert gather(ka=C.c_void_p(0x7f1000000008)) == -3 and gather(off=-1) == -1
    assert gather(st=(i64(4 * 300 * 128), i64(300 * 128), i64(64))) == -1       # token stride shorter than a row


def test_host_buffer_entry_points_reject_bad_arguments_before_any_cuda_call(oqm):
    L = oqm.lib()
    cfg = oqm.make_config(2, 8, 4, 128, 50, 10)
    desc = oqm.StoreDesc(*[0x7f0000000000 + 4096 * i for i in range(8)])
    p = C.c_void_p(0x7f1000000000)          # never dereferenced: every call below is refused on the host
    i64, i32 = C.c_int64, C.c_int32
    need_q = oqm.stom_oqm_quantize_host_scratch_bytes(cfg, 2, 10)
    assert need_q >= 2 * 2 * 10 * 4 * 50 * 128 * 2 and need_q % 256 == 0

    def quant(K=p, V=p, scr=p, nbytes=need_q, lc=2, gc=10):
        return L.stom_oqm_quantize_frame_host(C.byref(cfg), C.byref(desc), 0, i32(lc), 0, i32(gc), K, V, scr,
                                              i64(nbytes), None, None)
    assert quant(K=None) == -1 and quant(V=None) == -1 and quant(gc=-1) == -1
    assert quant(scr=None) == -8 and quant(nbytes=need_q - 1) == -8
    assert quant(scr=C.c_void_p(0x7f1000000004)) == -8        # scratch must be 16-byte aligned

    need_r = oqm.stom_oqm_retrieve_host_scratch_bytes(cfg, 2, 10, 4, 4, oqm.BF16)
    assert need_r > 2 * 2 * 4 * 4 * 50 * 128 * 2              # holds the reconstructed K and V of the call
    assert oqm.stom_oqm_retrieve_host_scratch_bytes(cfg, 2, 10, 0, 4, oqm.BF16) == -1
    assert oqm.stom_oqm_retrieve_host_scratch_bytes(cfg, 2, 10, 4, 4, oqm.FP32) == -6

    def retr(Q=p, idx=p, ka=p, va=p, scr=p, nbytes=need_r, od=0, k=4, Tq=4):
        return L.stom_oqm_retrieve_host(C.byref(cfg), C.byref(desc), 0, 2, 10, Q, i32(Tq), i32(k), idx, ka, va,
                                        i32(od), scr, i64(nbytes), None, None)
    assert retr(Q=None) == -1 and retr(idx=None) == -1 and retr(k=0) == -1 and retr(Tq=0) == -1
    assert retr(ka=None) == -1 and retr(va=None) == -1        # both cache pointers or neither
    assert retr(od=2) == -6
    assert retr(scr=None) == -8 and retr(nbytes=need_r - 1) == -8
    assert retr(scr=C.c_void_p(0x7f1000000010)) == -8         # scratch must be 256-byte aligned


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2510_18269_b200 import oqm as m
    monkeypatch.setattr(m, "_lib", None)
    monkeypatch.setattr(m, "LIB_PATH", tmp_path / "absent.so")
    with pytest.raises(ImportError):
        m.lib()


def test_quotient_by_reciprocal_and_one_correction_is_the_correctly_rounded_one():
    """The merge kernel divides a cluster's binary32 sums by its size n with y = rn(1/n), q = rn(s y), r = s - q n
    (exact), q' = rn(q + r y).  That this equals the correctly rounded s / n -- which is what the oracle's binary64
    mean, rounded once, is compared with -- is checked here in numpy for every n a frame can have."""
    rng = np.random.default_rng(97)
    for n in range(1, 225):
        y = np.float32(1) / np.float32(n)
        s = (rng.standard_normal(20000) * rng.choice([0.01, 1.0, 300.0], 20000)).astype(np.float32)
        q = (s * y).astype(np.float32)
        r = (s.astype(np.float64) - q.astype(np.float64) * n).astype(np.float32)      # exact: one FMA on the GPU
        got = (q.astype(np.float64) + r.astype(np.float64) * float(y)).astype(np.float32)
        want = (s.astype(np.float64) / n).astype(np.float32)
        assert np.array_equal(got, want), n
