"""CPU tests of the library's host side: exports, layout, plan, validation, classification.

No kernel is launched: every call either is host-only or fails its argument checks first."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest

from oracle import catekv_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ck():
    from paper_2608_30295_b200 import build
    build.build()
    from paper_2608_30295_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(ck):
    hdr = open(os.path.join(ROOT, "include", "catekv.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(catekv_[a-z_0-9]+)\s*\(", hdr))
    assert len(declared) >= 15
    lib = C.CDLL(ck.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(ck.EXPORTS)
    assert ck.catekv_version() == 2001
    assert ck._lib.catekv_error_string(-3) == b"segment capacity exceeded"


def test_cache_layout(ck):
    off, cap, total = ck.catekv_cache_layout(2, 3, [0, 1, 127, 128, 129, 1000], 16)
    assert list(cap) == [128, 128, 256, 256, 256, 1024]
    assert list(off) == [0, 128, 256, 512, 768, 1024]
    assert total == 2048
    with pytest.raises(ck.CatekvError) as e:
        ck.catekv_cache_layout(1, 2, [5, -1], 0)
    assert e.value.code == ck.ERR_INVALID_ARG


def _host_cache(ck, B, Hkv, lens, max_new=0):
    off, cap, total = ck.catekv_cache_layout(B, Hkv, lens, max_new)
    seg_len = np.array(lens, dtype=np.int32)
    keep = (off, cap, seg_len)
    fake = 0x10000  # non-null stand-ins for device pointers; nothing dereferences them in these tests
    st = ck.CacheStruct(B, Hkv, 128, 0, total, fake, fake, fake, fake, off.ctypes.data, cap.ctypes.data,
                        seg_len.ctypes.data)
    return st, keep


def _plan(ck, lens, B, Hkv, num_ctas):
    st, keep = _host_cache(ck, B, Hkv, lens)
    nbytes = ck._lib.catekv_decode_plan_bytes(B, Hkv, num_ctas)
    buf = np.zeros(nbytes, dtype=np.uint8)
    rc = ck._lib.catekv_decode_plan(C.byref(st), num_ctas, buf.ctypes.data, None, nbytes, None)
    assert rc == 0
    hdr = buf[:48].view(np.int32)
    n_items, n_slots = int(hdr[3]), int(hdr[4])
    off_cta, off_items, off_seg = int(hdr[8]), int(hdr[9]), int(hdr[10])
    ch = buf[off_cta:off_cta + 48 * num_ctas].view(np.int32).reshape(num_ctas, 12)
    cta = np.concatenate([ch[:, 0], ch[-1:, 1]])
    assert np.array_equal(ch[1:, 0], ch[:-1, 1])  # consecutive item ranges
    raw = buf[off_items:off_items + 32 * n_items].view(np.int32).reshape(-1, 8)
    seg_off = keep[0]
    for c in range(num_ctas):  # the inline copy of the CTA's first item
        if ch[c, 0] < ch[c, 1]:
            assert np.array_equal(ch[c, 4:12], raw[ch[c, 0]])
    for r in raw:  # pool row of the piece's first row
        assert int(r[4:6].view(np.int64)[0]) == int(seg_off[r[0]]) + int(r[1])
    # (seg, t0, t1 or -1 for the piece that follows the live length, slot)
    items = np.stack([raw[:, 0], raw[:, 1], np.where(raw[:, 6] == 1, -1, raw[:, 2]), raw[:, 3]], axis=1) \
        if n_items else np.zeros((0, 4), dtype=np.int32)
    segs = buf[off_seg:off_seg + 16 * B * Hkv].view(np.int32).reshape(-1, 4)
    return cta, items, segs, n_slots


@pytest.mark.parametrize("lens,num_ctas", [
    ([1024, 1024, 32768, 32768, 1024, 32768, 1024, 32768], 296),
    ([0, 5, 0, 17, 300, 1], 4),
    ([100], 7),
    ([0, 0], 3),
    ([64, 64, 64, 64], 2),
    (list(np.random.default_rng(5).integers(0, 5000, size=48)), 37),
])
def test_decode_plan_covers_every_row_once_and_balances(ck, lens, num_ctas):
    lens = [int(x) for x in lens]
    n = len(lens)
    cta, items, segs, n_slots = _plan(ck, lens, 1, n, num_ctas)
    assert cta[0] == 0 and np.all(np.diff(cta) >= 0) and cta[-1] == len(items)
    # every segment's rows are covered exactly once, in order, by consecutive items
    pos = {s: 0 for s in range(n)}
    pieces = {s: [] for s in range(n)}
    for i, (seg, t0, t1, slot) in enumerate(items):
        assert t0 == pos[seg]
        end = lens[seg] if t1 < 0 else t1
        assert end > t0 or (lens[seg] == 0 and t1 < 0)  # an empty segment still owns one item
        pos[seg] = end
        pieces[seg].append((i, t1, slot))
    for s in range(n):
        assert pos[s] == lens[s]
        sb, npieces, plan_len, _ = segs[s]
        assert plan_len == lens[s]
        assert npieces == len(pieces[s])
        assert npieces >= 1
        if npieces:
            assert pieces[s][-1][1] == -1  # the last piece follows the live length
            assert all(t1 >= 0 for (_, t1, _) in pieces[s][:-1])
        if npieces == 1:
            assert pieces[s][0][2] == -1
        elif npieces > 1:
            assert [sl for (_, _, sl) in pieces[s]] == list(range(sb, sb + npieces))
    assert n_slots == sum(len(p) for p in pieces.values() if len(p) > 1)
    # balance: every non-empty segment's end is charged 256 rows (the extra work of the CTA that owns it);
    # no CTA gets more than an equal share of the charged rows rounded up to 16 (a charge may overshoot it)
    charge = 256
    charged = sum(lens) + charge * sum(1 for x in lens if x > 0)
    quota = max(16, -(-(-(-charged // num_ctas)) // 16) * 16)
    for c in range(num_ctas):
        rows = ends = 0
        for seg, t0, t1, _ in items[cta[c]:cta[c + 1]]:
            rows += (lens[seg] if t1 < 0 else t1) - t0
            ends += 1 if (t1 < 0 and lens[seg] > 0) else 0
        assert rows <= quota and rows + charge * ends <= quota + charge


def test_append_capacity_is_checked_before_launch(ck):
    st, keep = _host_cache(ck, 1, 2, [128, 5], 0)  # segment 0 is exactly full
    rc = ck._lib.catekv_append(C.byref(st), 0x10000, 0x10000, None)
    assert rc == ck.ERR_CAPACITY
    assert list(keep[2]) == [128, 5]  # host mirror untouched
    assert ck._lib.catekv_append(C.byref(st), None, 0x10000, None) == ck.ERR_INVALID_ARG


def test_decode_attn_argument_checks(ck):
    st, keep = _host_cache(ck, 1, 2, [10, 10])
    nbytes = ck._lib.catekv_decode_plan_bytes(1, 2, 4)
    buf = np.zeros(nbytes, dtype=np.uint8)
    assert ck._lib.catekv_decode_plan(C.byref(st), 4, buf.ctypes.data, None, nbytes, None) == 0
    f = 0x10000
    call = lambda **kw: ck._lib.catekv_decode_attn(
        C.byref(st), kw.get("q", f), kw.get("Hq", 8), kw.get("scale", 0.0), f, kw.get("dt", 0), None,
        kw.get("ph", buf.ctypes.data), f, kw.get("pb", nbytes), f, kw.get("wsb", 1 << 30), None)
    assert call(q=None) == ck.ERR_INVALID_ARG
    assert call(Hq=7) == ck.ERR_INVALID_ARG          # not a multiple of Hkv
    assert call(Hq=18) == ck.ERR_UNSUPPORTED         # G = 9
    assert call(dt=5) == ck.ERR_UNSUPPORTED
    assert call(scale=-1.0) == ck.ERR_INVALID_ARG
    assert call(wsb=16) == ck.ERR_WORKSPACE
    assert call(pb=8) == ck.ERR_INVALID_ARG
    junk = np.zeros(nbytes, dtype=np.uint8)
    assert call(ph=junk.ctypes.data) == ck.ERR_INVALID_ARG   # not a plan
    st2, keep2 = _host_cache(ck, 1, 2, [10, 10])
    st2.d = 64
    assert ck._lib.catekv_decode_plan(C.byref(st2), 4, buf.ctypes.data, None, nbytes, None) == ck.ERR_UNSUPPORTED
    assert ck._lib.catekv_decode_plan(C.byref(st), 4, buf.ctypes.data, None, 8, None) == ck.ERR_WORKSPACE


def test_select_argument_checks(ck):
    st, keep = _host_cache(ck, 1, 2, [64, 200], 0)
    seq = np.array([200], dtype=np.int32)
    mask = np.array([1, 0], dtype=np.uint8)
    f = 0x10000

    def call(**kw):
        p = ck.SelectParams(1, kw.get("Hq", 8), 2, kw.get("d", 128), kw.get("L_obs", 16), 4, kw.get("local", 16),
                            kw.get("budget", 64), kw.get("eta", 1.0), kw.get("mode", 0), kw.get("param", 0), 0,
                            f, f, f, 0, 0, 128, seq.ctypes.data, mask.ctypes.data)
        return ck._lib.catekv_select_compact(C.byref(p), C.byref(st), None, 0, f, kw.get("wsb", 1 << 40), None)

    assert call(local=8) == ck.ERR_INVALID_ARG       # local window shorter than the observation window
    assert call(d=64) == ck.ERR_UNSUPPORTED
    assert call(Hq=18) == ck.ERR_UNSUPPORTED
    assert call(L_obs=129, local=129) == ck.ERR_UNSUPPORTED  # G * L_obs = 516 > 512
    assert call(mode=2, param=4) == ck.ERR_INVALID_ARG  # even window
    assert call(mode=1, param=0) == ck.ERR_INVALID_ARG
    assert call(mode=9) == ck.ERR_UNSUPPORTED
    assert call(wsb=64) == ck.ERR_WORKSPACE
    assert call(budget=150) == ck.ERR_CAPACITY       # 150 kept rows do not fit segment 0 (capacity 128)
    assert list(keep[2]) == [64, 200]


def test_head_cv_argument_checks(ck):
    seq = np.array([100], dtype=np.int32)
    f = 0x10000
    call = lambda **kw: ck._lib.catekv_head_cv(f, f, 0, 0, 128, seq.ctypes.data, 1, kw.get("Hq", 8), 2, kw.get("d", 128),
                                               kw.get("L_obs", 16), kw.get("L_init", 4), kw.get("L_rec", 4),
                                               kw.get("k", 0.99), 1.0, 1, f, f, kw.get("wsb", 1 << 40), None)
    assert call(d=64) == ck.ERR_UNSUPPORTED
    assert call(k=1.5) == ck.ERR_INVALID_ARG
    assert call(L_init=60, L_rec=40) == ck.ERR_INVALID_ARG   # no column left
    assert call(L_obs=129) == ck.ERR_UNSUPPORTED
    assert call(wsb=8) == ck.ERR_WORKSPACE
    assert ck.catekv_head_cv_workspace_bytes(1, 8, 2, 100, 16, 60, 40) == 0


def test_classify_heads_matches_oracle(ck):
    rng = np.random.default_rng(30)
    for N, H, r in [(8, 112, 0.5), (3, 4, 0.5), (5, 16, 0.4), (1, 7, 0.3), (4, 9, 0.0), (4, 9, 1.0)]:
        cv = rng.random((N, H)).astype(np.float32)
        want = orc.static_head_mask(cv.astype(np.float64), float(np.float32(r)))
        got = ck.catekv_classify_heads(cv, r)
        assert np.array_equal(got, want), (N, H, r)
    cv = np.array([[9, 1, 8, 2], [9, 7, 1, 2], [9, 1, 8, 2]], dtype=np.float32)
    assert list(ck.catekv_classify_heads(cv, 0.5)) == [1, 0, 1, 0]


def test_retrieve_lengths_match_the_oracle_selection_sizes(ck):
    from oracle import catekv_oracle as orc
    rng = np.random.default_rng(11)
    for _ in range(40):
        n_segs = int(rng.integers(1, 7))
        lens = [int(rng.integers(0, 3000)) for _ in range(n_segs)]
        cs = int(rng.choice([1, 2, 4, 8, 16, 32]))
        budget, sink, local = int(rng.integers(0, 1200)), int(rng.integers(0, 20)), int(rng.integers(0, 100))
        mask = rng.integers(0, 2, size=n_segs).astype(np.uint8)
        st, keep = _host_cache(ck, 1, n_segs, lens)
        got = np.zeros(n_segs, dtype=np.int32)
        rc = ck._lib.catekv_retrieve_lengths(C.byref(st), cs, mask.ctypes.data, budget, sink, local, got.ctypes.data)
        assert rc == 0
        for s, L in enumerate(lens):
            want = len(orc.retrieve_indices(np.zeros((L + cs - 1) // cs), L, sink, local, budget, cs)) if mask[s] else L
            assert got[s] == want, (lens, cs, budget, sink, local, s)
    assert ck._lib.catekv_retrieve_lengths(C.byref(st), 3, mask.ctypes.data, 10, 0, 0, got.ctypes.data) == ck.ERR_UNSUPPORTED


def _pages(ck, st, n_segs, n_pages, max_pages):
    table = np.full((n_segs, max_pages), -1, dtype=np.int32)
    seg_pages = np.zeros(n_segs, dtype=np.int32)
    fake = 0x10000
    pg = ck.PagesStruct(max_pages, n_pages, 0, 0, fake, fake, fake, table.ctypes.data, seg_pages.ctypes.data, fake)
    st.pages = C.pointer(pg)
    return pg, table, seg_pages


def test_pages_bookkeeping_without_a_device(ck):
    # the paths of catekv_pages_reserve that copy nothing: refusals, and requests the capacity already covers
    st, keep = _host_cache(ck, 1, 3, [128, 5, 200], 0)  # capacities 128, 128, 256
    assert ck._lib.catekv_pages_reserve(C.byref(st), 1, None) == ck.ERR_INVALID_ARG  # no pages attached
    pg, table, seg_pages = _pages(ck, st, 3, n_pages=2, max_pages=2)
    assert ck._lib.catekv_pages_reserve(C.byref(st), 0, None) == 0
    assert ck._lib.catekv_pages_reserve(C.byref(st), -1, None) == ck.ERR_INVALID_ARG
    # 129 more rows: segment 0 would need 3 pages (> max_pages); 100 more rows: 2 + 0 + 1 pages > the 2 of the pools
    for n_new in (129, 100):
        assert ck._lib.catekv_pages_reserve(C.byref(st), n_new, None) == ck.ERR_CAPACITY
        assert pg.next_free == 0 and not seg_pages.any() and (table == -1).all()
    # capacity seen by the other host checks: appends are refused while no page has been handed out
    assert ck._lib.catekv_append(C.byref(st), 0x10000, 0x10000, None) == ck.ERR_CAPACITY
    assert ck._lib.catekv_cache_advance(C.byref(st), 1) == ck.ERR_CAPACITY
    # with a page per segment on the books (as catekv_pages_reserve would leave them) 64 more rows fit
    seg_pages[:] = 1
    table[:, 0] = [0, 1, 2]
    pg.n_pages, pg.next_free = 3, 3
    assert ck._lib.catekv_cache_advance(C.byref(st), 64) == 0
    assert list(keep[2]) == [192, 69, 264]
    assert ck._lib.catekv_cache_advance(C.byref(st), 1) == ck.ERR_CAPACITY  # segment 0 is full again
    # plans accept lengths beyond the segment's own capacity and carry that capacity in every work item
    nbytes = ck._lib.catekv_decode_plan_bytes(1, 3, 4)
    buf = np.zeros(nbytes, dtype=np.uint8)
    assert ck._lib.catekv_decode_plan(C.byref(st), 4, buf.ctypes.data, None, nbytes, None) == 0
    hdr = buf[:48].view(np.int32)
    raw = buf[int(hdr[9]):int(hdr[9]) + 32 * int(hdr[3])].view(np.int32).reshape(-1, 8)
    assert all(int(r[7]) == int(keep[1][r[0]]) for r in raw)
    # calls that walk contiguous segments refuse the paged cache
    assert ck._lib.catekv_retrieval_meta_bytes(C.byref(st), 8) == 0
    got = np.zeros(3, dtype=np.int32)
    m = np.ones(3, dtype=np.uint8)
    assert ck._lib.catekv_retrieve_lengths(C.byref(st), 8, m.ctypes.data, 64, 0, 0, got.ctypes.data) == ck.ERR_UNSUPPORTED


def test_fused_append_refuses_lengths_below_the_plan(ck):
    st, keep = _host_cache(ck, 1, 2, [300, 40], 8)
    nbytes = ck._lib.catekv_decode_plan_bytes(1, 2, 3)
    buf = np.zeros(nbytes, dtype=np.uint8)
    assert ck._lib.catekv_decode_plan(C.byref(st), 3, buf.ctypes.data, None, nbytes, None) == 0
    keep[2][0] = 299  # the list has shrunk since
    f = 0x10000
    rc = ck._lib.catekv_append_decode_attn(C.byref(st), f, f, f, 8, 0.0, f, 0, None, buf.ctypes.data, f, nbytes, f, 1 << 30,
                                           None)
    assert rc == ck.ERR_INVALID_ARG and list(keep[2]) == [299, 40]


def test_bf16_tie_rule_of_the_attention_check():
    """helpers.bf16_tie_flips excuses a differing bf16 element only when the fp32 value sits at a rounding tie."""
    import helpers as H
    from oracle import catekv_oracle as orc

    def bits(v):
        return orc.f64_to_bf16(np.array(v, dtype=np.float64))

    lo, hi = 3.0, 3.015625          # adjacent bf16 values in [2, 4): one ulp = 2^-6
    mid = 0.5 * (lo + hi)
    ref = np.array([mid - 2e-7, mid - 2e-7, 1.0, mid - 2e-7])
    x32 = np.array([mid + 3e-7, mid + 3e-7, 1.0, 3.012])     # fp32 results; the last one is far from the tie
    got = bits([hi, 3.03125, 1.0, hi])                        # element 1 is two ulps away
    tie = H.bf16_tie_flips(got, bits(ref), x32, ref)
    # element 3 widens the measured error to 3e-3, which would excuse anything: use a tensor without it first
    assert list(H.bf16_tie_flips(got[:3], bits(ref[:3]), x32[:3], ref[:3])) == [True, False, False]
    assert list(tie[:3]) == [True, False, False]
    # a flip whose fp32 value is nowhere near the midpoint is not excused when the tensor's error is small
    ref2 = np.array([mid - 2e-7, 3.0001])
    x2 = np.array([mid + 3e-7, 3.0001])
    got2 = bits([hi, hi])                                     # second element: wrong neighbour without a tie
    assert list(H.bf16_tie_flips(got2, bits(ref2), x2, ref2)) == [True, False]
    # identical values are never flips; across zero the ordinals are still adjacent
    assert not H.bf16_tie_flips(bits([1.5]), bits([1.5]), np.array([1.5]), np.array([1.5])).any()
    assert abs(int(H._bf16_ordinal(bits([2.0 ** -126]))[0]) - int(H._bf16_ordinal(bits([0.0]))[0])) >= 1
