"""Pins for the CPU oracle's page codec: each check compares the oracle with something that
is not the oracle (numpy's binary16, exact rational arithmetic, exhaustive enumeration, a
hand-worked page, values printed in the paper)."""
import itertools
import os
import struct
from fractions import Fraction

import numpy as np
import pytest

from kvgen import gen
from oracle import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            k, *v = line.split()
            out[k] = v
    return out


def _hdr(rec):
    s, plen, mode, ver, n_runs, amax, rsv = struct.unpack_from("<IHBBHHI", rec, 0)
    return dict(s_bits=s, payload_len=plen, mode=mode, version=ver, n_runs=n_runs, amax_bits=amax, reserved=rsv)


def _f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16).astype(np.float64)


# ---------------------------------------------------------------- binary16 conversions

def test_half_to_float_exhaustive_vs_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    got = np.array([O.half_to_float(int(b)) for b in bits], np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_float_to_half_round_trip_and_midpoints():
    finite = [b for b in range(0x7C00)]
    vals = _f16(finite)
    for b in range(0, 65536, 1):  # every pattern converts back to itself
        f = np.uint16(b).view(np.float16).astype(np.float32)
        if not np.isnan(f):
            assert O.float_to_half(f) == b
    for lo in range(0x7BFF):  # exact midpoints go to the even neighbour, just off them to the nearer
        a, c = vals[lo], vals[lo + 1]
        mid = np.float32((a + c) / 2.0)
        assert float(mid) == (a + c) / 2.0
        even = lo if lo % 2 == 0 else lo + 1
        assert O.float_to_half(mid) == even
        assert O.float_to_half(np.nextafter(mid, np.float32(0))) == lo
        assert O.float_to_half(np.nextafter(mid, np.float32(np.inf))) == lo + 1
        assert O.float_to_half(-mid) == (even | 0x8000)
    assert O.float_to_half(np.float32(65519.99)) == 0x7BFF
    assert O.float_to_half(np.float32(65520.0)) == 0x7C00  # tie between 65504 and 2^16 -> Inf
    assert O.float_to_half(np.float32(2.0 ** -25)) == 0     # tie between 0 and 2^-24 -> 0
    assert O.float_to_half(np.nextafter(np.float32(2.0 ** -25), np.float32(1))) == 1


def test_float_to_half_random_vs_numpy():
    rng = np.random.default_rng(1)
    f = np.concatenate([rng.standard_normal(20000).astype(np.float32) * np.float32(10.0) ** rng.integers(-9, 6, 20000),
                        rng.integers(0, 2 ** 32, 20000, dtype=np.uint64).astype(np.uint32).view(np.float32)])
    f = f.astype(np.float32)
    f = f[~np.isnan(f)]
    with np.errstate(over="ignore"):
        ref = f.astype(np.float16).view(np.uint16)
    got = np.array([O.float_to_half(v) for v in f], np.uint16)
    assert np.array_equal(got, ref)


# ---------------------------------------------------------------- hand-worked page, paper constants

def test_hand_worked_page():
    g = _gold("worked_page_1x8.txt")
    x = np.array([int(v, 16) for v in g["x_bits"]], np.uint16)
    st = O.page_stages(x, 1, 8)
    assert st["q"].tolist() == [int(v) for v in g["q"]]
    assert st["sym"].tolist() == [int(v, 16) for v in g["sym"]]
    rec = O.compress_page(x, 3, 1, 8)
    assert rec == bytes(int(v, 16) for v in g["record"])
    rc, out = O.decompress_record(rec, 1, 8)
    assert rc == 0 and out.tolist() == [int(v, 16) for v in g["xhat"]]


def test_paper_constants():
    g = _gold("paper_constants.txt")
    x = gen.gen_pages(0, [3], np.ones((1, 2, 128), np.float32), 1 << 20, 8)[0]
    rec = O.compress_page(x, 1)
    h = _hdr(rec)
    assert O.PAGE_ELEMS * 2 == int(g["page_bytes"][0])
    assert O.PAGE_ELEMS * 2 / h["payload_len"] == float(g["int8_only_ratio"][0])  # INT8 only: 2.00x
    assert O.GRANULE * 8 == int(g["beat_bits"][0])


# ---------------------------------------------------------------- quantiser

def _exact_q(x_bits, amax_bits):
    """round-half-even(x * fl32(127/amax)) in exact rational arithmetic."""
    amax = np.uint16(amax_bits).view(np.float16).astype(np.float32)
    inv = Fraction(float(np.float32(127.0) / amax))
    out = []
    for b in x_bits:
        p = Fraction(float(np.uint16(b).view(np.float16))) * inv
        out.append(max(-127, min(127, round(p))))  # Python's round on Fraction: ties to even
    return out


@pytest.mark.parametrize("amax_bits", [0x3C00, 0x4500, 0x5140, 0x7BFF, 0x0001, 0x03FF, 0x0400, 0x2E66, 0x3555])
def test_quantiser_matches_exact_rounding_for_every_input(amax_bits):
    below = np.array([b for b in range(amax_bits + 1)], np.uint16)
    rng = np.random.default_rng(amax_bits)
    if below.size > 2047:
        pick = np.concatenate([rng.choice(below[:-1], 2046, replace=False), [amax_bits]])
    else:
        pick = np.concatenate([below, np.zeros(2047 - below.size, np.uint16)])
    pick = pick.astype(np.uint16)
    pick[::2] |= 0x8000  # both signs
    page = np.concatenate([pick, [amax_bits]]).astype(np.uint16)[:2048]
    page[-1] = amax_bits
    st = O.page_stages(page)
    assert st["amax_bits"] == amax_bits
    amax = np.uint16(amax_bits).view(np.float16).astype(np.float32)
    assert st["s"].view(np.uint32) == (amax / np.float32(127.0)).view(np.uint32)
    assert st["inv"].view(np.uint32) == (np.float32(127.0) / amax).view(np.uint32)
    assert st["q"].tolist() == _exact_q(page, amax_bits)
    assert np.abs(st["q"].astype(int)).max() == 127


def test_quantiser_error_bound_and_extremes():
    w_scales = gen.channel_scales(5, 1, "fixed4")
    x = gen.gen_pages(5, np.arange(16), w_scales, 1 << 20, 8)
    for page in x:
        st = O.page_stages(page)
        rec = O.compress_page(page, 3)
        rc, xh = O.decompress_record(rec)
        assert rc == 0
        xv, xhv, s = _f16(page), _f16(xh), float(st["s"])
        amax = float(np.uint16(st["amax_bits"]).view(np.float16))
        ulp = np.maximum(2.0 ** (np.floor(np.log2(np.maximum(np.abs(xhv), 2.0 ** -14))) - 10), 2.0 ** -24)
        assert np.all(np.abs(xv - xhv) <= s / 2 + ulp / 2 + s * 2.0 ** -20)
        top = np.abs(xv) == amax
        assert top.any() and np.array_equal(xhv[top], xv[top])      # +-amax is reproduced exactly
        assert np.all(np.abs(st["q"][top].astype(int)) == 127)
        assert np.abs(st["q"].astype(int)).max() <= 127


# ---------------------------------------------------------------- delta

def test_delta_exhaustive_pairs():
    """All 256 x 256 (previous, current) byte pairs: the wrapped running sum of the symbols is q.
    Values are fed through pages whose quantised values are exactly the chosen integers."""
    vals = np.arange(-127, 128)
    pairs = np.array(list(itertools.product(vals, vals)), np.int64)      # 65025 pairs, q in [-127,127]
    flat = pairs.reshape(-1)
    for start in range(0, flat.size, 2046):                               # pairs never straddle a row
        chunk = flat[start:start + 2046]
        qwant = np.zeros(2048, np.int64)
        qwant[:chunk.size] = chunk
        qwant[-1] = 127                                                   # pins amax = 127 -> q = x
        x = qwant.astype(np.float16).view(np.uint16)
        st = O.page_stages(x)
        assert np.array_equal(st["q"].astype(np.int64), qwant)
        q2 = qwant.reshape(16, 128)
        want = np.empty_like(q2)
        want[:, 0] = q2[:, 0]
        want[:, 1:] = q2[:, 1:] - q2[:, :-1]
        assert np.array_equal(st["sym"].reshape(16, 128), (want & 0xFF).astype(np.uint8))
        back = (np.cumsum(st["sym"].reshape(16, 128).astype(np.int64), axis=1) & 0xFF).astype(np.uint8).view(np.int8)
        assert np.array_equal(back.astype(np.int64), q2)


# ---------------------------------------------------------------- run-length coding

def _py_rle_decode(bitmap, values, n):
    out, r = [], -1
    for k in range(n):
        if (bitmap[k >> 3] >> (k & 7)) & 1:
            r += 1
        out.append(values[r])
    return out


def test_rle_brute_force_all_short_sequences():
    """Every length-8 sequence over 3 quantised levels, as a 1 x 8 page."""
    levels = [0, 5, -127]
    for seq in itertools.product(levels, repeat=8):
        q = np.array(seq, np.int64)
        if not (np.abs(q) == 127).any():
            q = q.copy()
            q[7] = 127
        x = q.astype(np.float16).view(np.uint16)
        st = O.page_stages(x, 1, 8)
        assert st["q"].tolist() == q.tolist()
        sym = st["sym"].tolist()
        n_runs = 1 + sum(sym[k] != sym[k - 1] for k in range(1, 8))
        assert st["n_runs"] == n_runs == bin(int(st["bitmap"][0])).count("1")
        assert st["bitmap"][0] & 1
        assert _py_rle_decode(st["bitmap"], st["values"], 8) == sym
        rec = O.compress_page(x, 3, 1, 8)
        assert len(rec) == 16 + 1 + n_runs
        rc, xh = O.decompress_record(rec, 1, 8)
        assert rc == 0 and np.array_equal(xh, x)      # integers <= 127 with amax 127: lossless


def test_rle_random_streams_and_payload_bounds():
    x = np.concatenate([gen.structured_pages(3, 24), gen.gen_pages(9, np.arange(8), np.ones((1, 2, 128), np.float32), 1 << 20, 8)])
    for page in x:
        st = O.page_stages(page)
        sym = st["sym"]
        heads = np.concatenate([[True], sym[1:] != sym[:-1]])
        assert st["n_runs"] == int(heads.sum())
        assert np.array_equal(np.unpackbits(st["bitmap"], bitorder="little").astype(bool), heads)
        assert np.array_equal(st["values"], sym[heads])
        assert _py_rle_decode(st["bitmap"], st["values"], 2048) == sym.tolist()
        h = _hdr(O.compress_page(page, 3))
        assert 257 <= h["payload_len"] == 256 + st["n_runs"] <= 2304


def test_structured_pages_reach_the_papers_ratio_range():
    x = gen.structured_pages(11, 64)
    tot = sum(64 * ((len(O.compress_page(p, 3)) + 63) // 64) for p in x)
    assert 2.5 <= 64 * 4096 / tot <= 4.5


def test_piecewise_linear_pages_are_stored_losslessly_at_the_papers_rle_ratio():
    """kvgen's piecewise-linear pages are u/128 with integer |u| <= 127 and 127 present: the scale is exactly
    1/128, the quantised bytes are the u themselves (checked from the generator's own definition, not from the
    codec), the delta symbols are the slopes, and the round trip returns the input bit for bit.  The run-length
    records land at the paper's ratio for that stage (3.21x) within a few percent."""
    x = gen.runs_pages(7, np.arange(96))
    u = x.view(np.float16).astype(np.float64) * 128.0
    assert np.array_equal(u, np.rint(u)) and np.abs(u).max(axis=1).tolist() == [127.0] * 96
    d = np.diff(u.reshape(96, 16, 128), axis=2)
    assert np.abs(d).max() <= 2
    tot = 0
    for p, up in zip(x, u):
        rec = O.compress_page(p, 4)                                   # adaptive: must keep the run-length stage
        h = _hdr(rec)
        assert h["mode"] == 3 and h["s_bits"] == 0x3C000000               # 1/128
        tot += 64 * ((len(rec) + 63) // 64)
        rc, back = O.decompress_record(rec)
        assert rc == 0 and np.array_equal(back, p)
        st = O.page_stages(p)
        assert np.array_equal(st["q"].astype(np.int64), up.astype(np.int64))
    assert 3.0 <= 96 * 4096 / tot <= 3.4
