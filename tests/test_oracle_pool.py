"""Pins for the oracle's pool level: special pages with closed-form records, idempotence,
placement, address translation, gather and prefetch, status reporting."""
import struct

import numpy as np
import pytest

from kvgen import gen, workloads
from oracle import oracle as O


def _hdr(rec):
    s, plen, mode, ver, n_runs, amax, rsv = struct.unpack_from("<IHBBHHI", rec, 0)
    return dict(s_bits=s, payload_len=plen, mode=mode, version=ver, n_runs=n_runs, amax_bits=amax, reserved=rsv)


def _h(v):
    return np.asarray(v, np.float16).view(np.uint16)


def _pool_for(w, pool_bytes=None):
    return O.Pool(w.n_layers, w.n_kv_heads, w.blocks_per_layer, w.max_blocks_per_seq, w.batch,
                  pool_bytes or w.n_slots * 4160)


# ---------------------------------------------------------------- special pages (closed form)

def test_all_zero_page():
    rec = O.compress_page(np.zeros(2048, np.uint16), 3)
    h = _hdr(rec)
    assert h == dict(s_bits=0, payload_len=257, mode=3, version=1, n_runs=1, amax_bits=0, reserved=0)
    assert len(rec) == 273 and (len(rec) + 63) // 64 == 5
    assert rec[16] == 1 and rec[17:16 + 256] == bytes(255) and rec[16 + 256] == 0
    rc, out = O.decompress_record(rec)
    assert rc == 0 and not out.any()
    assert not O.decompress_record(O.compress_page(_h(np.full(2048, -0.0)), 3))[1].any()   # -0 decodes to +0


@pytest.mark.parametrize("value,qv", [(3.5, 127), (-0.007, -127)])
def test_constant_page(value, qv):
    x = _h(np.full(2048, value))
    st = O.page_stages(x)
    assert np.all(st["q"] == qv)
    sym = st["sym"].reshape(16, 128)
    assert np.all(sym[:, 0] == (qv & 0xFF)) and not sym[:, 1:].any()
    assert st["n_runs"] == 32                                      # (q, 0) per row
    rec = O.compress_page(x, 3)
    assert _hdr(rec)["payload_len"] == 288
    assert np.array_equal(O.decompress_record(rec)[1], x)


def test_row_ramp_has_three_runs_per_row():
    q = np.tile(np.arange(-63, 65), (16, 1))                       # slope 1 in every row, max 64
    q[0, 127] = 127
    st = O.page_stages(_h(q.reshape(-1).astype(np.float64)))
    assert np.array_equal(st["q"].reshape(16, 128), q)
    heads = np.unpackbits(st["bitmap"], bitorder="little").reshape(16, 128)
    assert np.all(heads[1:].sum(axis=1) == 2) and heads[0].sum() == 3


@pytest.mark.parametrize("bad", [np.inf, -np.inf, np.nan])
def test_nonfinite_page_is_stored_raw(bad):
    x = gen.gen_pages(2, [0], np.ones((1, 2, 128), np.float32), 1 << 20, 8)[0].copy()
    x[777] = _h([bad])[0]
    for scheme in (1, 2, 3):
        rec = O.compress_page(x, scheme)
        assert _hdr(rec) == dict(s_bits=0, payload_len=4096, mode=0, version=1, n_runs=0, amax_bits=0, reserved=0)
        assert rec[16:] == x.tobytes() and rec == O.compress_page(x, 0)
        assert np.array_equal(O.decompress_record(rec)[1], x)      # bypass is the identity


def test_extreme_values_and_subnormals():
    x = np.zeros(2048, np.uint16)
    x[0::2], x[1::2] = 0x7BFF, 0xFBFF                              # alternating +-65504
    for scheme in (1, 2, 3):
        assert np.array_equal(O.decompress_record(O.compress_page(x, scheme))[1], x)
    sub = (np.arange(2048) % 1024).astype(np.uint16)               # subnormals, amax = 1023 * 2^-24
    st = O.page_stages(sub)
    want = np.rint(np.arange(2048) % 1024 * (float(st["inv"]) * 2.0 ** -24))
    assert np.array_equal(st["q"].astype(np.float64), want)       # exact products here (powers of two apart)


def test_modes_1_2_3_decode_to_the_same_page():
    w = workloads.tiny()
    for page in w.gen_pages(np.arange(0, 256, 17)):
        outs = [O.decompress_record(O.compress_page(page, m))[1] for m in (1, 2, 3)]
        assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
        assert _hdr(O.compress_page(page, 2))["payload_len"] == 2048


def test_idempotence_compress_of_decompress():
    w = workloads.tiny(seed=4)
    pages = np.concatenate([w.gen_pages(np.arange(40)), gen.structured_pages(1, 8)])
    for page in pages:
        for mode in (1, 2, 3):
            rec = O.compress_page(page, mode)
            rc, xh = O.decompress_record(rec)
            assert rc == 0 and O.compress_page(xh, mode) == rec


def test_corrupt_headers_are_rejected():
    rec = bytearray(O.compress_page(workloads.tiny().gen_pages([5])[0], 3))
    for off, val in [(7, 2), (6, 9), (4, 0), (8, 0)]:
        bad = bytearray(rec)
        bad[off] = val
        assert O.decompress_record(bytes(bad))[0] == O.ST_BAD_RECORD
    bad = bytearray(rec)
    bad[16] &= 0xFE                                                # first symbol must start a run
    assert O.decompress_record(bytes(bad))[0] == O.ST_BAD_RECORD
    assert O.decompress_record(bytes(rec[:100]))[0] == O.ST_BAD_RECORD


# ---------------------------------------------------------------- placement, page table

def test_placement_is_the_prefix_sum_in_list_order():
    w = workloads.tiny(seed=1)
    src = np.concatenate([w.gen_pages(np.arange(200)), gen.structured_pages(2, 56)])
    rng = np.random.default_rng(0)
    order = rng.permutation(256).astype(np.uint32)
    slots = rng.permutation(256).astype(np.uint32)
    pool = _pool_for(w)
    assert pool.compress(src, order[:100], slots[:100], 3) == 0
    assert pool.compress(src, order[100:], slots[100:], 1) == 0
    off = 0
    for i in range(256):
        rec = O.compress_page(src[order[i]], 3 if i < 100 else 1)
        gran = (len(rec) + 63) // 64
        e = int(pool.pte[slots[i]])
        assert e & 0xFFFFFFFF == off and (e >> 32) & 0xFFFF == len(rec) and (e >> 48) & 0xFF == rec[6] and e >> 56 == 1
        assert pool.pool[off * 64:off * 64 + len(rec)].tobytes() == rec
        assert not pool.pool[off * 64 + len(rec):(off + gran) * 64].any()
        off += gran
    assert pool.cursor.value == off == pool.stats.granules
    assert pool.stats.pages_mode[3] == 100 and pool.stats.pages_mode[1] == 156
    assert sum(pool.status.count) == 0


def test_pool_full_and_bad_indices():
    w = workloads.tiny()
    src = w.gen_pages(np.arange(8))
    valid = [0, 1, 3, 4, 5, 6]                                      # source pages that get compressed
    sizes = [(len(O.compress_page(src[p], 3)) + 63) // 64 for p in valid]
    pool = _pool_for(w, pool_bytes=64 * (sum(sizes[:4]) + 3))
    sp = np.array([0, 1, 99, 2, 3, 4, 5, 6], np.uint32)
    ds = np.array([0, 1, 2, 100000, 3, 4, 5, 6], np.uint32)
    pool.compress(src, sp, ds, 3)
    assert pool.status.count[O.ST_BAD_INDEX] == 2 and pool.status.first[O.ST_BAD_INDEX] == 2
    assert pool.status.count[O.ST_POOL_FULL] == 2 and pool.status.first[O.ST_POOL_FULL] == 6
    assert [int(pool.pte[s]) >> 56 for s in range(7)] == [1, 1, 0, 1, 1, 0, 0]
    assert pool.cursor.value == sum(sizes)


# ---------------------------------------------------------------- translate / gather

def _fill(w, scheme=3, order=None, raw_every=0):
    pool = _pool_for(w)
    for layer in range(w.n_layers):
        slots = w.layer_slots(layer)
        if order is not None:
            slots = slots[order(len(slots))]
        src = w.gen_pages(slots)
        if raw_every:
            for i in range(0, len(slots), raw_every):
                pool.compress(src, np.arange(i, min(i + raw_every, len(slots)), dtype=np.uint32), slots[i:i + raw_every],
                              0 if (i // raw_every) % 3 == 0 else scheme)
        else:
            pool.compress(src, np.arange(len(slots), dtype=np.uint32), slots, scheme)
    return pool


def _expected_page(w, slot):
    page = w.gen_pages([slot])[0]
    return O.decompress_record(O.compress_page(page, 3))[1]


def test_translate_brute_force():
    w = workloads.llama70b(seed=3, n_layers=2, batch=3, seq=64)     # 12 blocks, permuted table
    pool = _fill(w)
    va = np.zeros(0, O.VADDR)
    rows = [(b, l, kv, h, pos, 0) for b in range(3) for l in range(2) for kv in range(2) for h in range(8) for pos in (0, 15, 16, 63)]
    va = np.array(rows, O.VADDR)
    pa = pool.translate(w.block_table, va)
    offs = set()
    for r, p in zip(rows, pa):
        b, l, kv, h, pos, _ = r
        phys = w.block_table[b][pos // 16]
        slot = ((l * w.blocks_per_layer + phys) * 2 + kv) * 8 + h
        e = int(pool.pte[slot])
        assert p["status"] == 0 and p["byte_off"] == 64 * (e & 0xFFFFFFFF) and p["rec_len"] == (e >> 32) & 0xFFFF
        assert p["byte_off"] % 64 == 0 and p["byte_off"] + p["rec_len"] <= pool.cursor.value * 64
        offs.add(int(p["byte_off"]))
    assert len(offs) == 3 * 2 * 2 * 8 * 3                          # pos 0 and 15 share a page
    bad = np.array([(3, 0, 0, 0, 0, 0), (0, 0, 0, 0, 64, 0), (0, 2, 0, 0, 0, 0), (0, 0, 0, 8, 0, 0)], O.VADDR)
    assert pool.translate(w.block_table, bad)["status"].tolist() == [O.ST_UNMAPPED] * 4
    bt = w.block_table.copy()
    bt[1, 2] = -1
    assert pool.translate(bt, np.array([(1, 0, 1, 3, 40, 0)], O.VADDR))["status"][0] == O.ST_UNMAPPED
    slot_of = lambda r: ((r[1] * w.blocks_per_layer + w.block_table[r[0]][r[4] // 16]) * 2 + r[2]) * 8 + r[3]
    victim = slot_of(rows[37])
    pool.pte[victim] = 0
    hit = [i for i, r in enumerate(rows) if slot_of(r) == victim]
    assert hit and all(pool.translate(w.block_table, va[hit])["status"] == O.ST_BAD_PTE)


def _gather(w, pool, layer, seq_lens=None, pf=None):
    sl = w.seq_lens if seq_lens is None else seq_lens
    dst = np.full(w.demand_tokens(sl) * 2 * w.n_kv_heads * 128, 0xCDCD, np.uint16)
    l2 = np.full(w.batch * 4 * 2 * w.n_kv_heads * 2048, 0xCDCD, np.uint16)
    assert pool.decompress_gather(layer, w.block_table, sl, w.dst_tok_off(sl), pf, dst, l2) == 0
    return dst, l2


def test_gather_places_every_page_by_the_address_formula():
    w = workloads.llama70b(seed=7, n_layers=2, batch=3, seq=80)     # 5 blocks per sequence
    w.seq_lens = np.array([80, 33, 1], np.uint32)                   # ragged: 5, 3, 1 blocks
    pool = _fill(w)
    H = 8
    for layer in (0, 1):
        dst, _ = _gather(w, pool, layer)
        off = w.dst_tok_off()
        seen = np.zeros(dst.size, bool)
        for b in range(3):
            nblk = (int(w.seq_lens[b]) + 15) // 16
            for n in range(nblk):
                for kv in range(2):
                    for h in range(H):
                        slot = ((layer * w.blocks_per_layer + w.block_table[b][n]) * 2 + kv) * H + h
                        el = int(off[b]) * 2 * H * 128 + ((kv * H + h) * nblk * 16 + 16 * n) * 128
                        assert np.array_equal(dst[el:el + 2048], _expected_page(w, slot))
                        seen[el:el + 2048] = True
        assert seen.all()
    assert pool.stats.pages_decoded == 2 * 9 * 16 and sum(pool.status.count) == 0


def test_gather_is_invariant_under_a_permutation_of_the_physical_pool():
    w = workloads.llama70b(seed=7, n_layers=1, batch=2, seq=64)
    a = _gather(w, _fill(w), 0)[0]
    b = _gather(w, _fill(w, order=lambda n: np.random.default_rng(5).permutation(n)), 0)[0]
    assert np.array_equal(a, b)
    c = _gather(w, _fill(w, raw_every=16), 0)[0]                    # a third of the pages stored raw
    raw_pages = np.count_nonzero(np.any(a.reshape(-1, 2048) != c.reshape(-1, 2048), axis=1))
    assert 0 < raw_pages <= a.size // 2048


def test_prefetch_residency_filter_and_unmapped_blocks():
    w = workloads.decode_fetch(seed=2, n_layers=2, batch=3, steps=4, max_blocks_per_seq=48, len_lo=64, len_hi=512)
    pool = _fill(w)
    H = w.n_kv_heads
    layer, lens, pf = workloads.decode_step(w, 0)
    assert len(pf) >= 3
    dst, l2 = _gather(w, pool, layer, lens, pf)
    assert pool.stats.pf_issued == len(pf) and pool.stats.pf_skipped == 0
    for e in pf:
        for kv in range(2):
            for h in range(H):
                slot = ((layer * w.blocks_per_layer + w.block_table[e["seq"]][e["block"]]) * 2 + kv) * H + h
                el = ((((int(e["seq"]) * 4 + int(e["l2_slot"])) * 2 + kv) * H + h) * 16) * 128
                assert np.array_equal(l2[el:el + 2048], _expected_page(w, slot))
        assert int(pool.l2_tag[int(e["seq"]) * 4 + int(e["l2_slot"])]) == (1 << 32) | (layer * (1 << 20) + int(e["block"]) + 1)
    _, l2b = _gather(w, pool, layer, lens, pf)                      # same list again: everything resident
    assert pool.stats.pf_skipped == len(pf) and np.all(l2b == 0xCDCD)
    pf2 = pf.copy()
    pf2["block"][0] += 1                                            # a different block overwrites the slot
    _gather(w, pool, layer, lens, pf2)
    assert pool.stats.pf_issued == len(pf) + 1
    pf3 = pf[:1].copy()
    pf3["block"][0] = w.max_blocks_per_seq - 1                      # not populated -> unmapped
    before = pool.status.count[O.ST_UNMAPPED]
    _gather(w, pool, layer, lens, pf3)
    assert pool.status.count[O.ST_UNMAPPED] == before + 2 * H


def test_gather_reports_unmapped_and_unwritten_pages_and_leaves_them_untouched():
    w = workloads.llama70b(seed=1, n_layers=1, batch=2, seq=32)
    pool = _fill(w)
    bt = w.block_table.copy()
    bt[1, 0] = -1
    w.block_table = bt
    victim = ((0 * w.blocks_per_layer + bt[0][1]) * 2 + 1) * 8 + 2
    pool.pte[victim] = 0
    dst, _ = _gather(w, pool, 0)
    assert pool.status.count[O.ST_UNMAPPED] == 16 and pool.status.count[O.ST_BAD_PTE] == 1
    pages = dst.reshape(-1, 2048)
    assert np.count_nonzero(np.all(pages == 0xCDCD, axis=1)) == 17
    assert pool.status.first[O.ST_BAD_PTE] == (0 * 2 + 1) * 16 + 8 + 2   # block index 1 of seq 0, V, head 2


# ---------------------------------------------------------------- adaptive scheme

def test_auto_scheme_keeps_the_smaller_of_delta_and_delta_rle():
    w = workloads.tiny(seed=6)
    pages = np.concatenate([w.gen_pages(np.arange(12)), gen.structured_pages(8, 12), np.zeros((1, 2048), np.uint16)])
    modes = set()
    for page in pages:
        r2, r3, ra = O.compress_page(page, 2), O.compress_page(page, 3), O.compress_page(page, 4)
        assert ra == (r3 if len(r3) < len(r2) else r2)                # ties go to the simpler mode
        assert np.array_equal(O.decompress_record(ra)[1], O.decompress_record(r3)[1])
        modes.add(ra[6])
    assert modes == {2, 3}
    # break-even on 1 x 8 pages: run-length coding is kept iff 1 + n_runs < 8 (equal size -> delta stream)
    import itertools
    seen = set()
    for seq in itertools.product([0, 9, -127], repeat=7):
        qv = np.array(seq + (127,), np.int64)
        xb = qv.astype(np.float16).view(np.uint16)
        n_runs = O.page_stages(xb, 1, 8)["n_runs"]
        assert O.compress_page(xb, 4, 1, 8)[6] == (3 if n_runs < 7 else 2)
        seen.add(n_runs)
    assert {6, 7, 8} <= seen
    nan = gen.gen_pages(1, [0], np.ones((1, 2, 128), np.float32), 1 << 20, 8)[0].copy(); nan[5] = 0x7E00
    assert O.compress_page(nan, 4)[6] == 0                          # non-finite pages still bypass


# ---------------------------------------------------------------- pool lifecycle: rewrites and compaction

def test_tail_page_rewrites_then_compaction_keeps_exactly_the_live_records():
    """A decode loop rewrites each sequence's tail page as it fills (16 versions of one slot); the log
    keeps every version, the page table only the newest; compaction drops the rest."""
    rng = np.random.default_rng(5)
    H, nblk = 2, 3
    pool = O.Pool(1, H, nblk, nblk, 1, 1 << 20)
    full = gen.gen_pages(3, np.arange(nblk * 2 * H), np.ones((1, 2, 128), np.float32), nblk * 2 * H, H)
    slots = np.arange(nblk * 2 * H, dtype=np.uint32)
    pool.compress(full[:2 * 2 * H], np.arange(2 * 2 * H), slots[:2 * 2 * H], 3)            # two complete blocks
    tail_slots = slots[2 * 2 * H:]
    for t in range(1, 17):                                                                 # block 2 fills token by token
        tail = full[2 * 2 * H:].copy().reshape(-1, 16, 128)
        tail[:, t:, :] = 0
        pool.compress(tail.reshape(-1, 2048), np.arange(2 * H), tail_slots, 3)
    before_cursor = pool.cursor.value
    live = {}
    for s in slots:
        e = int(pool.pte[s]); off, ln = (e & 0xFFFFFFFF) * 64, (e >> 32) & 0xFFFF
        live[int(s)] = bytes(pool.pool[off:off + (ln + 63) // 64 * 64])
    # the newest version is the complete page
    for s in tail_slots:
        assert live[int(s)][:len(O.compress_page(full[s], 3))] == O.compress_page(full[s], 3)
    want_gran = sum(len(r) // 64 for r in live.values())
    assert before_cursor > want_gran + 15 * 2 * H * 4                                       # the log holds the old versions too
    d0 = np.zeros(48 * 2 * H * 128, np.uint16); l2 = np.zeros(4 * 2 * H * 2048, np.uint16)
    bt = np.arange(nblk, dtype=np.int32).reshape(1, -1)
    pool.decompress_gather(0, bt, [48], [0], None, d0, l2)
    assert pool.compact() == 0
    assert pool.cursor.value == want_gran
    at = 0
    for s in slots:                                                                        # slot order, back to back
        e = int(pool.pte[s])
        assert (e & 0xFFFFFFFF) == at and (e >> 56) & 1 and bytes(pool.pool[at * 64:at * 64 + len(live[int(s)])]) == live[int(s)]
        at += len(live[int(s)]) // 64
    d1 = np.zeros_like(d0)
    pool.decompress_gather(0, bt, [48], [0], None, d1, l2)
    assert np.array_equal(d0, d1) and sum(pool.status_dict()["count"]) == 0
    assert pool.compact() == 0 and pool.cursor.value == want_gran                           # idempotent


def test_compaction_reorders_to_slot_order_and_clears_entries_outside_the_pool():
    pool = O.Pool(1, 1, 8, 8, 1, 64 * 400)
    src = gen.structured_pages(6, 16)
    order = np.array([5, 1, 7, 3, 0, 2, 6, 4, 9, 8], np.uint32)                             # log order != slot order
    pool.compress(src, np.arange(10), order, 4)
    recs = {int(s): bytes(pool.pool[(int(pool.pte[s]) & 0xFFFFFFFF) * 64:][:((int(pool.pte[s]) >> 32) & 0xFFFF)]) for s in order}
    pool.pte[12] = (399) | (4112 << 32) | (1 << 56)                                         # would end beyond the pool
    pool.pte[13] = (0) | (8 << 32) | (1 << 56)                                              # shorter than a header
    pool.clear_status()
    assert pool.compact() == 0
    st = pool.status_dict()
    assert st["count"][O.ST_BAD_RECORD] == 2 and st["first"][O.ST_BAD_RECORD] == 12 and pool.pte[12] == 0 and pool.pte[13] == 0
    at = 0
    for s in sorted(recs):
        e = int(pool.pte[s])
        assert (e & 0xFFFFFFFF) == at and bytes(pool.pool[at * 64:at * 64 + len(recs[s])]) == recs[s]
        at += (len(recs[s]) + 63) // 64
    assert pool.cursor.value == at


def test_compaction_with_entries_that_share_records_in_a_pool_too_small_for_the_copies():
    """Entries may share a record (nothing forbids two slots pointing at one copy); compaction gives every
    entry a copy of its own, so the kept total can exceed the pool.  Worked by hand: a 12-granule pool, an
    all-zero page (273 B -> 5 granules) in slot 0 and a constant page (304 B -> 5 granules) in slot 2, then
    slot 1 shares slot 0's record and slot 3 shares slot 2's.  In slot order: slot 0 -> granules 0-4,
    slot 1 -> 5-9, slot 2 would need 10-14 > 12: reported, cleared, and the count still advances to 15 (the
    cursor rule of the compressor); slot 3 likewise at 15-19.  Cursor 20."""
    pool = O.Pool(1, 1, 4, 4, 1, 64 * 12)
    zero, const = np.zeros(2048, np.uint16), _h(np.full(2048, 3.5))
    pool.compress(np.stack([zero, const]), [0, 1], [0, 2], 3)
    assert pool.cursor.value == 10
    rec0, rec2 = O.compress_page(zero, 3), O.compress_page(const, 3)
    assert (len(rec0), len(rec2)) == (273, 304)
    pool.pte[1], pool.pte[3] = pool.pte[0], pool.pte[2]
    pool.clear_status()
    assert pool.compact() == 0
    valid = 1 << 56
    assert [int(e) for e in pool.pte[:4]] == [0 | (273 << 32) | (3 << 48) | valid, 5 | (273 << 32) | (3 << 48) | valid, 0, 0]
    assert not pool.pte[4:].any()
    assert pool.cursor.value == 20
    st = pool.status_dict()
    assert st["count"][O.ST_POOL_FULL] == 2 and st["first"][O.ST_POOL_FULL] == 2
    assert sum(st["count"]) == 2
    for at in (0, 5):                                               # both copies complete, with their zero padding
        assert bytes(pool.pool[at * 64:at * 64 + 320]) == rec0 + bytes(320 - 273)
    # a pool with room for three copies keeps three, in slot order
    pool = O.Pool(1, 1, 4, 4, 1, 64 * 15)
    pool.compress(np.stack([zero, const]), [0, 1], [0, 2], 3)
    pool.pte[1], pool.pte[3] = pool.pte[0], pool.pte[2]
    assert pool.compact() == 0
    assert [int(e) & 0xFFFFFFFF for e in pool.pte[:3]] == [0, 5, 10] and pool.pte[3] == 0 and pool.cursor.value == 20
    assert bytes(pool.pool[10 * 64:10 * 64 + 320]) == rec2 + bytes(320 - 304)
    assert pool.status_dict()["first"][O.ST_POOL_FULL] == 3


def test_gather_skips_a_sequence_whose_rows_pass_the_destination_capacity():
    """Three sequences of 3, 2 and 1 blocks; the destination holds 64 token rows, the second sequence is
    placed at row 48 (48 + 32 > 64).  All 2 blocks x 2 x H pages of that sequence are reported with the index
    of its first page = the 3*2*H pages of sequence 0, nothing of it is written, the others are delivered."""
    w = workloads.llama70b(seed=4, n_layers=1, batch=3, seq=48)
    w.seq_lens = np.array([48, 20, 5], np.uint32)
    pool = _fill(w)
    H = w.n_kv_heads
    tok = np.array([0, 48, 16 + 32], np.uint64)                     # sequence 2 shares rows 48.. with the skipped one
    dst = np.full(64 * 2 * H * 128, 0xCDCD, np.uint16)
    l2 = np.zeros(w.batch * 4 * 2 * H * 2048, np.uint16)
    assert pool.decompress_gather(0, w.block_table, w.seq_lens, tok, None, dst, l2) == 0
    st = pool.status_dict()
    assert st["count"][O.ST_BAD_DST] == 2 * 2 * H and st["first"][O.ST_BAD_DST] == 3 * 2 * H
    assert sum(st["count"]) == 2 * 2 * H and pool.stats.pages_decoded == (3 + 1) * 2 * H
    rows = dst.reshape(64, 2 * H * 128)
    for kv in range(2):                                            # sequence 0: rows 0-47 as [K|V][head][48][128]
        for h in range(H):
            for n in range(3):
                slot = ((0 * w.blocks_per_layer + w.block_table[0][n]) * 2 + kv) * H + h
                el = ((kv * H + h) * 48 + 16 * n) * 128
                assert np.array_equal(dst[el:el + 2048], _expected_page(w, slot))
    for kv in range(2):                                            # sequence 2: one block at row 48
        for h in range(H):
            slot = ((0 * w.blocks_per_layer + w.block_table[2][0]) * 2 + kv) * H + h
            el = 48 * 2 * H * 128 + (kv * H + h) * 16 * 128
            assert np.array_equal(dst[el:el + 2048], _expected_page(w, slot))
    assert np.all(rows[48 + 16:] == 0xCDCD)                        # nothing of the skipped sequence was written
    # exactly at capacity is accepted
    pool.clear_status()
    dst2 = np.full(80 * 2 * H * 128, 0xCDCD, np.uint16)
    assert pool.decompress_gather(0, w.block_table, w.seq_lens[:2], np.array([0, 48], np.uint64), None, dst2, l2) == 0
    assert sum(pool.status_dict()["count"]) == 0 and not np.any(np.all(dst2.reshape(-1, 2048) == 0xCDCD, axis=1))


def test_free_slots_clears_entries_and_counts_what_compaction_will_reclaim():
    """Worked by hand: an all-zero page (5 granules) in slot 0, a constant page (5) in slot 2, a raw page (65) in
    slot 5.  Freeing [2, 7, 2, 99, 5]: slot 2 once (5 granules), slot 7 was empty, 99 is beyond the 8 slots
    (reported at list position 3), slot 5 (65 granules) -> 2 entries, 70 granules; compaction then keeps
    slot 0 alone."""
    pool = O.Pool(1, 1, 4, 4, 1, 64 * 200)
    zero, const = np.zeros(2048, np.uint16), _h(np.full(2048, 3.5))
    pool.compress(np.stack([zero, const]), [0, 1], [0, 2], 3)
    pool.compress(np.stack([const]), [0], [5], 0)
    assert pool.cursor.value == 75
    assert pool.free_slots([2, 7, 2, 99, 5]) == [2, 70]
    st = pool.status_dict()
    assert st["count"][O.ST_BAD_INDEX] == 1 and st["first"][O.ST_BAD_INDEX] == 3 and sum(st["count"]) == 1
    assert [bool(e >> 56 & 1) for e in pool.pte] == [True] + [False] * 7
    assert pool.cursor.value == 75                                  # the log itself is untouched
    assert pool.compact() == 0 and pool.cursor.value == 5
    assert pool.free_slots([0, 0]) == [1, 5] and not pool.pte.any()
    assert pool.compact() == 0 and pool.cursor.value == 0


def test_a_sequence_longer_than_the_block_table_is_reported_once_and_left_out():
    """Block table 6 wide; lengths 48, 16*6 + 1 (seven blocks: one too many) and 5.  The long sequence is reported
    once as unmapped, at the index its first page would have had (3 blocks * 2 * H), and takes no place in the
    numbering: the third sequence's missing page is numbered right behind the first sequence's pages."""
    w = workloads.llama70b(seed=4, n_layers=1, batch=3, seq=96)
    assert w.max_blocks_per_seq == 6
    pool = _fill(w)
    H = w.n_kv_heads
    lens = np.array([48, 97, 5], np.uint32)
    victim = ((0 * w.blocks_per_layer + w.block_table[2][0]) * 2 + 1) * H + 3          # V page, head 3, of the third sequence
    pool.pte[victim] = 0
    dst = np.full(64 * 2 * H * 128, 0xCDCD, np.uint16)
    l2 = np.zeros(w.batch * 4 * 2 * H * 2048, np.uint16)
    assert pool.decompress_gather(0, w.block_table, lens, np.array([0, 48, 48], np.uint64), None, dst, l2) == 0
    st = pool.status_dict()
    assert st["count"][O.ST_UNMAPPED] == 1 and st["first"][O.ST_UNMAPPED] == 3 * 2 * H
    assert st["count"][O.ST_BAD_PTE] == 1 and st["first"][O.ST_BAD_PTE] == 3 * 2 * H + H + 3
    assert pool.stats.pages_decoded == 4 * 2 * H - 1
    el = 48 * 2 * H * 128                                                               # the third sequence sits at row 48
    slot = ((0 * w.blocks_per_layer + w.block_table[2][0]) * 2 + 0) * H + 0
    assert np.array_equal(dst[el:el + 2048], _expected_page(w, slot))
    # exactly as wide as the table is fine; an absurd length is the same single report
    pool.clear_status()
    big = np.full(112 * 2 * H * 128, 0xCDCD, np.uint16)
    assert pool.decompress_gather(0, w.block_table, np.array([96, 0xFFFFFFFF], np.uint32), np.array([0, 96], np.uint64), None, big, l2) == 0
    st = pool.status_dict()
    assert st["count"][O.ST_UNMAPPED] == 1 and st["first"][O.ST_UNMAPPED] == 6 * 2 * H and sum(st["count"]) == 1
    # the attention reading of the same rule: zero rows for the sequence that is left out
    q = np.random.default_rng(0).standard_normal((2, H, 128)).astype(np.float16)
    pool.clear_status()
    out = pool.attend(0, w.block_table, np.array([97, 48], np.uint32), q.view(np.uint16), H)
    assert not out[0].any() and out[1].any()
    st = pool.status_dict()
    assert st["count"][O.ST_UNMAPPED] == 1 and st["first"][O.ST_UNMAPPED] == 0 and sum(st["count"]) == 1
