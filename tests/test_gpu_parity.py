"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

Bars: compressed bytestream, page table, cursor, translated addresses, prefetch tags, status
and counters bit-exact; decompressed fp16 within 1 ulp (bit-exact is what is asserted, since
both sides take the same IEEE steps: exact-product rounding, binary32 multiply, RN to binary16).
"""
import numpy as np
import pytest

from kvgen import gen, workloads
from oracle import oracle as O
from tests.parity_util import Pair

pytestmark = pytest.mark.gpu


def _h(v):
    return np.asarray(v, np.float16).view(np.uint16)


def _special_pages():
    rng = np.random.default_rng(0)
    pages = [np.zeros(2048, np.uint16), _h(np.full(2048, -0.0)), _h(np.full(2048, 3.5)), _h(np.full(2048, -0.007))]
    alt = np.zeros(2048, np.uint16); alt[0::2], alt[1::2] = 0x7BFF, 0xFBFF
    pages.append(alt)
    pages.append((np.arange(2048) % 1024).astype(np.uint16))                     # subnormals only
    spike = np.zeros(2048, np.uint16); spike[1234] = 0x7BFF
    pages.append(spike)
    one = np.zeros(2048, np.uint16); one[0] = 0x0001
    pages.append(one)
    q = np.tile(np.arange(-63, 65), (16, 1)).astype(np.float64); q[0, 127] = 127
    pages.append(_h(q.reshape(-1)))
    base = gen.gen_pages(1, [0], np.ones((1, 2, 128), np.float32), 1 << 20, 8)[0]
    for bad in (0x7C00, 0xFC00, 0x7E00, 0xFFFF, 0x7C01):                           # Inf, -Inf, NaNs
        p = base.copy(); p[int(rng.integers(2048))] = bad
        pages.append(p)
    ties = _h((rng.integers(-254, 255, 2048) / 2.0) / 127.0 * 1.0)               # many values near .5 ties
    ties[7] = _h([1.0])[0]
    pages.append(ties)
    pages.extend(gen.structured_pages(4, 7))
    return np.stack(pages)


@pytest.mark.parametrize("scheme", [3, 1, 2, 0, 4, 19, 17, 18, 20, 16])      # 16 = one scale per channel group
def test_tiny_round_trip(scheme):
    w = workloads.tiny(seed=0)
    pr = Pair.for_workload(w, pool_bytes=256 * 4160)
    slots = w.layer_slots(0)
    pr.compress(w.gen_pages(slots), np.arange(256), slots, scheme)
    pr.check_state()
    pr.gather(0, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    assert pr.gpu.stats()["pages_decoded"] == 256 and sum(pr.gpu.status()["count"]) == 0
    pr.close()


@pytest.mark.parametrize("scheme", [3, 1, 2, 4, 19, 17, 18, 20])
def test_special_pages_and_ragged_tiles(scheme):
    src = _special_pages()
    n = len(src)                                                                 # not a multiple of the tile
    pr = Pair(1, 1, 64, 64, 1, 64 * 4160)
    rng = np.random.default_rng(scheme)
    order = rng.permutation(n)
    slots = rng.permutation(128)[:n]
    pr.compress(src, order, slots, scheme)
    pr.check_state()
    assert pr.gpu.stats()["nonfinite"] == 5
    # a second and a third call append behind the cursor (1 page, then an odd count)
    pr.compress(src, [3], [slots[0]], scheme)
    pr.compress(src, order[:13], (slots[:13] + 1) % 128, 3)
    pr.check_state()
    bt = np.full((1, 64), -1, np.int32)
    blocks = np.nonzero(pr.cpu.pte.reshape(64, 2)[:, 0] >> 56)[0]                 # blocks whose K page exists
    bt[0, :len(blocks)] = blocks
    pr.gather(0, bt, [16 * len(blocks)], [0])                                    # V pages partly missing -> BAD_PTE
    pr.check_state()
    pr.close()


def test_empty_calls_and_argument_errors():
    import torch
    from paper_2512_11920_b200 import SpeckvError
    pr = Pair(1, 2, 4, 4, 2, 64 * 100)
    e32 = torch.zeros(0, dtype=torch.int32, device="cuda")
    pr.gpu.compress(torch.zeros(2048, dtype=torch.float16, device="cuda"), e32, e32, 3)      # n = 0
    pr.gpu.decompress_gather(0, pr.t(np.zeros((2, 4), np.int32)), None, None, None)           # B = 0, n_pf = 0
    pr.gather(0, np.zeros((2, 4), np.int32), [0, 0], [0, 0], cap_tokens=16)                   # zero-length sequences
    pr.check_state()
    assert pr.gpu.cursor() == 0
    for bad_scheme in (7, 5 | 16, 3 | 32, -1):
        with pytest.raises(SpeckvError):
            pr.gpu.compress(torch.zeros(2048, dtype=torch.float16, device="cuda"), e32, e32, bad_scheme)
    with pytest.raises(SpeckvError):
        pr.gpu.decompress_gather(5, pr.t(np.zeros((2, 4), np.int32)), None, None, None)
    # host-side checks only, nothing is launched: misaligned index lists, a list longer than the context has slots
    src = torch.zeros(2048, dtype=torch.float16, device="cuda")
    lib, two = pr.gpu._lib, torch.zeros(4, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert lib.speckv_compress(pr.gpu._h, src.data_ptr(), 1, two.data_ptr() + 2, two.data_ptr(), 2, 3, st) == -1
    assert lib.speckv_compress(pr.gpu._h, src.data_ptr(), 1, two.data_ptr(), two.data_ptr() + 1, 2, 3, st) == -1
    long = torch.zeros(pr.gpu.n_slots + 64, dtype=torch.int32, device="cuda")
    with pytest.raises(SpeckvError, match="too many pages"):
        pr.gpu.compress(src, long, long, 3)
    pool = torch.zeros(64 * 100, dtype=torch.uint8, device="cuda")
    ctl = torch.zeros(168, dtype=torch.uint8, device="cuda")
    pte = torch.zeros(17, dtype=torch.int64, device="cuda")
    args = lambda pte_p, ctl_p, sp=two.data_ptr(), ds=two.data_ptr(): (
        src.data_ptr(), 1, sp, ds, 2, 3, pool.data_ptr(), pool.numel(), pte_p, 16, ctl_p, st)
    assert lib.speckv_compress_static(*args(pte.data_ptr(), ctl.data_ptr() + 4)) == -1          # control block at an odd address
    assert lib.speckv_compress_static(*args(pte.data_ptr() + 4, ctl.data_ptr())) == -1          # page table at an odd address
    assert lib.speckv_compress_static(*args(pte.data_ptr(), ctl.data_ptr(), sp=two.data_ptr() + 2)) == -1
    assert lib.speckv_compress_static(*args(pte.data_ptr(), ctl.data_ptr(), ds=two.data_ptr() + 1)) == -1
    torch.cuda.synchronize()
    assert pr.gpu.cursor() == 0 and sum(pr.gpu.status()["count"]) == 0
    pr.close()


def test_pool_full_and_bad_indices():
    w = workloads.tiny(seed=3)
    src = w.gen_pages(np.arange(40))
    sizes = [(len(O.compress_page(p, 3)) + 63) // 64 for p in src]
    pr = Pair.for_workload(w, pool_bytes=64 * (sum(sizes[:29]) + 5))
    sp = np.arange(40).astype(np.uint32); ds = np.arange(40).astype(np.uint32)
    sp[11] = 4000; ds[17] = 1 << 30
    pr.compress(src, sp, ds, 3)
    pr.check_state()
    st = pr.gpu.status()
    assert st["count"][O.ST_BAD_INDEX] == 2 and st["count"][O.ST_POOL_FULL] > 0
    pr.compress(src, [0, 1], [50, 51], 1)                                         # everything after is full too
    pr.check_state()
    pr.close()


def test_many_tiles_chained_scan_and_permuted_block_table():
    w = workloads.llama70b(seed=2, n_layers=3, batch=4, seq=448)                  # 112 blocks, 1792 pages per layer
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 3008)
    rng = np.random.default_rng(1)
    for layer in range(w.n_layers):
        slots = w.layer_slots(layer)
        src = w.gen_pages(slots)
        if layer == 1:                                                            # list order != memory order
            order = rng.permutation(len(slots))
            pr.compress(src, order, slots[order], 3)
        elif layer == 2:                                                          # mixed pool: a third raw
            third = len(slots) // 3
            pr.compress(src, np.arange(third), slots[:third], 0)
            pr.compress(src, np.arange(third, len(slots)), slots[third:], 3)
        else:
            pr.compress(src, np.arange(len(slots)), slots, 3)
    pr.check_state()
    lens = np.array([448, 17, 300, 1], np.uint32)
    for layer in range(w.n_layers):
        pr.gather(layer, w.block_table, lens, w.dst_tok_off(lens))
    pr.gather(0, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    pr.close()


def test_translate_matches_oracle():
    w = workloads.llama70b(seed=3, n_layers=2, batch=3, seq=64)
    pr = Pair.for_workload(w)
    for layer in range(2):
        slots = w.layer_slots(layer)
        pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3 if layer else 1)
    rows = [(b, l, kv, h, pos, 0) for b in range(4) for l in range(3) for kv in range(2) for h in (0, 7, 8) for pos in (0, 15, 16, 63, 64)]
    bt = w.block_table.copy(); bt[1, 2] = -1; bt[2, 0] = 4096
    victim = (int(bt[0, 0]) * 2 + 1) * 8 + 7                                      # layer 0, seq 0, block 0, V, head 7
    pr.cpu.pte[victim] = 0
    pte = pr.gpu.pte_view().view(pr.torch.int64); pte[victim] = 0
    pa = pr.translate(bt, np.array(rows, O.VADDR))
    assert (pa["status"] == 0).sum() > 50 and (pa["status"] == O.ST_UNMAPPED).sum() > 50 and (pa["status"] == O.ST_BAD_PTE).sum() >= 1
    pr.check_state()
    pr.close()


def test_decode_steps_with_prefetch_and_injected_faults():
    w = workloads.decode_fetch(seed=5, n_layers=3, batch=5, steps=7, max_blocks_per_seq=40, len_lo=40, len_hi=500)
    pr = Pair.for_workload(w)
    for layer in range(w.n_layers):
        slots = w.layer_slots(layer)
        pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3)
    for step in range(w.steps):
        layer, lens, pf = workloads.decode_step(w, step)
        pr.gather(layer, w.block_table, lens, w.dst_tok_off(lens), pf)
    layer, lens, pf = workloads.decode_step(w, 3)                                 # same layer as step 0 and 6: tags from step 6
    pr.gather(layer, w.block_table, lens, w.dst_tok_off(lens), pf)
    pr.check_state()
    assert pr.gpu.stats()["pf_skipped"] > 0 and pr.gpu.stats()["pf_issued"] > 0
    # faults injected on the host: unmapped block, cleared PTE, damaged header bytes, short destination
    bt = w.block_table.copy(); bt[0, 1] = -1
    victim = int(np.nonzero(pr.cpu.pte >> 56)[0][40])
    for pte in (pr.cpu.pte, pr.gpu.pte_view().view(pr.torch.int64)):
        pte[victim] = 0
    off = lambda slot: int(pr.cpu.pte[slot] & 0xFFFFFFFF) * 64
    slots = [(int(bt[1, 0]) * 2 + 1) * w.n_kv_heads + h for h in range(5)]        # layer 0, seq 1, block 0, V, heads 0-4
    gp = pr.gpu.pool_view()
    for slot, byte, val in ((slots[0], 7, 9), (slots[1], 6, 1), (slots[2], 4, 0), (slots[3], 8, 5), (slots[4], 16, 0xFE)):
        pr.cpu.pool[off(slot) + byte] = val
        gp[off(slot) + byte] = val
    pf_bad = np.array([(0, 39, 0), (9, 0, 1), (1, 2, 7), (2, 3, 3)], O.PREFETCH)
    lens = np.minimum(w.seq_lens, 200).astype(np.uint32)
    tok = w.dst_tok_off(lens)
    pr.gather(0, bt, lens, tok, pf_bad, cap_tokens=int(tok[-1]) + 8)              # last sequence does not fit
    pr.check_state()
    st = pr.gpu.status()
    assert st["count"][O.ST_UNMAPPED] and st["count"][O.ST_BAD_RECORD] == 5 and st["count"][O.ST_BAD_DST]
    pr.close()


def test_prefetched_block_rewritten_then_prefetched_again():
    """The residency tags know (layer, block), not the record behind it: after a block's pages are rewritten, a
    prefetch of that block is still skipped as resident until the caller clears the tag (the lazy invalidation of
    Sec. 3.4.3 is the caller's step); after the clear the new version is fetched."""
    w = workloads.decode_fetch(seed=8, n_layers=2, batch=3, steps=2, max_blocks_per_seq=12, len_lo=60, len_hi=150)
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 2368 * 2)
    for layer in range(w.n_layers):
        slots = w.layer_slots(layer)
        pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3)
    lens = np.minimum(w.seq_lens, 40).astype(np.uint32)
    tok = w.dst_tok_off(lens)
    pf = np.array([(1, 3, 2)], O.PREFETCH)                                        # sequence 1, block 3 -> slot 2
    _, first = pr.gather(1, w.block_table, lens, tok, pf)
    assert pr.gpu.stats()["pf_issued"] == 1
    # the block's pages get new contents (those of another block), raw this time
    slots = w.layer_slots(1, [int(w.block_table[1, 3])])
    other = w.layer_slots(1, [int(w.block_table[0, 0])])
    pr.compress(w.gen_pages(other), np.arange(len(slots)), slots, 0)
    _, again = pr.gather(1, w.block_table, lens, tok, pf)
    assert pr.gpu.stats()["pf_skipped"] == 1 and np.all(again == 0xCDCD)          # taken for resident: nothing moved
    t = 1 * 4 + 2
    pr.cpu.l2_tag[t] = 0
    pr.gpu.l2_tag_view().view(pr.torch.int64)[t] = 0
    _, fresh = pr.gather(1, w.block_table, lens, tok, pf)
    assert pr.gpu.stats()["pf_issued"] == 2
    page = lambda buf: buf.reshape(-1, 2048)[(1 * 4 + 2) * 2 * w.n_kv_heads:(1 * 4 + 3) * 2 * w.n_kv_heads]
    assert np.array_equal(page(fresh), w.gen_pages(other)) and not np.array_equal(page(fresh), page(first))
    pr.check_state()
    pr.close()


def test_device_generator_matches_numpy_generator():
    import torch
    from kvgen import device
    w = workloads.llama13b(seed=6, n_layers=3)
    first, n = w.pages_per_layer - 37, 2 * 37 + 11                                # straddles a layer boundary
    out = torch.empty(n * 2048, dtype=torch.int16, device="cuda")
    device.fill(out, w.seed, first, n, torch.from_numpy(w.scales).cuda(), w.pages_per_layer, w.n_kv_heads)
    want = w.gen_pages(np.arange(first, first + n))
    assert np.array_equal(out.cpu().numpy().view(np.uint16).reshape(n, 2048), want)


def test_piecewise_linear_pages_device_twin_and_codec_parity():
    """The device generator of the piecewise-linear pages equals the numpy one; on those pages (records a third of
    the page, one to eight run heads per group) every packed scheme matches the oracle and the fetch is lossless."""
    import torch
    from kvgen import device
    w = workloads.llama70b(seed=23, n_layers=2, batch=3, seq=192)
    w.data = "runs"
    first, n = w.pages_per_layer - 21, 2 * 21 + 5                                # straddles the layer boundary
    out = torch.empty(n * 2048, dtype=torch.int16, device="cuda")
    device.fill_runs(out, w.seed, first, n)
    assert np.array_equal(out.cpu().numpy().view(np.uint16).reshape(n, 2048), w.gen_pages(np.arange(first, first + n)))
    for scheme in (3, 4, 19, 2):
        pr = Pair.for_workload(w)
        for layer in range(w.n_layers):
            slots = w.layer_slots(layer)
            pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, scheme)
        pr.check_state()
        if scheme != 2:
            assert pr.gpu.stats()["pages_mode"][3] == len(w.layer_slots(0)) * 2
        d, _ = pr.gather(1, w.block_table, w.seq_lens, w.dst_tok_off())
        if scheme in (3, 4):                                                      # one scale per page: exactly 1/128
            H, tpad = w.n_kv_heads, ((w.seq_lens.astype(np.int64) + 15) // 16) * 16
            page = d[:2048]                                                       # sequence 0, K, head 0, block 0
            slot = ((1 * w.blocks_per_layer + int(w.block_table[0, 0])) * 2 + 0) * H + 0
            assert np.array_equal(page.reshape(16, 128), w.gen_pages([slot])[0].reshape(16, 128)[:16])
        pr.close()


@pytest.mark.parametrize("H,batch", [(5, 7), (40, 3), (1, 3000)])
def test_odd_head_counts_and_many_sequences(H, batch):
    """Head counts that do not divide the warp count, and a batch long enough to need the large
    shared-memory prefix array."""
    rng = np.random.default_rng(H)
    mbs = 6 if batch < 100 else 2
    bpl = batch * mbs
    pr = Pair(2, H, bpl, mbs, batch, 64 * 40 * 2 * bpl * 2 * H // 2)
    bt = rng.permutation(bpl).astype(np.int32).reshape(batch, mbs)
    scales = gen.channel_scales(H, 2, "fixed4")
    for layer in range(2):
        slots = (layer * bpl * 2 * H + np.arange(bpl * 2 * H)).astype(np.uint32)
        src = gen.gen_pages(11, slots, scales, bpl * 2 * H, H)
        pr.compress(src, np.arange(len(slots)), slots, 3 if layer else 1)
    lens = rng.integers(0, 16 * mbs + 1, batch).astype(np.uint32)
    tpad = ((lens.astype(np.int64) + 15) // 16) * 16
    tok = np.concatenate([[0], np.cumsum(tpad)[:-1]]).astype(np.uint64)
    pf = np.array([(b, int(rng.integers(mbs)), int(rng.integers(4))) for b in rng.permutation(batch)[:5]], O.PREFETCH)
    for layer in range(2):
        pr.gather(layer, bt, lens, tok, pf)
    pr.check_state()
    pr.close()


def test_adaptive_scheme_mixes_modes_in_one_pool():
    """scheme AUTO over Gaussian pages (kept as delta streams) and pages with long runs (run-length coded)."""
    w = workloads.llama70b(seed=4, n_layers=1, batch=4, seq=256)                 # 1,024 pages
    pr = Pair.for_workload(w)
    slots = w.layer_slots(0)
    src = w.gen_pages(slots)
    src[::3] = gen.structured_pages(12, len(src[::3]))
    pr.compress(src, np.arange(len(slots)), slots, 4)
    pr.check_state()
    modes = pr.gpu.stats()["pages_mode"]
    assert modes[2] > 300 and modes[3] > 300 and modes[0] == modes[1] == 0
    pr.gather(0, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    pr.close()


def test_grouped_and_page_scales_mixed_in_one_pool_and_damaged_group_tables():
    """Per-channel-group scales: records of both kinds in one pool, the adaptive choice on top, the
    worst-case record (every symbol a run), and group tables damaged on the host."""
    w = workloads.llama70b(seed=9, n_layers=2, batch=4, seq=256)                 # 1,024 pages per layer
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 2432)
    rng = np.random.default_rng(3)
    slots = w.layer_slots(0)
    src = w.gen_pages(slots)
    src[::5] = gen.structured_pages(13, len(src[::5]))
    noisy = rng.integers(0, 2, (7, 2048)).astype(np.uint16) * 0xBC00             # +-... every other symbol differs
    noisy[:, ::2] = 0x3C00
    noisy = (noisy.astype(np.uint32) | rng.integers(0, 512, (7, 2048))).astype(np.uint16)
    src[1:8] = noisy
    half = len(slots) // 2
    pr.compress(src, np.arange(half), slots[:half], 3 | 16)
    pr.compress(src, np.arange(half, len(slots)), slots[half:], 3)
    slots1 = w.layer_slots(1)
    pr.compress(src, np.arange(len(slots1)), slots1, 4 | 16)
    pr.check_state()
    modes = {int(m) for m in (pr.cpu.pte[pr.cpu.pte != 0] >> 48) & 0xFF}
    assert modes == {3, 18, 19}
    longest = int(((pr.cpu.pte[slots[:half]] >> 32) & 0xFFFF).max())
    assert longest > 2320                                                        # longer than any page-scale record
    for layer in range(2):
        pr.gather(layer, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    assert sum(pr.gpu.status()["count"]) == 0
    # damage: an Inf pattern in a group table, a raw record flagged as grouped (header and PTE agree)
    off = lambda slot: int(pr.cpu.pte[slot] & 0xFFFFFFFF) * 64
    gp = pr.gpu.pool_view()
    a, b = int(slots[3]), int(slots[10])
    for pool in (pr.cpu.pool, gp):
        pool[off(a) + 16 + 2 * 9 + 1] = 0x7C
        pool[off(b) + 6] = 16
    for pte in (pr.cpu.pte, pr.gpu.pte_view().view(pr.torch.int64)):
        pte[b] = (int(pte[b]) & ~(0xFF << 48)) | (16 << 48)
    pr.gather(0, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    assert pr.gpu.status()["count"][O.ST_BAD_RECORD] == 2
    pr.close()


def test_back_to_back_gathers_keep_stream_order():
    """Gather calls issued without any synchronisation in between: launches with disjoint
    destinations may overlap on the GPU, a launch that reuses a destination must still come after
    the earlier writer."""
    import torch
    w = workloads.llama70b(seed=8, n_layers=3, batch=4, seq=448)
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 2368)
    for layer in range(3):
        slots = w.layer_slots(layer)
        pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3)
    n = w.demand_tokens() * 2 * w.n_kv_heads * 128
    x = torch.full((n,), -1, dtype=torch.int16, device="cuda")
    y = torch.full((n,), -1, dtype=torch.int16, device="cuda")
    bt, lens, tok = pr.t(w.block_table), pr.t(w.seq_lens), pr.t(w.dst_tok_off())
    for rep in range(3):
        pr.gpu.decompress_gather(0, bt, lens, tok, x)
        pr.gpu.decompress_gather(1, bt, lens, tok, y)
        pr.gpu.decompress_gather(2, bt, lens, tok, x)          # same destination as the first call
    want = {}
    for layer in (1, 2):
        d = np.zeros(n, np.uint16)
        l2 = np.zeros(w.batch * 4 * 2 * w.n_kv_heads * 2048, np.uint16)
        pr.cpu.decompress_gather(layer, w.block_table, w.seq_lens, w.dst_tok_off(), None, d, l2)
        want[layer] = d
    assert np.array_equal(x.cpu().numpy().view(np.uint16), want[2])
    assert np.array_equal(y.cpu().numpy().view(np.uint16), want[1])
    pr.close()


def test_a_foreign_consumer_after_chained_gathers_sees_every_earlier_gather():
    """Gather into x, then an independent gather into y (which the library launches without waiting for the
    first), then a kernel that is not the library's reads x on the same stream with no synchronisation in
    between.  Stream order promises that x is complete; 200 repetitions, x refilled each time."""
    import torch
    w = workloads.llama70b(seed=8, n_layers=2, batch=16, seq=2048)             # 32,768 pages per layer: a long first gather
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 2368)
    for layer in range(2):
        slots = w.layer_slots(layer)
        pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3)
    n = w.demand_tokens() * 2 * w.n_kv_heads * 128
    small_lens = np.full(w.batch, 16, np.uint32)                                # the second gather is short: it ends first
    x = torch.empty(n, dtype=torch.int16, device="cuda")
    y = torch.empty(16 * w.batch * 2 * w.n_kv_heads * 128, dtype=torch.int16, device="cuda")
    bt, lens, tok = pr.t(w.block_table), pr.t(w.seq_lens), pr.t(w.dst_tok_off())
    lens2, tok2 = pr.t(small_lens), pr.t(w.dst_tok_off(small_lens))
    d = np.zeros(n, np.uint16)
    l2 = np.zeros(w.batch * 4 * 2 * w.n_kv_heads * 2048, np.uint16)
    pr.cpu.decompress_gather(0, w.block_table, w.seq_lens, w.dst_tok_off(), None, d, l2)
    want = int(d.view(np.int16).astype(np.int64).sum())
    sums = torch.zeros(200, dtype=torch.int64, device="cuda")
    for rep in range(200):
        x.fill_(1)
        pr.gpu.clear_status()                                                   # the first gather of a repetition is an ordinary launch
        pr.gpu.decompress_gather(0, bt, lens, tok, x)
        pr.gpu.decompress_gather(1, bt, lens2, tok2, y)
        sums[rep] = x.sum(dtype=torch.int64)
    got = sums.cpu().numpy()
    assert np.all(got == want), f"{np.count_nonzero(got != want)} of 200 reductions ran before the first gather had finished"
    pr.close()


def test_gather_warps_walk_several_batches_of_pages_with_faults_and_prefetch():
    """A layer large enough that every warp of the gather delivers more than 32 pages (its translation
    runs lane-parallel in batches of 32): mixed raw and packed records, unmapped blocks, cleared
    entries, damaged headers and a prefetch list, all spread over the page range; every byte compared."""
    w = workloads.llama70b(seed=9, n_layers=1, batch=72, seq=2048)                # 9,216 blocks, 147,456 pages
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 2624)
    slots = w.layer_slots(0)
    src = w.gen_pages(slots)
    src[::97, 5] = 0x7C00                                                         # an Inf: stored raw
    pr.compress(src, np.arange(len(slots)), slots, 3)
    rng = np.random.default_rng(3)
    bt = w.block_table.copy()
    for b, n in zip(rng.integers(0, 72, 40), rng.integers(0, 128, 40)):
        bt[b, n] = -1 if (b + n) % 2 else w.blocks_per_layer + 5
    victims = rng.choice(np.nonzero(pr.cpu.pte >> 56)[0], 60, replace=False)
    gp_pte = pr.gpu.pte_view().view(pr.torch.int64)
    for v in victims[:30]:
        pr.cpu.pte[v] = 0
        gp_pte[int(v)] = 0
    gp = pr.gpu.pool_view()
    for v in victims[30:]:                                                        # version byte of the header
        o = int(pr.cpu.pte[v] & 0xFFFFFFFF) * 64 + 7
        pr.cpu.pool[o] = 3
        gp[o] = 3
    lens = np.full(72, 2048, np.uint32)
    lens[5], lens[40], lens[71] = 0, 1000, 17
    pf = np.array([(b, int(n), int(s)) for b, n, s in zip(rng.integers(0, 72, 100), rng.integers(0, 128, 100), rng.integers(0, 4, 100))], O.PREFETCH)
    _, first = np.unique(pf["seq"].astype(np.int64) * 4 + pf["l2_slot"], return_index=True)   # (seq, slot) pairs must be distinct
    pf = pf[np.sort(first)]
    pr.gather(0, bt, lens, w.dst_tok_off(lens), pf)
    pr.gather(0, bt, lens, w.dst_tok_off(lens), pf)                               # second time: the entries are resident
    pr.check_state()
    st = pr.gpu.status()["count"]
    assert st[O.ST_UNMAPPED] and st[O.ST_BAD_PTE] and st[O.ST_BAD_RECORD] and pr.gpu.stats()["pf_skipped"] > 0
    pr.close()


def test_sequences_longer_than_the_block_table_are_reported_and_left_out():
    """Lengths beyond what the block table describes — one block too many, and an absurd value whose block count
    would wrap a 32-bit prefix sum: each is reported once (unmapped, at its first page's index) and nothing of
    it is written; the others are delivered; the fused attention gives zero rows for them."""
    w = workloads.llama70b(seed=4, n_layers=1, batch=4, seq=96)
    pr = Pair.for_workload(w)
    slots = w.layer_slots(0)
    pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3)
    lens = np.array([48, 97, 0xFFFFFFF0, 5], np.uint32)
    pr.gather(0, w.block_table, lens, np.array([0, 48, 48, 48], np.uint64), cap_tokens=64)
    pr.check_state()
    st = pr.gpu.status()
    assert st["count"][O.ST_UNMAPPED] == 2 and st["first"][O.ST_UNMAPPED] == 3 * 16 and sum(st["count"]) == 2
    import torch
    q = np.random.default_rng(1).standard_normal((4, 16, 128)).astype(np.float16)
    want = pr.cpu.attend(0, w.block_table, lens, q.view(np.uint16), 16)
    assert not want[1].any() and not want[2].any() and want[0].any()
    # error bound from the sequences that take part (the helper would size buffers by the absurd length)
    valid = np.array([48, 0, 0, 5], np.uint32)
    _, tpad, tok = pr._layout(valid)
    d = np.zeros(int(tpad.sum()) * 2 * w.n_kv_heads * 128, np.uint16)
    scratch = O.Pool.__new__(O.Pool)
    scratch.__dict__.update(pr.cpu.__dict__)
    scratch.status, scratch.stats, scratch.l2_tag = O.Status(), O.Stats(), pr.cpu.l2_tag.copy()
    scratch.decompress_gather(0, w.block_table, valid, tok, None, d, np.zeros(w.batch * 4 * 2 * w.n_kv_heads * 2048, np.uint16))
    ws = torch.empty(pr.gpu.attend_workspace_bytes(4), dtype=torch.uint8, device="cuda")
    out = torch.full((4, 16, 128), float("nan"), dtype=torch.float16, device="cuda")
    pr.gpu.decompress_attend(0, pr.t(w.block_table), pr.t(lens), pr.t(q).view(torch.float16), out, ws)
    pr._attend_check(out.cpu().numpy(), want, pr._vmax(d, valid, tpad, tok), 2, "decompress_attend")
    pr.check_state()
    pr.close()


def test_reads_on_one_stream_while_another_layer_is_compressed_on_a_second():
    """The header allows reading calls to run at the same time as a compress call whose slots they do not read
    (the compressor only appends behind the cursor and writes its own slots' entries).  Layer 0 is fetched and
    attended on one stream while layers 1..3 are compressed on another, with no ordering between the streams;
    afterwards everything equals the oracle's state, and every fetch of layer 0 equals the oracle's pages."""
    import torch
    w = workloads.llama70b(seed=41, n_layers=4, batch=4, seq=1024)
    pr = Pair.for_workload(w)
    slots0 = w.layer_slots(0)
    pr.compress(w.gen_pages(slots0), np.arange(len(slots0)), slots0, 3)
    want = np.zeros(w.demand_tokens() * 2 * w.n_kv_heads * 128, np.uint16)
    l2 = np.zeros(w.batch * 4 * 2 * w.n_kv_heads * 2048, np.uint16)
    pr.cpu.decompress_gather(0, w.block_table, w.seq_lens, w.dst_tok_off(), None, want, l2)
    want_t = torch.from_numpy(want.view(np.int16)).cuda()
    bt, lens, tok = pr.t(w.block_table), pr.t(w.seq_lens), pr.t(w.dst_tok_off())
    srcs = [(pr.t(w.gen_pages(w.layer_slots(l))), pr.t(np.arange(w.pages_per_layer, dtype=np.uint32)), pr.t(w.layer_slots(l))) for l in (1, 2, 3)]
    writer, reader = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = [torch.empty_like(want_t) for _ in range(12)]
    with torch.cuda.stream(writer):
        for src, idx, slots in srcs:
            pr.gpu.compress(src, idx, slots, 3)
    with torch.cuda.stream(reader):
        for o in outs:
            pr.gpu.decompress_gather(0, bt, lens, tok, o)
    torch.cuda.synchronize()
    for i, o in enumerate(outs):
        assert torch.equal(o, want_t), f"fetch {i} of layer 0 differs while other layers were being compressed"
    for l in (1, 2, 3):                                                            # the oracle catches up
        slots = w.layer_slots(l)
        pr.cpu.compress(w.gen_pages(slots), np.arange(len(slots), dtype=np.uint32), slots, 3)
    for _ in outs[1:]:                                                             # its counters count twelve fetches too (one was made above)
        pr.cpu.decompress_gather(0, w.block_table, w.seq_lens, w.dst_tok_off(), None, want.copy(), l2)
    pr.check_state()
    pr.close()


def test_gathers_with_chaining_switched_off_give_the_same_pages():
    import torch
    w = workloads.llama70b(seed=8, n_layers=2, batch=4, seq=448)
    pr = Pair.for_workload(w)
    for layer in range(2):
        slots = w.layer_slots(layer)
        pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3)
    pr.gpu.set_gather_chaining(False)
    for rep in range(3):
        for layer in range(2):
            pr.gather(layer, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.gpu.set_gather_chaining(True)
    for layer in range(2):
        pr.gather(layer, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    pr.close()
