"""speckv_compress_static: the compressor for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option (an inference server that
gave all device memory to its own allocator at start-up, a plug-in that only receives
buffers).  For them the library has one entry point that takes every buffer from the caller
and keeps its scan scratch in a fixed array inside the library.  This test drives it through
the C ABI and requires the same bytes as the context-based speckv_compress and as the CPU
oracle: record log, page table, cursor, status block and counters bit for bit, on two calls in a row (the second appends behind the first and
reuses the fixed scratch, which still holds the first call's contents).
Collected last on purpose: a failure here must not hide any other test's result."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _ctl_block(torch):
    ctl = torch.zeros(160, dtype=torch.uint8, device="cuda")
    ctl[40:72] = 0xFF                                   # "first index" words start at 0xFFFFFFFF
    return ctl


def test_static_entry_point_matches_context_compress_on_two_calls():
    import torch
    from kvgen import workloads
    from oracle import oracle as O
    from paper_2512_11920_b200 import Context, SpeckvError, compress_static, STATIC_MAX_PAGES

    w = workloads.llama70b(seed=9, n_layers=2, batch=4, seq=448)              # 1,792 pages per layer
    dev = torch.device("cuda:0")
    pool_bytes = w.n_slots * 2368
    ref = Context(w.n_layers, w.n_kv_heads, w.blocks_per_layer, w.max_blocks_per_seq, w.batch, pool_bytes)
    cpu = O.Pool(w.n_layers, w.n_kv_heads, w.blocks_per_layer, w.max_blocks_per_seq, w.batch, pool_bytes)
    pool = torch.zeros(pool_bytes, dtype=torch.uint8, device=dev)
    pte = torch.zeros(w.n_slots, dtype=torch.int64, device=dev)
    ctl = _ctl_block(torch)
    rng = np.random.default_rng(3)
    for call, layer in enumerate((0, 1)):
        slots = w.layer_slots(layer)
        src = w.gen_pages(slots)
        if call == 1:                                                         # ragged count, permuted list, one bad index
            order = rng.permutation(len(slots))[:1001].astype(np.uint32)
            dst = slots[order].copy()
            dst[17] = 1 << 30
        else:
            order, dst = np.arange(len(slots), dtype=np.uint32), slots
        t_src = torch.from_numpy(src.view(np.int16)).to(dev)
        t_order = torch.from_numpy(order.view(np.int32)).to(dev)
        t_dst = torch.from_numpy(dst.view(np.int32)).to(dev)
        ref.compress(t_src, t_order, t_dst, 3)
        cpu.compress(src, order, dst, 3)
        compress_static(t_src, t_order, t_dst, 3, pool, pte, ctl)
        torch.cuda.synchronize()
        cursor = int(ctl[:8].view(torch.int64).item())
        assert cursor == ref.cursor() > 0
        assert torch.equal(pte, ref.pte_view().view(torch.int64)), f"page table differs after call {call}"
        used = cursor * 64
        assert torch.equal(pool[:used], ref.pool_view(used)), f"record log differs after call {call}"
        got = ctl.cpu().numpy()
        st, stats = ref.status(), ref.stats()
        assert got[8:40].view(np.uint32).tolist() == st["count"] and got[40:72].view(np.uint32).tolist() == st["first"]
        assert got[72:104].view(np.uint64).tolist() == stats["pages_mode"] and int(got[104:112].view(np.uint64)[0]) == stats["granules"]
        # and against the oracle directly, not only through the other entry point
        assert cursor == cpu.cursor.value
        assert np.array_equal(pte.cpu().numpy().view(np.uint64), cpu.pte), f"page table differs from the oracle's after call {call}"
        assert np.array_equal(pool[:used].cpu().numpy(), cpu.pool[:used]), f"record log differs from the oracle's after call {call}"
        want = cpu.status_dict()
        assert got[8:40].view(np.uint32).tolist() == want["count"] and got[40:72].view(np.uint32).tolist() == want["first"]
        cs = cpu.stats.as_dict()
        assert got[72:160].view(np.uint64).tolist() == cs["pages_mode"] + [cs[k] for k in (
            "granules", "payload_bytes", "n_runs", "nonfinite", "pages_decoded", "pf_issued", "pf_skipped")]
    assert ref.status()["count"][5] == 1                                      # the bad index was reported by both
    # beyond the fixed capacity: refused with a clear error, nothing enqueued
    big = torch.zeros(STATIC_MAX_PAGES + 1, dtype=torch.int32, device=dev)
    with pytest.raises(SpeckvError, match="too many pages"):
        compress_static(torch.zeros(2048, dtype=torch.int16, device=dev), big, big, 3, pool, pte, ctl)
    ref.close()


def test_static_entry_point_at_its_largest_size():
    """SPECKV_STATIC_MAX_PAGES pages in one call (2 GiB of K/V, 26,215 tiles of the fixed scratch): the same log,
    table and cursor as the context-based call; then, as a raw call (32,768 tiles of 16 pages: the whole array)."""
    import torch
    from kvgen import device as gen_device, workloads
    from paper_2512_11920_b200 import Context, compress_static, STATIC_MAX_PAGES
    if torch.cuda.mem_get_info()[0] < 12 << 30:
        pytest.skip("needs 12 GiB of free device memory")
    w = workloads.llama70b(seed=2, n_layers=8)                                  # 65,536 pages per layer: 8 layers = the maximum
    n = STATIC_MAX_PAGES
    assert w.n_slots == n
    dev = torch.device("cuda:0")
    src = torch.empty(n * 2048, dtype=torch.int16, device=dev)
    scales = torch.from_numpy(w.scales).to(dev)
    gen_device.fill(src, w.seed, 0, n, scales, w.pages_per_layer, w.n_kv_heads)
    idx = torch.arange(n, dtype=torch.int32, device=dev)
    for scheme, per_page in ((3, 2368), (0, 4160)):
        pool_bytes = n * per_page
        ref = Context(w.n_layers, w.n_kv_heads, w.blocks_per_layer, w.max_blocks_per_seq, w.batch, pool_bytes)
        pool = torch.zeros(pool_bytes, dtype=torch.uint8, device=dev)
        pte = torch.zeros(n, dtype=torch.int64, device=dev)
        ctl = _ctl_block(torch)
        ref.compress(src, idx, idx, scheme)
        compress_static(src, idx, idx, scheme, pool, pte, ctl)
        torch.cuda.synchronize()
        cursor = int(ctl[:8].view(torch.int64).item())
        assert cursor == ref.cursor() and sum(ref.status()["count"]) == 0
        assert torch.equal(pte, ref.pte_view().view(torch.int64))
        assert torch.equal(pool[:cursor * 64], ref.pool_view(cursor * 64))
        ref.close()
        del pool, pte
        torch.cuda.empty_cache()
