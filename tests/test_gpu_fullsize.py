"""Parity at the benchmarked size, in the launch configuration bench.py times: the 70B-shaped
workload (80 layers x 65,536 pages, 20 GiB), one compress call and one gather call per layer.
Also the 7B-shaped workload in full (32 layers, 8 GiB) and the 13B-shaped one in full (40 layers, 50 GiB of
K/V, about 140 GB resident with pool and destination; its per-layer outlier channels differ from layer to
layer).
The oracle cannot process 20 GiB in a test, so: (a) sampled pages are compared bit for bit
(record bytes, page-table entry, gathered fp16), (b) properties that hold at any size are
checked over ALL pages on the device (placement = prefix sum in list order, every page
delivered, nothing reported), (c) idempotence over ALL pages: the gathered K/V of every layer is
compressed again and must give the first pass's records byte for byte (the oracle's pinned property
compress(decompress(C)) == C), so a rare wrong page in either direction cannot hide among the unsampled."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _free_gib():
    import torch
    return torch.cuda.mem_get_info()[0] / 2 ** 30


@pytest.mark.parametrize("name,layers,scheme", [("llama2-70b-gqa", 80, 3), ("llama2-7b", 32, 3), ("llama2-13b", 40, 3),
                                                ("llama2-70b-gqa", 80, 3 | 16)])     # 16: one scale per channel group
def test_full_size_sampled_parity_and_placement(name, layers, scheme):
    import torch
    import bench
    from kvgen import workloads
    w = workloads.BY_NAME[name](seed=0, n_layers=layers)
    need = (2.6 + 0.6 / layers) * w.n_slots * 4096 / 2 ** 30
    torch.cuda.empty_cache()                                                     # blocks cached from earlier tests count as used
    if _free_gib() < need + 4:
        pytest.skip(f"needs {need:.0f} GiB of free device memory")
    b = bench.Bench(w, torch.device("cuda:0"), scheme, pool_page_bytes=2368)
    grp = 32 if scheme & 16 else 0                                               # bytes of group maxima per record
    b.dst.fill_(-1)
    b.step()
    torch.cuda.synchronize()
    st, stats = b.ctx.status(), b.ctx.stats()
    assert sum(st["count"]) == 0, st
    assert stats["pages_mode"][3] == b.pages and stats["pages_decoded"] == b.demand_pages == b.pages
    # (b) placement: list order is slot order here, so offsets are the running sum of record sizes
    pte = b.ctx.pte_view().view(torch.int64)
    assert bool(((pte >> 56) & 1).all()) and bool((((pte >> 48) & 0xFF) == scheme).all())
    off = pte & 0xFFFFFFFF
    gran = (((pte >> 32) & 0xFFFF) + 63) // 64
    assert int(off[0]) == 0 and bool((off[1:] == off[:-1] + gran[:-1]).all())
    assert int(off[-1] + gran[-1]) == b.ctx.cursor() == stats["granules"]
    rec_len = (pte >> 32) & 0xFFFF
    assert int(rec_len.min()) >= 273 + grp and int(rec_len.max()) <= 2320 + grp
    assert int((rec_len - 16).sum()) == stats["payload_bytes"] and int((rec_len - 272 - grp).sum()) == stats["n_runs"]
    # every destination page was written (the fill pattern 0xFFFF is a NaN the codec never emits here)
    untouched = sum(int((b.dst_layer(l).view(-1, 2048) == -1).all(dim=1).sum()) for l in range(w.n_layers))   # layer by layer: small temporaries
    assert untouched == 0
    # (a) sampled pages against the oracle
    res = b.sampled_parity(n_samples=64, seed=7)
    assert res["mismatches"] == 0, res
    # (c) idempotence, every page of every layer: where slot s of the layer sits in the gathered workspace
    from paper_2512_11920_b200 import Context
    H, ppl = w.n_kv_heads, w.pages_per_layer
    nblk = (w.seq_lens.astype(np.int64) + 15) // 16
    tok = w.dst_tok_off().astype(np.int64)
    where = np.full(ppl, -1, np.int64)
    for s_ in range(w.batch):
        p = w.block_table[s_, :nblk[s_]].astype(np.int64)                         # physical blocks of the sequence, in logical order
        for kv in range(2):
            for h in range(H):
                where[(p * 2 + kv) * H + h] = tok[s_] * 2 * H // 16 + (kv * H + h) * nblk[s_] + np.arange(nblk[s_])
    assert (where >= 0).all()
    again = Context(1, H, w.blocks_per_layer, w.max_blocks_per_seq, w.batch, ((ppl * 2368 + (1 << 20)) // 64) * 64)
    src_page = torch.from_numpy(where.astype(np.int32)).cuda()
    slots = torch.arange(ppl, dtype=torch.int32, device="cuda")
    pool1 = b.ctx.pool_view()
    for l in range(w.n_layers):
        again.reset()
        again.compress(b.dst_layer(l), src_page, slots, scheme)
        n64 = again.cursor()
        first = int(pte[l * ppl].item()) & 0xFFFFFFFF
        assert torch.equal(again.pool_view(n64 * 64), pool1[first * 64:(first + n64) * 64]), f"layer {l}: recompressed records differ"
        assert torch.equal(again.pte_view().view(torch.int64) + first, pte[l * ppl:(l + 1) * ppl]), f"layer {l}: entries differ"
    assert sum(again.status()["count"]) == 0
    again.close()
    b.ctx.close()


def test_repeated_fast_scheme_runs_keep_every_record():
    """The schemes without run-length coding encode faster than the scan places records, so the encoders
    reach the end of the page list several tiles ahead of it.  Every run must still describe every page:
    same counters and cursor run after run, no page-table entry shorter than a header (a ragged page count
    and a few raw pages included, whose encoders take a record stage without building a record)."""
    import torch
    import bench
    from kvgen import workloads
    w = workloads.BY_NAME["llama2-70b-gqa"](seed=0, n_layers=80)
    torch.cuda.empty_cache()
    if _free_gib() < 2.7 * w.n_slots * 4096 / 2 ** 30 + 4:
        pytest.skip("needs 54 GiB of free device memory")
    b = bench.Bench(w, torch.device("cuda:0"), 4, pool_page_bytes=2368)
    nan = torch.tensor([0x7E00], dtype=torch.int16, device="cuda")
    for page in (5, 2_000_003, b.pages - 9, b.pages - 4):                       # raw pages, two of them in the last tiles
        b.src[page * 2048 + 77] = nan[0]
    idx = b.idx_all[:-3]                                                         # a ragged last tile
    ref = None
    for rep in range(150):
        scheme = (4, 2, 4 | 16)[rep % 3]
        b.ctx.reset()
        b.ctx.compress(b.src, idx, idx, scheme)
        st, status = b.ctx.stats(), b.ctx.status()
        key = (st["pages_mode"][0], sum(st["pages_mode"]), st["granules"], b.ctx.cursor())
        ref = ref or key
        assert key == ref and sum(status["count"]) == 0, (rep, key, ref, status)
        if rep % 25 == 0:
            pte = b.ctx.pte_view().view(torch.int64)[:len(idx)]
            assert bool(((pte >> 56) & 1).all()) and int(((pte >> 32) & 0xFFFF).min()) >= 2064
    assert ref[0] == 4 and ref[1] == len(idx) and ref[2] == ref[3] == (len(idx) - 4) * 33 + 4 * 65
    b.ctx.close()
