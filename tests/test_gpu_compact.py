"""GPU parity of speckv_compact (pool lifecycle): pool bytes, page table, cursor and statuses after
compaction equal the oracle's, and the pool reads back the same pages."""
import numpy as np
import pytest

from kvgen import gen, workloads
from oracle import oracle as O
from tests.parity_util import Pair

pytestmark = pytest.mark.gpu


def test_tail_page_rewrites_then_compaction():
    H, nblk = 2, 3
    pr = Pair(1, H, nblk, nblk, 1, 1 << 20)
    full = gen.gen_pages(3, np.arange(nblk * 2 * H), np.ones((1, 2, 128), np.float32), nblk * 2 * H, H)
    slots = np.arange(nblk * 2 * H, dtype=np.uint32)
    pr.compress(full[:2 * 2 * H], np.arange(2 * 2 * H), slots[:2 * 2 * H], 3)
    for t in range(1, 17):                                                         # the tail block fills token by token
        tail = full[2 * 2 * H:].copy().reshape(-1, 16, 128)
        tail[:, t:, :] = 0
        pr.compress(tail.reshape(-1, 2048), np.arange(2 * H), slots[2 * 2 * H:], 3 if t % 2 else 3 | 16)
    pr.check_state()
    grown = pr.gpu.cursor()
    bt = np.arange(nblk, dtype=np.int32).reshape(1, -1)
    before, _ = pr.gather(0, bt, [48], [0])
    pr.compact()
    pr.check_state()
    assert pr.gpu.cursor() < grown // 3
    after, _ = pr.gather(0, bt, [48], [0])
    assert np.array_equal(before, after)
    pr.compact()                                                                   # nothing left to drop
    pr.check_state()
    pr.close()


def test_compaction_over_many_blocks_with_rewrites_raw_pages_and_bad_entries():
    w = workloads.llama70b(seed=12, n_layers=3, batch=4, seq=448)                  # 5,376 slots: several 1,024-slot blocks
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 2368 * 2)
    rng = np.random.default_rng(2)
    for layer in (2, 0, 1):                                                        # log order != slot order
        slots = w.layer_slots(layer)
        order = rng.permutation(len(slots))
        pr.compress(w.gen_pages(slots), order, slots[order], [3, 4 | 16, 1][layer])
    slots = w.layer_slots(1)
    again = rng.permutation(len(slots))[:700]
    pr.compress(w.gen_pages(slots), again, slots[again], 0)                        # a third of layer 1 rewritten raw
    victims = rng.permutation(w.n_slots)[:5]
    assert pr.free_slots([victims[0]])[0] == 1                                     # a freed slot
    for pte in (pr.cpu.pte, pr.gpu.pte_view().view(pr.torch.int64)):
        pte[int(victims[1])] = (int(pr.cpu.cfg.pool_bytes // 64) - 1) | (4112 << 32) | (1 << 56)   # ends beyond the pool
        pte[int(victims[2])] = 5 | (9 << 32) | (1 << 56)                           # shorter than a header
    pr.compact()
    pr.check_state()
    st = pr.gpu.status()
    assert st["count"][O.ST_BAD_RECORD] == 2
    live = int((pr.cpu.pte >> 56 & 1).sum())
    assert live == w.n_slots - 3
    for layer in range(3):
        pr.gather(layer, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    pr.close()


def test_entries_sharing_records_overflow_the_pool():
    """Two slots pointing at one record each get a copy of their own; when the copies no longer fit, the
    excess is reported POOL_FULL, cleared, and still counted by the cursor.  Same case as the oracle's
    hand-worked pin, then a larger one that crosses 1,024-slot blocks."""
    pr = Pair(1, 1, 4, 4, 1, 64 * 12)
    zero, const = np.zeros(2048, np.uint16), np.full(2048, 3.5, np.float16).view(np.uint16)
    pr.compress(np.stack([zero, const]), [0, 1], [0, 2], 3)
    for pte in (pr.cpu.pte, pr.gpu.pte_view().view(pr.torch.int64)):
        pte[1] = int(pr.cpu.pte[0]); pte[3] = int(pr.cpu.pte[2])
    pr.compact()
    pr.check_state(pool_defined_bytes=10 * 64)                                     # two copies of 5 granules fitted
    st = pr.gpu.status()
    assert pr.gpu.cursor() == 20 and st["count"][O.ST_POOL_FULL] == 2 and st["first"][O.ST_POOL_FULL] == 2
    pr.close()

    w = workloads.llama70b(seed=3, n_layers=2, batch=4, seq=448)                   # 1,792 slots per layer, layer 0 written
    pool_bytes = 64 * 70000
    pr = Pair.for_workload(w, pool_bytes=pool_bytes)
    slots = w.layer_slots(0)
    pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3)
    used = pr.gpu.cursor()
    assert used < 70000 < 2 * used                                                 # one copy fits, two do not
    free = w.layer_slots(1).astype(np.int64)                                       # layer 1's entries share layer 0's records
    gpte = pr.gpu.pte_view().view(pr.torch.int64)
    gpte[pr.torch.from_numpy(free).to(pr.dev)] = gpte[pr.torch.from_numpy(slots.astype(np.int64)).to(pr.dev)]
    pr.cpu.pte[free] = pr.cpu.pte[slots]
    pr.compact()
    live_end = max((int(e) & 0xFFFFFFFF) + (((int(e) >> 32) & 0xFFFF) + 63) // 64 for e in pr.cpu.pte if (int(e) >> 56) & 1)
    pr.check_state(pool_defined_bytes=live_end * 64)
    st = pr.gpu.status()
    assert pr.gpu.cursor() == 2 * used and 0 < st["count"][O.ST_POOL_FULL] < len(slots)
    live = int((pr.cpu.pte >> 56 & 1).sum())
    assert live == 2 * len(slots) - st["count"][O.ST_POOL_FULL]
    pr.close()


def test_free_slots_then_compaction_reclaims_a_finished_sequence():
    """A request ends: every slot of its blocks is freed (some named twice, one out of range), the counts
    equal the oracle's, gathers of the other sequences are unchanged, the freed one reads as never written,
    and compaction shrinks the log by exactly the granules that were reported."""
    w = workloads.llama70b(seed=21, n_layers=2, batch=3, seq=320)                  # 20 blocks per sequence
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 4160)
    for layer in range(2):
        slots = w.layer_slots(layer)
        pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3 if layer else 0)
    before = pr.gpu.cursor()
    gone = np.concatenate([w.layer_slots(layer, blocks=w.block_table[1]) for layer in range(2)])
    listed = np.concatenate([gone, gone[:40], [w.n_slots + 7]]).astype(np.uint32)
    entries, gran = pr.free_slots(listed)
    assert entries == len(gone) == 2 * 20 * 16
    pr.check_state()
    st = pr.gpu.status()
    assert st["count"][O.ST_BAD_INDEX] == 1 and st["first"][O.ST_BAD_INDEX] == len(listed) - 1
    for layer in range(2):
        pr.gather(layer, w.block_table, w.seq_lens, w.dst_tok_off())              # sequence 1: BAD_PTE, left untouched
    assert pr.gpu.status()["count"][O.ST_BAD_PTE] == len(gone)
    pr.compact()
    pr.check_state()
    assert pr.gpu.cursor() == before - gran
    pr.close()


def test_compaction_moves_records_straight_into_vacated_space():
    """Every slot written twice: the log is [old versions][live versions], so every record's new place lies in
    garbage and no live record is in the way — the records are moved without the detour through the scratch
    area (which the test leaves poisoned: nothing of it may reach the pool)."""
    w = workloads.llama70b(seed=23, n_layers=2, batch=4, seq=448)
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * (4160 + 2368))
    slots = np.concatenate([w.layer_slots(0), w.layer_slots(1)])
    pages = w.gen_pages(slots)
    pr.compress(pages, np.arange(len(slots)), slots, 0)                             # old versions: raw, larger than what replaces them
    pr.compress(pages, np.arange(len(slots)), slots, 3)                             # live versions behind them
    half = pr.gpu.cursor()
    pr.cpu.compact()
    scratch = pr.torch.full((pr.gpu.compact_scratch_bytes(),), 0xA5, dtype=pr.torch.uint8, device=pr.dev)
    pr.gpu.compact(scratch)
    live_end = pr.cpu.cursor.value
    assert live_end < half - live_end                                               # the live records fit into the garbage in front
    pr.check_state(pool_defined_bytes=live_end * 64)
    assert bool((scratch[:live_end * 64] == 0xA5).all()), "a record went through the scratch area"
    for layer in range(2):
        pr.gather(layer, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.close()
