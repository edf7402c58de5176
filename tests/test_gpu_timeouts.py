"""The bounded waits of the compressor, made to run out on purpose and safely.

Every wait inside compress_kernel has a limit.  The failure is made on the host: the context is told not
to hand out the first tile of the next call, so every later tile waits for a size that is never
published.  With short limits the waits run out, the call ends, the condition comes back as
SPECKV_ST_TIMEOUT, nothing is placed, and the next ordinary call on the same context is bit-exact with
the oracle again.  Nothing here faults, traps or waits without a limit."""
import time

import numpy as np
import pytest

from kvgen import workloads
from oracle import oracle as O
from tests.parity_util import Pair

pytestmark = pytest.mark.gpu

TILE = 20   # pages per tile of the compressor


def test_raw_scheme_look_back_runs_out_too():
    """The copy kernel of scheme 0 has the same chained scan (tiles of 16 pages) and two bounded waits of its
    own (a page landing in shared memory, the scan): tile 0 withheld, four tiles requested."""
    w = workloads.tiny(seed=0)
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 4160)
    pr.gpu.set_wait_limits(lookback_polls=2000, wait_ns=50_000_000)
    dt = _timed_out_call(pr, w, 4 * 16, scheme=0)
    st = pr.gpu.status()
    assert st["count"][O.ST_TIMEOUT] == 3 and st["first"][O.ST_TIMEOUT] == 16 and sum(st["count"]) == 3
    assert dt < 1.0
    _nothing_was_placed(pr)
    pr.gpu.clear_status()
    pr.gpu.set_wait_limits()
    slots = w.layer_slots(0)
    pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 0)
    pr.check_state()
    pr.gather(0, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    pr.close()


def _timed_out_call(pr, w, n_pages, scheme=3):
    """Compress the first n_pages slots of layer 0 on the GPU only, with tile 0 withheld."""
    torch = pr.torch
    slots = w.layer_slots(0)[:n_pages]
    src = pr.t(w.gen_pages(slots))
    idx = pr.t(np.arange(n_pages, dtype=np.uint32))
    pr.gpu.inject_missing_tiles(1)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    pr.gpu.compress(src, idx, pr.t(slots), scheme)
    torch.cuda.synchronize()
    return time.perf_counter() - t0


def _nothing_was_placed(pr):
    assert pr.gpu.cursor() == pr.cpu.cursor.value
    assert not pr.gpu.pte_view().any().item(), "a page-table entry was written by a call that timed out"
    assert pr.gpu.stats() == pr.cpu.stats.as_dict()


def test_look_back_wait_runs_out_and_the_failure_travels_down_the_chain():
    """Three tiles, tile 0 withheld: the scan of tile 1 polls tile 0's status word until its limit, marks
    its own word failed; tile 2 either sees that mark or runs out itself.  Both are counted."""
    w = workloads.tiny(seed=0)
    pr = Pair.for_workload(w)
    pr.gpu.set_wait_limits(lookback_polls=2000, wait_ns=50_000_000)
    dt = _timed_out_call(pr, w, 3 * TILE)
    st = pr.gpu.status()
    assert st["count"][O.ST_TIMEOUT] == 2 and st["first"][O.ST_TIMEOUT] == 1 * TILE
    assert sum(st["count"]) == 2
    assert dt < 1.0, f"the call took {dt:.2f} s with a limit of 2,000 polls"
    _nothing_was_placed(pr)
    # the same context, ordinary calls: as if nothing had happened
    pr.gpu.clear_status()
    pr.gpu.set_wait_limits()                                        # defaults
    slots = w.layer_slots(0)
    pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, 3)
    pr.check_state()
    pr.gather(0, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    pr.close()


def test_barrier_waits_run_out_while_the_scan_is_stuck():
    """Enough tiles that every CTA has several: with tile 0 withheld every scanner is stuck in its look-back
    (limit: tens of milliseconds), the encoders run three record stages ahead and then wait for a stage that
    is never released; that wait has a limit of one millisecond.  They give up, raise the CTA's abort flag,
    the loader waits for its copies in flight and leaves, the scanner follows when its own limit ends."""
    w = workloads.llama70b(seed=5, n_layers=1, batch=8, seq=2048)    # 16,384 pages = 820 tiles, 5-6 per CTA
    pr = Pair.for_workload(w)
    pr.gpu.set_wait_limits(lookback_polls=20000, wait_ns=1_000_000)
    n = len(w.layer_slots(0))
    dt = _timed_out_call(pr, w, n)
    st = pr.gpu.status()
    assert st["count"][O.ST_TIMEOUT] >= 2 and st["first"][O.ST_TIMEOUT] == 1 * TILE
    assert sum(st["count"]) == st["count"][O.ST_TIMEOUT]
    assert dt < 5.0, f"the call took {dt:.2f} s"
    _nothing_was_placed(pr)
    pr.gpu.clear_status()
    pr.gpu.set_wait_limits()
    slots = w.layer_slots(0)
    order = np.random.default_rng(1).permutation(n)
    pr.compress(w.gen_pages(slots), order, slots[order], 3)
    pr.check_state()
    pr.gather(0, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    pr.close()
