"""Random call sequences on the CUDA library and on the oracle, compared after every call and in full at the end:
compress (whole layers, partial lists, rewrites; Gaussian, piecewise-linear, segment and sparse pages with planted
Inf/NaN/extreme values; every scheme; roomy and tight pools), gathers with random lengths and prefetch lists (invalid
entries included), free_slots, compaction and translation of random addresses, on small 7B- and 70B-shaped caches.
A fixed set of seeds; the same generator ran for 1,200 further seeds while the kernels were developed."""
import numpy as np
import pytest

from kvgen import gen, workloads
from oracle import oracle as O
from tests.parity_util import Pair

pytestmark = pytest.mark.gpu

SCHEMES = [0, 1, 2, 3, 4, 17, 18, 19, 20]


def random_pages(rng, w, slots):
    kind = rng.integers(4)
    if kind == 0:
        pages = w.gen_pages(slots)
    elif kind == 1:
        pages = gen.runs_pages(int(rng.integers(1 << 30)), slots, int(rng.integers(10, 250)))
    elif kind == 2:
        pages = gen.structured_pages(int(rng.integers(1 << 30)), len(slots))
    else:
        pages = w.gen_pages(slots).copy()
        # sparsify: many zeros -> long runs of zero deltas mixed with noise
        mask = rng.random(pages.shape) < rng.uniform(0.3, 0.98)
        pages[mask] = 0
    pages = pages.copy()
    # a few special values
    for _ in range(int(rng.integers(0, 4))):
        p = int(rng.integers(len(pages)))
        pages[p, int(rng.integers(2048))] = rng.choice([0x7C00, 0xFC00, 0x7E00, 0x7BFF, 0xFBFF, 0x0001, 0x8000])
    return pages


def one_case(seed):
    rng = np.random.default_rng(seed)
    n_layers = int(rng.integers(1, 4))
    batch = int(rng.integers(1, 5))
    mb = int(rng.integers(2, 16))
    w = workloads.decode_fetch(seed=seed, n_layers=n_layers, batch=batch, steps=3, max_blocks_per_seq=mb,
                               len_lo=1, len_hi=16 * mb)
    # decode_fetch is the 7B shape (32 heads); shrink sometimes by using llama70b's
    if rng.integers(2):
        seq = 16 * int(rng.integers(1, 24))
        w = workloads.llama70b(seed=seed, n_layers=n_layers, batch=batch, seq=seq)
        w.seq_lens = rng.integers(1, seq + 1, size=batch).astype(np.uint32)
    tight = rng.integers(4) == 0
    pool_bytes = int(w.n_slots * (1200 if tight else 4160 * 2)) // 64 * 64 + 64
    pr = Pair.for_workload(w, pool_bytes=pool_bytes)
    n_ops = int(rng.integers(3, 9))
    for layer in range(w.n_layers):
        slots = w.layer_slots(layer)
        perm = rng.permutation(len(slots))
        k = int(rng.integers(0, len(slots) + 1)) if rng.integers(3) == 0 else len(slots)
        pages = random_pages(rng, w, slots)
        pr.compress(pages, perm[:k], slots[perm[:k]], int(rng.choice(SCHEMES)))
    for _ in range(n_ops):
        op = rng.integers(6)
        layer = int(rng.integers(w.n_layers))
        if op == 0:      # rewrite part of a layer
            slots = w.layer_slots(layer)
            take = rng.permutation(len(slots))[: int(rng.integers(1, len(slots) + 1))]
            pages = random_pages(rng, w, slots)
            pr.compress(pages, take, slots[take], int(rng.choice(SCHEMES)))
        elif op in (1, 2):   # gather, sometimes with a prefetch list
            lens = np.minimum(w.seq_lens, rng.integers(1, 16 * w.max_blocks_per_seq + 1, size=w.batch)).astype(np.uint32)
            pf = None
            if rng.integers(2):
                n = int(rng.integers(1, 12))
                pf = np.zeros(n, O.PREFETCH)
                pf["seq"] = rng.integers(0, w.batch + 1, n)
                pf["block"] = rng.integers(0, w.max_blocks_per_seq + 2, n)
                pf["l2_slot"] = rng.integers(0, 5, n)
                # distinct (seq, slot) pairs: two entries of one call aimed at one slot have no defined winner
                _, first = np.unique(pf["seq"].astype(np.int64) * 8 + pf["l2_slot"], return_index=True)
                pf = pf[np.sort(first)]
            pr.gather(layer, w.block_table, lens, w.dst_tok_off(lens), pf)
        elif op == 3:    # free some slots
            slots = w.layer_slots(layer)
            take = rng.permutation(len(slots))[: int(rng.integers(1, max(2, len(slots) // 3)))]
            pr.free_slots(slots[take])
        elif op == 4:
            pr.compact()
        else:            # translate
            n = int(rng.integers(1, 200))
            va = np.zeros(n, O.VADDR)
            va["seq"] = rng.integers(0, w.batch + 1, n); va["layer"] = rng.integers(0, w.n_layers + 1, n)
            va["kv"] = rng.integers(0, 3, n); va["head"] = rng.integers(0, w.n_kv_heads + 1, n)
            va["pos"] = rng.integers(0, 16 * w.max_blocks_per_seq + 20, n)
            pr.translate(w.block_table, va)
    pr.check_state()
    pr.close()


@pytest.mark.parametrize("seed0", [100, 200, 300])
def test_random_call_sequences_match_the_oracle(seed0):
    for seed in range(seed0, seed0 + 8):
        one_case(seed)


# ---- the attention consumers on random caches: lengths down to zero, 1-8 query heads per KV head, sharp and flat
# softmax, rewritten and freed pages, an unmapped block

def pages_for(rng, w, slots):
    kind = rng.integers(3)
    if kind == 0:
        p = w.gen_pages(slots)
    elif kind == 1:
        p = gen.runs_pages(int(rng.integers(1 << 30)), slots, int(rng.integers(10, 250)))
    else:
        p = w.gen_pages(slots).copy()
        p[rng.random(p.shape) < rng.uniform(0.3, 0.95)] = 0
    return p


def one_attention_case(seed):
    rng = np.random.default_rng(seed)
    n_layers, batch = int(rng.integers(1, 3)), int(rng.integers(1, 6))
    if rng.integers(2):
        mb = int(rng.integers(2, 12))
        w = workloads.decode_fetch(seed=seed, n_layers=n_layers, batch=batch, steps=3, max_blocks_per_seq=mb, len_lo=1, len_hi=16 * mb)
        w.seq_lens = rng.integers(1, 16 * mb + 1, size=batch).astype(np.uint32)
    else:
        seq = 16 * int(rng.integers(1, 40))
        w = workloads.llama70b(seed=seed, n_layers=n_layers, batch=batch, seq=seq)
        w.seq_lens = rng.integers(1, seq + 1, size=batch).astype(np.uint32)
    pr = Pair.for_workload(w, pool_bytes=w.n_slots * 4160 * 2)
    for layer in range(w.n_layers):
        slots = w.layer_slots(layer)
        pr.compress(pages_for(rng, w, slots), np.arange(len(slots)), slots, int(rng.choice([0, 1, 2, 3, 4, 17, 18, 19, 20])))
    if rng.integers(2):
        layer = int(rng.integers(w.n_layers)); slots = w.layer_slots(layer)
        take = rng.permutation(len(slots))[: int(rng.integers(1, len(slots) + 1))]
        pr.compress(pages_for(rng, w, slots), take, slots[take], int(rng.choice([0, 1, 2, 3, 4, 19])))
    if rng.integers(3) == 0:
        slots = w.layer_slots(int(rng.integers(w.n_layers)))
        pr.free_slots(slots[rng.permutation(len(slots))[: int(rng.integers(1, 6))]])
    bt = w.block_table.copy()
    if rng.integers(4) == 0:
        bt[int(rng.integers(batch)), 0] = -1
    for _ in range(int(rng.integers(1, 4))):
        layer = int(rng.integers(w.n_layers))
        G = int(rng.choice([1, 2, 3, 4, 8]))
        lens = rng.integers(0, w.seq_lens + 1).astype(np.uint32)
        if not lens.any():
            lens[0] = 1
        q = (rng.standard_normal((batch, w.n_kv_heads * G, 128)) * rng.choice([0.3, 1.0, 6.0])).astype(np.float16).view(np.uint16)
        if rng.integers(2):
            pr.attend_fused(layer, bt, lens, q, w.n_kv_heads * G)
        else:
            pr.attend_dense(layer, bt, lens, q, w.n_kv_heads * G)
    pr.check_state()
    pr.close()


def test_random_attention_calls_match_the_oracle():
    for seed in range(400, 440):
        one_attention_case(seed)
