"""GPU parity of the per-layer compression selection (Sec. 3.6.3): speckv_probe_pages against the oracle's
probe (integer fields bit-exact, the three binary64 sums within 1e-11 relative: same exact terms, other order
of addition), speckv_select_scheme against the oracle's selection on the same numbers, and the policy at work
on a cache whose early layers have long runs and whose late layers are Gaussian."""
import numpy as np
import pytest

from kvgen import gen, workloads
from oracle import oracle as O
from tests.parity_util import Pair

pytestmark = pytest.mark.gpu

COST = [0.39, 0.47, 0.82, 0.85, 0.41, 0.49, 0.84, 0.87]     # warp instructions per page / 1000, measured


def _gpu_probe(pages, idx):
    import torch
    from paper_2512_11920_b200 import probe_pages, PROBE_DTYPE
    acc = torch.zeros(PROBE_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    src = torch.from_numpy(np.ascontiguousarray(pages).view(np.int16)).cuda()
    idx = np.asarray(idx, np.uint32)
    half = len(idx) // 2                                      # two calls: the accumulator is added to
    for part in (idx[:half], idx[half:]):
        if len(part):
            probe_pages(src, torch.from_numpy(part.view(np.int32)).cuda(), acc)
    return acc.cpu().numpy().view(PROBE_DTYPE)[0]


def _same(got, want):
    for f in ("pages", "nonfinite", "bad_index"):
        assert int(got[f]) == int(want[f]), f
    assert got["granules"].tolist() == want["granules"].tolist()
    assert np.allclose(got["sq_err"], want["sq_err"], rtol=1e-11, atol=0) and np.isclose(got["sq_sum"], want["sq_sum"], rtol=1e-11)


def test_probe_matches_oracle_on_mixed_pages():
    w = workloads.tiny(seed=4)
    pages = np.concatenate([w.gen_pages(np.arange(120)), gen.structured_pages(3, 40)])
    special = np.zeros((6, 2048), np.uint16)
    special[1] = np.full(2048, 3.5, np.float16).view(np.uint16)
    special[2] = (np.arange(2048) % 1024).astype(np.uint16)               # subnormals only
    special[3, 0::2], special[3, 1::2] = 0x7BFF, 0xFBFF                   # +-65504
    special[4] = pages[0]; special[4, 100] = 0x7C00                       # Inf: skipped
    special[5] = pages[1]; special[5, 7] = 0xFE00                         # NaN: skipped
    pages = np.concatenate([pages, special])
    idx = np.concatenate([np.random.default_rng(0).permutation(len(pages)), [len(pages) + 3, 5, 5]])
    want = O.probe_pages(pages, idx)[0]
    got = _gpu_probe(pages, idx)
    _same(got, want)
    assert int(got["nonfinite"]) == 2 and int(got["bad_index"]) == 1 and int(got["pages"]) == len(pages)


def test_selection_matches_oracle_and_follows_the_layers():
    """Six layers: 0-1 built from constant-slope segments (long runs, the early-layer shape the paper reports as
    3-4x), 2-5 Gaussian with outlier channels in K.  Per layer: probe 256 sampled pages, select, compress the
    layer with the selected scheme on both sides, compare everything; then fetch everything back."""
    from paper_2512_11920_b200 import select_scheme
    w = workloads.llama70b(seed=17, n_layers=6, batch=2, seq=512)
    pr = Pair.for_workload(w)
    rng = np.random.default_rng(1)
    chosen = []
    for layer in range(w.n_layers):
        slots = w.layer_slots(layer)
        pages = gen.structured_pages(100 + layer, len(slots)) if layer < 2 else w.gen_pages(slots)
        sample = rng.permutation(len(slots))[:256]
        want = O.probe_pages(pages, sample)[0]
        got = _gpu_probe(pages, sample)
        _same(got, want)
        for pol in ((1.0, 0.05, 1.0, 30.0), (1.0, 0.0, 1.0, 0.0), (1.0, 0.05, 1.0, 45.0), (0.0, 1.0, 0.0, 0.0), (1.0, 0.05, 1.0, 300.0)):
            s_gpu, j_gpu = select_scheme(got, *pol, COST)
            s_cpu, j_cpu = O.select_scheme(got, O.make_policy(*pol, COST))               # the same numbers on both sides
            assert s_gpu == s_cpu and np.array_equal(j_gpu, j_cpu), (layer, pol)
        scheme, _ = select_scheme(got, 1.0, 0.05, 1.0, 30.0, COST)
        chosen.append(scheme)
        pr.compress(pages, np.arange(len(slots)), slots, scheme)
    pr.check_state()
    assert all(c in (3, 19) for c in chosen[:2]) and all(c in (1, 17) for c in chosen[2:]), chosen
    stats = pr.gpu.stats()
    assert stats["pages_mode"][3] == 2 * w.pages_per_layer and stats["pages_mode"][1] == 4 * w.pages_per_layer
    for layer in range(w.n_layers):
        pr.gather(layer, w.block_table, w.seq_lens, w.dst_tok_off())
    pr.check_state()
    pr.close()


def test_argument_errors():
    import torch
    from paper_2512_11920_b200 import probe_pages, select_scheme, SpeckvError, PROBE_DTYPE
    acc = torch.zeros(PROBE_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    probe_pages(torch.zeros(2048, dtype=torch.int16, device="cuda"), torch.zeros(0, dtype=torch.int32, device="cuda"), acc)   # n = 0
    with pytest.raises(SpeckvError):
        select_scheme(np.zeros(1, PROBE_DTYPE), 1.0, 0.0, 0.0, 0.0, COST)                 # empty sample
