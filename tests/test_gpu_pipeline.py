"""speckv_pipeline_layers / speckv_pipeline_attend: the multi-layer pipelined prefetch of Sec. 3.4.4.

Gathers run ahead on the context's fetch stream into a ring of workspaces that is smaller than the number
of layers; the per-layer computation runs on the caller's stream.  If an ordering edge were missing (a slot
refilled while its layer is still being read, a layer computed before its pages have arrived) the outputs
would differ from the oracle's, which computes every layer from the pool directly."""
import numpy as np
import pytest

from kvgen import workloads
from oracle import oracle as O
from tests.parity_util import Pair

pytestmark = pytest.mark.gpu


def _filled(w, schemes):
    pr = Pair.for_workload(w)
    for layer in range(w.n_layers):
        slots = w.layer_slots(layer)
        pr.compress(w.gen_pages(slots), np.arange(len(slots)), slots, schemes[layer % len(schemes)])
    return pr


def _vmax(pr, w, layer):
    seq_lens, tpad, tok = pr._layout(w.seq_lens)
    d = np.zeros(int(tpad.sum()) * 2 * w.n_kv_heads * 128, np.uint16)
    l2 = np.zeros(w.batch * 4 * 2 * w.n_kv_heads * 2048, np.uint16)
    scratch = O.Pool.__new__(O.Pool)
    scratch.__dict__.update(pr.cpu.__dict__)
    scratch.status, scratch.stats, scratch.l2_tag = O.Status(), O.Stats(), pr.cpu.l2_tag.copy()
    scratch.decompress_gather(layer, w.block_table, seq_lens, tok, None, d, l2)
    return pr._vmax(d, seq_lens, tpad, tok)


@pytest.mark.parametrize("ring_slots", [3, 2, 1])
def test_pipelined_attention_over_eight_layers_equals_the_oracle_layer_by_layer(ring_slots):
    """70B shape (8 KV heads, 64 query heads), 8 layers, a ring of 3, 2 or 1 workspaces; repeated so that
    a late gather of one pass can collide with the next pass if the start edge were missing."""
    import torch
    w = workloads.llama70b(seed=31, n_layers=8, batch=6, seq=1024)
    w.seq_lens = np.array([1024, 700, 16, 1, 333, 1000], np.uint32)
    pr = _filled(w, [3, 19, 1, 4])
    L, B, Hq = w.n_layers, w.batch, 64
    rng = np.random.default_rng(5)
    q = (rng.standard_normal((L, B, Hq, 128)) * 2).astype(np.float16)
    seq_lens, tpad, tok = pr._layout(w.seq_lens)
    want = [pr.cpu.attend(l, w.block_table, seq_lens, q[l].view(np.uint16), Hq) for l in range(L)]
    vmax = [_vmax(pr, w, l) for l in range(L)]
    slot_tokens = int(tpad.sum())
    ring = torch.empty(ring_slots * slot_tokens * 2 * w.n_kv_heads * 128, dtype=torch.int16, device="cuda")
    ws = torch.empty(pr.gpu.attend_workspace_bytes(B), dtype=torch.uint8, device="cuda")
    qd = torch.from_numpy(q).cuda()
    bt, lens, tokd = pr.t(w.block_table), pr.t(seq_lens), pr.t(tok)
    for rep in range(5):
        out = torch.full((L, B, Hq, 128), float("nan"), dtype=torch.float16, device="cuda")
        ring.fill_(0x7E00)                                        # NaN patterns: a layer computed too early shows
        pr.gpu.pipeline_attend(0, L, bt, lens, tokd, ring, ring_slots, qd, out, ws)
        got = out.cpu().numpy()
        for l in range(L):
            pr._attend_check(got[l], want[l], vmax[l], Hq // w.n_kv_heads, f"pipelined attention, layer {l}, pass {rep}")
    assert sum(pr.gpu.status()["count"]) == 0
    pr.close()


def test_pipeline_with_a_callers_own_layer_function_and_a_layer_range():
    """The general entry: the per-layer work is the caller's (here: copy the first page of the workspace and
    run the library's attention), layers 2..6 of 8 only, ring of 2."""
    import torch
    w = workloads.llama70b(seed=32, n_layers=8, batch=3, seq=256)
    pr = _filled(w, [3])
    B, Hq = w.batch, 16
    q = np.random.default_rng(6).standard_normal((B, Hq, 128)).astype(np.float16)
    seq_lens, tpad, tok = pr._layout(w.seq_lens)
    slot_tokens = int(tpad.sum())
    elems = slot_tokens * 2 * w.n_kv_heads * 128
    ring = torch.zeros(2 * elems, dtype=torch.int16, device="cuda")
    ws = torch.empty(pr.gpu.attend_workspace_bytes(B), dtype=torch.uint8, device="cuda")
    qd = torch.from_numpy(q).cuda()
    lens_d, tok_d = pr.t(seq_lens), pr.t(tok)
    outs, firsts, seen = {}, {}, []

    def consume(layer, kv_ptr, stream_ptr):
        slot = (kv_ptr - ring.data_ptr()) // (elems * 2)
        assert stream_ptr == torch.cuda.current_stream().cuda_stream
        seen.append((layer, slot))
        view = ring[slot * elems:(slot + 1) * elems]
        firsts[layer] = view[:2048].clone()
        outs[layer] = torch.empty(B, Hq, 128, dtype=torch.float16, device="cuda")
        pr.gpu.attend_dense(view, lens_d, tok_d, qd, outs[layer], ws)

    pr.gpu.pipeline_layers(2, 5, pr.t(w.block_table), lens_d, tok_d, ring, 2, consume)
    torch.cuda.synchronize()
    assert seen == [(2, 0), (3, 1), (4, 0), (5, 1), (6, 0)]
    for layer in range(2, 7):
        want = pr.cpu.attend(layer, w.block_table, seq_lens, q.view(np.uint16), Hq)
        pr._attend_check(outs[layer].cpu().numpy(), want, _vmax(pr, w, layer), Hq // w.n_kv_heads, f"layer {layer}")
        slot0 = ((layer * w.blocks_per_layer + int(w.block_table[0][0])) * 2 + 0) * w.n_kv_heads + 0
        rc, page = O.decompress_record(O.compress_page(w.gen_pages([slot0])[0], 3))
        assert rc == 0 and np.array_equal(firsts[layer].cpu().numpy().view(np.uint16), page)
    # a failing layer function ends the call with its error
    with pytest.raises(ZeroDivisionError):
        pr.gpu.pipeline_layers(0, 3, pr.t(w.block_table), lens_d, tok_d, ring, 2, lambda *a: 1 // 0)
    torch.cuda.synchronize()
    pr.close()
