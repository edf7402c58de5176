#!/usr/bin/env python
"""Benchmark of the speckv hot path: compress, then decompress+gather, over a KV cache.

A step = one pass of the whole hot path over the workload: every layer is compressed
(speckv_compress, scheme INT8+delta+RLE, one call over the page list of the whole cache) and then every layer is fetched
back through block table and page table (speckv_decompress_gather, one call per layer).
Inputs are seeded synthetic K/V, resident in HBM and far larger than L2.  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--layers L]

With --gpus N > 1 (under torchrun) every rank runs an independent replica on its own GPU:
pages are independent units and the path has no exchange step, so there is no collective.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from kvgen import workloads  # noqa: E402

METRIC = "compress & decompress+gather GB/s (uncompressed KV)"
PAGE = 4096


# DRAM bytes per page (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture, divided by the
# pages of that launch; see profiles/), valid only for the kernel sources they were captured from.
NCU_TRAFFIC = {
    "speckv_compress": {"bytes_per_page": 6281.2, "sources": ["compress.cu", "async_ptx.cuh", "speckv_dev.cuh"], "sha1": "7897d4c1a5d75e099104426be54e8dfea1e8346b"},
    "speckv_decompress_gather": {"bytes_per_page": 5579.5, "sources": ["gather.cu", "decode.cuh", "async_ptx.cuh", "speckv_dev.cuh"], "sha1": "23e3782040c977f97380f6469fb4665f084055e3"},
}


def kernel_source_hash(files):
    import hashlib
    h = hashlib.sha1()
    for f in files:
        with open(os.path.join(ROOT, "paper_2512_11920_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic(kernel: str, pages_per_launch: int):
    """DRAM traffic of one launch from the committed ncu capture, or None if the kernel changed since."""
    rec = NCU_TRAFFIC[kernel]
    if rec["bytes_per_page"] is None or kernel_source_hash(rec["sources"]) != rec["sha1"]:
        return None
    return rec["bytes_per_page"] * pages_per_launch


def measured_peak_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i",
                                          str(self.index), "-lms", "50"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i].lower() == "active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


class Bench:
    """Device-resident state of one replica: source K/V, context, index tensors, destination."""

    def __init__(self, w, dev, scheme=3):
        import torch
        from kvgen import device as gen_device
        from paper_2512_11920_b200 import Context
        self.torch, self.w, self.dev, self.scheme = torch, w, dev, scheme
        ppl = w.pages_per_layer
        self.pages = w.n_layers * ppl
        self.src = torch.empty(self.pages * 2048, dtype=torch.int16, device=dev)
        self.scales = torch.from_numpy(w.scales).to(dev)
        for l in range(w.n_layers):
            gen_device.fill(self.src[l * ppl * 2048:(l + 1) * ppl * 2048], w.seed, l * ppl, ppl, self.scales, ppl, w.n_kv_heads)
        pool_bytes = ((self.pages * (4160 if (scheme & 15) == 0 else 2368) + (64 << 20)) // 64) * 64   # largest record per page
        self.ctx = Context(w.n_layers, w.n_kv_heads, w.blocks_per_layer, w.max_blocks_per_seq, w.batch, pool_bytes)
        # compress lists a layer's pages in physical slot order (source and page table share the numbering)
        self.idx_all = torch.arange(self.pages, dtype=torch.int32, device=dev)
        self.idx = [self.idx_all[l * ppl:(l + 1) * ppl] for l in range(w.n_layers)]
        self.bt = torch.from_numpy(w.block_table).to(dev)
        self.lens = torch.from_numpy(w.seq_lens.view(np.int32)).to(dev)
        self.tok = torch.from_numpy(w.dst_tok_off().view(np.int64)).to(dev)
        self.layer_elems = w.demand_tokens() * 2 * w.n_kv_heads * 128
        self.dst = torch.empty(w.n_layers * self.layer_elems, dtype=torch.int16, device=dev)
        self.demand_pages = w.demand_tokens() // 16 * 2 * w.n_kv_heads * w.n_layers
        torch.cuda.synchronize()

    def dst_layer(self, l):
        return self.dst[l * self.layer_elems:(l + 1) * self.layer_elems]

    def step(self, ev=None):
        """One pass of the hot path; ev = (e0, e1, e2) CUDA events recorded around the two phases."""
        w, c = self.w, self.ctx
        c.reset()
        if ev:
            ev[0].record()
        c.compress(self.src, self.idx_all, self.idx_all, self.scheme)
        if ev:
            ev[1].record()
        for l in range(w.n_layers):
            c.decompress_gather(l, self.bt, self.lens, self.tok, self.dst_layer(l))
        if ev:
            ev[2].record()

    def launches_per_step(self):
        return 1 + self.w.n_layers

    # ---- the consumer: decode-step attention per layer ---------------------------------------
    def consumer(self, n_q_heads: int, reps: int = 3):
        """Per-layer decode-step attention over the whole cache, three ways: (serial) gather a layer, then
        attend over the gathered workspace, one stream; (pipelined) the multi-layer prefetch pipeline of
        Sec. 3.4.4: gathers run up to two layers ahead on a second stream, into a ring of three workspaces;
        (fused) attention straight from the compressed pages.  Returns milliseconds per pass over all layers."""
        torch, w, c = self.torch, self.w, self.ctx
        L, B = w.n_layers, w.batch
        g = torch.Generator(device=self.dev).manual_seed(7)
        q = torch.randn(B, n_q_heads, 128, device=self.dev, generator=g).to(torch.float16)
        out = torch.empty_like(q)
        ws = torch.empty(c.attend_workspace_bytes(B), dtype=torch.uint8, device=self.dev)
        R = min(3, L)                                   # workspaces in flight: the layer being attended and two ahead
        ring = [self.dst_layer(i) for i in range(R)]
        ev = lambda: torch.cuda.Event(enable_timing=True)

        def timed(fn):
            fn()
            torch.cuda.synchronize()
            e0, e1 = ev(), ev()
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps

        def gather_only():
            for l in range(L):
                c.decompress_gather(l, self.bt, self.lens, self.tok, ring[l % R])

        def attend_only():
            for l in range(L):
                c.attend_dense(ring[l % R], self.lens, self.tok, q, out, ws)

        def serial():
            for l in range(L):
                c.decompress_gather(l, self.bt, self.lens, self.tok, ring[l % R])
                c.attend_dense(ring[l % R], self.lens, self.tok, q, out, ws)

        def fused():
            for l in range(L):
                c.decompress_attend(l, self.bt, self.lens, q, out, ws)

        side = torch.cuda.Stream(device=self.dev)
        main = torch.cuda.current_stream()

        def pipelined():
            gathered = [torch.cuda.Event() for _ in range(L)]
            attended = [torch.cuda.Event() for _ in range(L)]
            start = torch.cuda.Event()
            start.record(main)
            side.wait_event(start)
            for l in range(L):
                if l >= R:
                    side.wait_event(attended[l - R])            # the ring slot is free again
                with torch.cuda.stream(side):
                    c.decompress_gather(l, self.bt, self.lens, self.tok, ring[l % R])
                    gathered[l].record(side)
                main.wait_event(gathered[l])
                c.attend_dense(ring[l % R], self.lens, self.tok, q, out, ws)
                attended[l].record(main)

        res = {"n_q_heads": n_q_heads, "layers": L,
               "gather_ms": timed(gather_only), "attend_dense_ms": timed(attend_only), "serial_ms": timed(serial),
               "pipelined_ms": timed(pipelined), "fused_ms": timed(fused)}
        kv_bytes = self.demand_pages * PAGE
        t_layer, t_pref = res["attend_dense_ms"] / L, res["gather_ms"] / L
        res["t_effective_model_ms"] = res["attend_dense_ms"] + max(t_pref - 2 * t_layer, 0.0)
        res["kv_gbs"] = {k[:-3]: kv_bytes / (res[k] * 1e-3) / 1e9 for k in ("attend_dense_ms", "serial_ms", "pipelined_ms", "fused_ms")}
        return res

    # ---- pool lifecycle: compaction after rewrites ------------------------------------------
    def lifecycle(self, reps: int = 3):
        """Half of the cache is written twice (the first copies become garbage), then the log is compacted."""
        torch, c = self.torch, self.ctx
        half = self.idx_all[:self.pages // 2]
        scratch = torch.empty(c.compact_scratch_bytes(), dtype=torch.uint8, device=self.dev)
        ms = []
        for _ in range(reps):
            c.reset()
            c.compress(self.src, half, half, self.scheme)
            c.compress(self.src, half, half, self.scheme)
            torch.cuda.synchronize()
            before = c.cursor()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            c.compact(scratch)
            e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        after = c.cursor()
        t = float(np.median(ms))
        return {"log_gib_before": before * 64 / 2 ** 30, "log_gib_after": after * 64 / 2 ** 30, "compact_ms": t,
                "live_gbs": after * 64 / (t * 1e-3) / 1e9, "status_counts": c.status()["count"]}

    # ---- end to end through the host-buffer entry points --------------------------------
    def e2e(self, steps: int, ring: int = 4):
        """The same step through the host-buffer entry points: every layer's pages come from pinned host memory
        and every layer's gathered K/V goes back to pinned host memory.  Uploads + compression run on one
        stream, gathers + downloads on a second one that follows layer by layer (an event per layer), so the
        two directions of the host link are busy at the same time."""
        torch, w, c = self.torch, self.w, self.ctx
        ppl = w.pages_per_layer
        ring = min(ring, w.n_layers)
        h_in = torch.empty(ring * ppl * 2048, dtype=torch.int16).pin_memory()
        h_out = torch.empty(ring * self.layer_elems, dtype=torch.int16).pin_memory()
        h_in.copy_(self.src[:ring * ppl * 2048])
        staging = torch.empty(ring * ppl * 2048, dtype=torch.int16, device=self.dev)
        local = torch.arange(ppl, dtype=torch.int32, device=self.dev)
        up, down = torch.cuda.Stream(device=self.dev), torch.cuda.Stream(device=self.dev)
        main = torch.cuda.current_stream()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(main)
        up.wait_event(e0)
        down.wait_event(e0)
        for _ in range(steps):
            with torch.cuda.stream(up):
                up.wait_stream(down)                     # the previous step's gathers are done with the pool
                c.reset()
            done = [torch.cuda.Event() for _ in range(w.n_layers)]
            for l in range(w.n_layers):
                r = l % ring
                with torch.cuda.stream(up):
                    c.compress_host(h_in[r * ppl * 2048:(r + 1) * ppl * 2048], staging[r * ppl * 2048:(r + 1) * ppl * 2048],
                                    local, self.idx[l], self.scheme)
                    done[l].record(up)
                with torch.cuda.stream(down):
                    down.wait_event(done[l])
                    c.decompress_gather_host(l, self.bt, self.lens, self.tok, self.dst_layer(l),
                                             h_out[r * self.layer_elems:(r + 1) * self.layer_elems])
        main.wait_stream(up)
        main.wait_stream(down)
        e1.record(main)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        h2d = w.n_layers * ppl * PAGE
        d2h = w.n_layers * self.layer_elems * 2
        # what came back for the last layers is what the device holds, and every page went both ways
        stats, status = c.stats(), c.status()
        last = w.n_layers - 1
        same = bool((h_out[(last % ring) * self.layer_elems:(last % ring + 1) * self.layer_elems] == self.dst_layer(last).cpu()).all())
        if not same or sum(status["count"]) or sum(stats["pages_mode"]) != self.pages or stats["pages_decoded"] != self.demand_pages:
            raise RuntimeError(f"end-to-end step inconsistent: {stats} {status} host copy equal: {same}")
        return ms, h2d, d2h

    # ---- sampled parity at the benchmarked size -------------------------------------------
    def sampled_parity(self, n_samples: int = 48, seed: int = 123):
        """Sampled pages: record bytes, PTE and gathered fp16 against the CPU oracle."""
        from oracle import oracle as O
        torch, w = self.torch, self.w
        rng = np.random.default_rng(seed)
        H, ppl = w.n_kv_heads, w.pages_per_layer
        pte = self.ctx.pte_view().view(torch.int64)
        pool = self.ctx.pool_view()
        bad = 0
        for _ in range(n_samples):
            l = int(rng.integers(w.n_layers)); b = int(rng.integers(w.batch))
            n = int(rng.integers((int(w.seq_lens[b]) + 15) // 16)); kv = int(rng.integers(2)); h = int(rng.integers(H))
            slot = ((l * w.blocks_per_layer + int(w.block_table[b][n])) * 2 + kv) * H + h
            page = w.gen_pages([slot])[0]
            rec = O.compress_page(page, self.scheme)
            e = int(pte[slot].item()) & 0xFFFFFFFFFFFFFFFF
            off, rec_len, mode, valid = (e & 0xFFFFFFFF) * 64, (e >> 32) & 0xFFFF, (e >> 48) & 0xFF, (e >> 56) & 1
            got_rec = pool[off:off + ((len(rec) + 63) // 64) * 64].cpu().numpy().tobytes()
            want_rec = rec + bytes(-len(rec) % 64)
            rc, xh = O.decompress_record(rec)
            tpad = ((int(w.seq_lens[b]) + 15) // 16) * 16
            el = int(w.dst_tok_off()[b]) * 2 * H * 128 + ((kv * H + h) * tpad + 16 * n) * 128
            got_page = self.dst_layer(l)[el:el + 2048].cpu().numpy().view(np.uint16)
            ok = valid == 1 and rec_len == len(rec) and mode == rec[6] and got_rec == want_rec and rc == 0 and \
                np.array_equal(got_page, xh)
            bad += 0 if ok else 1
        return {"pages_checked": n_samples, "mismatches": bad}


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the time)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_gbs(bytes_per_replica: int, world: int, ms_per_step: float) -> float:
    """Replicas only: every rank processes the same number of bytes, the job's rate is their sum."""
    return world * bytes_per_replica / (ms_per_step * 1e-3) / 1e9


def run_decode_fetch(args, w, dev):
    """--workload decode-fetch-7b: the decode-step paged fetch (7B shape, 64 sequences with lognormal lengths,
    block table a random permutation of a 2M-page pool per layer).  The pool is filled once (untimed); then
    every decode step is one speckv_decompress_gather over the pages touched plus a prefetch list of the next
    1-4 blocks per sequence.  One JSON line: aggregate and per-step GB/s of uncompressed K/V delivered."""
    import torch
    from kvgen import device as gen_device
    from paper_2512_11920_b200 import Context
    H, L, ppl = w.n_kv_heads, w.n_layers, w.pages_per_layer
    n_pop = len(w.mapped_blocks()) * 2 * H
    ctx = Context(L, H, w.blocks_per_layer, w.max_blocks_per_seq, w.batch, ((L * n_pop * 2368) // 64 + 1024) * 64)
    src = torch.empty(ppl * 2048, dtype=torch.int16, device=dev)
    scales = torch.from_numpy(w.scales).to(dev)
    local = torch.from_numpy(w.layer_slots(0).view(np.int32)).to(dev)
    for layer in range(L):
        gen_device.fill(src, w.seed, layer * ppl, ppl, scales, ppl, H)
        ctx.compress(src, local, local + layer * ppl, args.scheme)
    torch.cuda.synchronize()
    del src
    bt = torch.from_numpy(w.block_table).to(dev)
    max_tok = int(sum(((min(int(l) + w.steps, 16 * w.max_blocks_per_seq) + 15) // 16) * 16 for l in w.seq_lens))
    dst = torch.empty(max_tok * 2 * H * 128, dtype=torch.int16, device=dev)
    l2 = torch.empty(w.batch * 4 * 2 * H * 2048, dtype=torch.int16, device=dev)
    steps = []
    for s in range(w.steps):                                  # every step's inputs resident before the clock starts
        layer, lens, pf = workloads.decode_step(w, s)
        steps.append((layer, torch.from_numpy(lens.view(np.int32)).to(dev), torch.from_numpy(w.dst_tok_off(lens).view(np.int64)).to(dev),
                      torch.from_numpy(pf.view(np.uint8)).to(dev) if len(pf) else None,
                      int(((lens.astype(np.int64) + 15) // 16).sum()) * 2 * H))

    def one_pass(evs=None):
        ctx.l2_tag_view().zero_()                             # residency as at the start of the decode loop
        for i, (layer, lens, tok, pf, _) in enumerate(steps):
            if evs:
                evs[i][0].record()
            ctx.decompress_gather(layer, bt, lens, tok, dst, pf, l2)
            if evs:
                evs[i][1].record()

    for _ in range(max(args.warmup, 3)):
        one_pass()
    torch.cuda.synchronize()
    ctx.clear_status()
    st0 = ctx.stats()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    passes = max(1, args.steps // 10)
    evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in steps] for _ in range(passes)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for p in range(passes):
        one_pass(evs[p])
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    st1, status = ctx.stats(), ctx.status()
    pages = st1["pages_decoded"] - st0["pages_decoded"]
    total_ms = t0.elapsed_time(t1)
    per_step = np.array([[steps[i][4] * PAGE / (evs[p][i][0].elapsed_time(evs[p][i][1]) * 1e-3) / 1e9 for i in range(len(steps))]
                         for p in range(passes)])
    out = {"metric": METRIC, "value": pages * PAGE / (total_ms * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": 1, "steps": passes * len(steps),
           "warmup": max(args.warmup, 3) * len(steps), "ms_per_step": total_ms / (passes * len(steps)), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f16->i8", "data": "synthetic",
           "config": {"workload": w.name, "layers": L, "kv_heads": H, "batch": w.batch, "decode_steps_per_pass": len(steps),
                      "passes": passes, "scheme": args.scheme, "calls_per_step": 1, "timed": "decompress+gather only (the pool is filled before)",
                      "l2": "each step reads other records than the one before (a different layer); 1.3-1.6 GiB per step"},
           "gpu_launches": passes * len(steps), "clocks": clocks,
           "per_step_demand_gbs": {"min": float(per_step.min()), "median": float(np.median(per_step)), "max": float(per_step.max())},
           "pages_delivered": pages, "prefetch": {"issued": st1["pf_issued"] - st0["pf_issued"], "skipped_resident": st1["pf_skipped"] - st0["pf_skipped"]},
           "status_counts": status["count"]}
    ctx.close()
    return out


def run_managed_prefetch(args, w, dev):
    """--workload managed-prefetch-7b: decode steps through speckv_prefetch_step (7B shape, 64 sequences with
    lognormal lengths, block table a random permutation of the pool).  Every step of every layer reads 1-4 blocks
    per sequence and hands in the predictions for the next step (a stand-in predictor that is right 95 % of the
    time, the paper's top-4 accuracy); reads found in the readable bank are served from the buffer, the others
    are fetched synchronously, and the other bank is refilled at the depth the UCB rule picks.  One JSON line:
    GB/s of K/V delivered, time per step, and the rows of the paper's prefetch-statistics table."""
    import torch
    from kvgen import device as gen_device
    from paper_2512_11920_b200 import Context
    from paper_2512_11920_b200.binding import PF_SEQ_DTYPE, PF_COUNTER_NAMES
    H, L, ppl, B = w.n_kv_heads, w.n_layers, w.pages_per_layer, w.batch
    n_pop = len(w.mapped_blocks()) * 2 * H
    ctx = Context(L, H, w.blocks_per_layer, w.max_blocks_per_seq, B, ((L * n_pop * 2368) // 64 + 1024) * 64)
    src = torch.empty(ppl * 2048, dtype=torch.int16, device=dev)
    scales = torch.from_numpy(w.scales).to(dev)
    local = torch.from_numpy(w.layer_slots(0).view(np.int32)).to(dev)
    for layer in range(L):
        gen_device.fill(src, w.seed, layer * ppl, ppl, scales, ppl, H)
        ctx.compress(src, local, local + layer * ppl, args.scheme)
    torch.cuda.synchronize()
    del src
    visits, accuracy, beta = 100, 0.95, 0.3
    access, cand = workloads.prefetch_trace(w, visits, seed=0, accuracy=accuracy)
    access_d, cand_d = torch.from_numpy(access).to(dev), torch.from_numpy(cand).to(dev)
    bt = torch.from_numpy(w.block_table).to(dev)
    state = torch.zeros(L, B * 80, dtype=torch.uint8, device=dev)          # one set of depth statistics per layer
    cnt = torch.zeros(10, dtype=torch.int64, device=dev)
    l2 = torch.empty(L, 2 * B * 4 * 2 * H * 2048, dtype=torch.int16, device=dev)
    miss = torch.empty(B * 4 * 2 * H * 2048, dtype=torch.int16, device=dev)
    where = torch.empty(L, B, 4, dtype=torch.int32, device=dev)

    def one_pass():
        state.zero_()
        cnt.zero_()
        for v in range(visits):
            for layer in range(L):
                ctx.prefetch_step(layer, v & 1, bt, access_d[v], cand_d[v], beta, state[layer], cnt, l2[layer], miss, where[layer])

    for _ in range(max(args.warmup, 3)):
        one_pass()
    torch.cuda.synchronize()
    passes = max(1, args.steps // 10)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(passes):
        one_pass()
    t1.record()
    torch.cuda.synchronize()
    eager_ms = t0.elapsed_time(t1)                            # call by call from the host: bound by the host's launch rate
    # A pass is 400 short calls: captured once as a CUDA graph and replayed, so that the device time is what is timed
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        one_pass()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    ctx.clear_status()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    t0.record()
    for _ in range(passes):
        graph.replay()
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    total_ms = t0.elapsed_time(t1)
    c = dict(zip(PF_COUNTER_NAMES, (int(x) for x in cnt.cpu().numpy())))      # one pass (the counters are reset per pass)
    depth = np.bincount(state.cpu().numpy().view(PF_SEQ_DTYPE)["depth"].reshape(-1), minlength=5)[1:5]
    n_calls = passes * visits * L
    out = {"metric": METRIC, "value": passes * c["pages"] * PAGE / (total_ms * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": 1,
           "steps": n_calls, "warmup": max(args.warmup, 3) * visits * L, "ms_per_step": total_ms / n_calls, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f16->i8", "data": "synthetic",
           "config": {"workload": "managed-prefetch-7b", "layers": L, "kv_heads": H, "batch": B, "decode_steps_per_pass": visits,
                      "passes": passes, "scheme": args.scheme, "calls_per_step": 1, "predictor_accuracy": accuracy, "beta": beta,
                      "timed": "speckv_prefetch_step only (the pool is filled before), one pass replayed as a CUDA graph; reads per sequence and step: 1-4 blocks",
                      "l2": "each call reads other records than the one before (a different layer)"},
           "gpu_launches": 2 * n_calls, "clocks": clocks, "eager_ms_per_step": eager_ms / n_calls,
           "prefetch": {"hit_rate": c["hits"] / max(c["accesses"], 1), "coverage": (c["hits"] + c["late"]) / max(c["accesses"], 1),
                        "precision": c["evicted_used"] / max(c["evicted"], 1), "counters": {k: v for k, v in c.items() if k != "rsvd"},
                        "final_depths_1_to_4": [int(x) for x in depth],
                        "paper_table": {"hit_rate": 0.947, "coverage": 0.963, "precision": 0.872,
                                        "note": "LLaMA-2 70B chatbot trace with the paper's LSTM predictor: context, not a target"}},
           "status_counts": ctx.status()["count"]}
    ctx.close()
    return out


def oracle_pages(w, n_pages: int, use_gpu_gen: bool):
    """The first n_pages of layer 0 on the host (generated on the GPU when there is one: same values, faster)."""
    if use_gpu_gen:
        import torch
        from kvgen import device as gen_device
        buf = torch.empty(n_pages * 2048, dtype=torch.int16, device="cuda")
        gen_device.fill(buf, w.seed, 0, n_pages, torch.from_numpy(w.scales).cuda(), w.pages_per_layer, w.n_kv_heads)
        return buf.cpu().numpy().view(np.uint16).reshape(n_pages, 2048)
    return w.gen_pages(np.arange(n_pages, dtype=np.uint32))


def oracle_sample(w, src, n_threads: int = 1):
    """Times the CPU oracle, as it stands, on the pages `src` (a multiple of 2*H pages per thread): compress
    into a one-layer pool, then decompress+gather them as one long sequence whose block i is physical block i.
    With n_threads > 1 the pages are split evenly and every thread runs the same two calls on a pool of its
    own (the oracle itself is single-threaded; its C calls release the interpreter lock).
    Returns (seconds_compress, seconds_gather, bytes): the slowest thread's time per phase."""
    import threading
    from oracle import oracle as O
    H = w.n_kv_heads
    per = (len(src) // n_threads) // (2 * H) * (2 * H)
    assert per > 0
    nblk = per // (2 * H)
    slots = np.arange(per, dtype=np.uint32)
    bt = np.arange(nblk, dtype=np.int32).reshape(1, nblk)
    pools = [O.Pool(1, H, nblk, nblk, 1, per * 2368) for _ in range(n_threads)]
    dsts = [np.zeros(nblk * 16 * 2 * H * 128, np.uint16) for _ in range(n_threads)]
    l2 = [np.zeros(4 * 2 * H * 2048, np.uint16) for _ in range(n_threads)]
    O.lib()                                               # build/load before the clock starts

    def phase(fn):
        ths = [threading.Thread(target=fn, args=(t,)) for t in range(n_threads)]
        t0 = time.perf_counter()
        for th in ths:
            th.start()
        for th in ths:
            th.join()
        return time.perf_counter() - t0

    tc = phase(lambda t: pools[t].compress(src[t * per:(t + 1) * per], slots, slots, 3))
    tg = phase(lambda t: pools[t].decompress_gather(0, bt, [nblk * 16], [0], None, dsts[t], l2[t]))
    assert all(p.stats.pages_decoded == per for p in pools)
    return tc, tg, n_threads * per * PAGE


def run_reference(args, w):
    """--impl reference: the CPU oracle on the host cores, on a bounded sample per step."""
    have_gpu = False
    try:
        import torch
        have_gpu = torch.cuda.is_available() and os.path.exists(os.path.join(ROOT, "kvgen", "libkvgen.so"))
    except Exception:
        pass
    n_pages = 16384 if have_gpu else 2048
    n_pages -= n_pages % (2 * w.n_kv_heads)
    times = []
    src = oracle_pages(w, n_pages, have_gpu)
    for i in range(args.warmup + args.steps):
        tc, td, nbytes = oracle_sample(w, src)
        if i >= args.warmup:
            times.append(tc + td)
    ms = 1e3 * float(np.mean(times))
    value = 2 * nbytes / (ms * 1e-3) / 1e9
    sample = f"first {n_pages} pages of layer 0 ({n_pages * PAGE >> 20} MiB): compress, then decompress+gather"
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16->i8", "data": "synthetic", "config": {"workload": w.name, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="speckv", choices=["speckv", "reference"])
    ap.add_argument("--workload", default="llama2-70b-gqa", choices=["llama2-70b-gqa", "llama2-7b", "decode-fetch-7b", "managed-prefetch-7b"])
    ap.add_argument("--layers", type=int, default=0, help="use only this many layers (small cases for profiling)")
    ap.add_argument("--scheme", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-adaptive", action="store_true", help="skip the extra runs with the adaptive and grouped schemes")
    ap.add_argument("--consumer", type=int, default=-1, metavar="N_Q_HEADS",
                    help="also time decode-step attention over the cache with N_Q_HEADS query heads (serial, pipelined, "
                         "fused) and the log compaction after rewrites; -1 = the model's head count (64 for the 70B shape, else one "
                         "per KV head), 0 = skip both")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    kw = {"n_layers": args.layers} if args.layers else {}
    if args.workload == "managed-prefetch-7b":               # the decode-fetch shape, four layers resident unless --layers says otherwise
        w = workloads.decode_fetch(seed=0, n_layers=args.layers or 4)
    else:
        w = workloads.BY_NAME[args.workload](seed=0, **kw)

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args, w)), flush=True)
        return

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the speckv path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    if args.workload == "decode-fetch-7b":                    # its own line: one gather per decode step, demand + prefetch
        if rank == 0:
            print(json.dumps(run_decode_fetch(args, w, dev)), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return

    if args.workload == "managed-prefetch-7b":               # its own line: one speckv_prefetch_step per layer and decode step
        if rank == 0:
            print(json.dumps(run_managed_prefetch(args, w, dev)), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return

    b = Bench(w, dev, args.scheme)
    for _ in range(max(args.warmup, 3)):
        b.step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    end = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    for s in range(args.steps):
        b.step(evs[s])
    end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = evs[0][0].elapsed_time(end)
    comp_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    gath_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    total_ms, comp_ms, gath_ms = max_over_ranks([total_ms, comp_ms, gath_ms], dev)
    if world > 1:
        dist.barrier()
    ms_per_step = total_ms / args.steps

    stats, status = b.ctx.stats(), b.ctx.status()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- algorithmic bytes (per layer launch) ----------------------------------------------
    L, H = w.n_layers, w.n_kv_heads
    ppl, dpl = w.pages_per_layer, b.demand_pages // L
    gran_layer = stats["granules"] / L                       # counters were reset at the start of the last step
    comp_bytes = ppl * (PAGE + 8 + 8) + 64 * gran_layer
    gath_bytes = 64 * gran_layer * (dpl / ppl) + dpl * (8 + 4.0 / (2 * H) + PAGE)
    peak, peak_kind = measured_peak_gbs()
    comp_gbs_unc = b.pages * PAGE / (comp_ms * 1e-3) / 1e9
    gath_gbs_unc = b.demand_pages * PAGE / (gath_ms * 1e-3) / 1e9
    comp_hbm = comp_bytes * L / (comp_ms * 1e-3) / 1e9
    gath_hbm = gath_bytes * L / (gath_ms * 1e-3) / 1e9
    dom = "speckv_compress" if comp_ms >= gath_ms else "speckv_decompress_gather"
    dom_hbm = comp_hbm if comp_ms >= gath_ms else gath_hbm
    dom_pages = b.pages if comp_ms >= gath_ms else dpl          # pages per launch of the dominant kernel
    value = whole_job_gbs((b.pages + b.demand_pages) * PAGE, world, ms_per_step)

    out = {"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
           "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16->i8",
           "data": "synthetic",
           "config": {"workload": w.name, "layers": L, "kv_heads": H, "batch": w.batch, "seq": int(w.seq_lens.max()),
                      "pages": b.pages, "uncompressed_gib": b.pages * PAGE / 2 ** 30, "scheme": args.scheme,
                      "block_table": "seeded random permutation", "l2": "inputs larger than L2 (no flush)",
                      "parallelism": "replicas only" if world > 1 else "1 GPU", "calls_per_step": b.launches_per_step()},
           "gpu_launches": b.launches_per_step() * args.steps, "clocks": clocks,
           "kernels": {"speckv_compress": {"ms_per_step": comp_ms, "uncompressed_gbs": comp_gbs_unc, "hbm_gbs": comp_hbm,
                                           "hbm_frac_of_measured": comp_hbm / peak, "hbm_frac_of_8000": comp_hbm / 8000.0},
                       "speckv_decompress_gather": {"ms_per_step": gath_ms, "uncompressed_gbs": gath_gbs_unc, "hbm_gbs": gath_hbm,
                                                    "hbm_frac_of_measured": gath_hbm / peak, "hbm_frac_of_8000": gath_hbm / 8000.0}},
           "roofline": {"bound": "hbm", "kernel": dom, "achieved": dom_hbm, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                        "frac": dom_hbm / peak, "traffic": ncu_traffic(dom, dom_pages),
                        "algorithmic_bytes_per_launch": (comp_bytes * L) if comp_ms >= gath_ms else gath_bytes},
           "compression": {"stored_ratio": b.pages * PAGE / (64.0 * stats["granules"]) if stats["granules"] else None,
                           "pages_mode": stats["pages_mode"], "status_counts": status["count"]}}
    # The same step with other schemes, reported beside the headline (which keeps every stage of the
    # compression algorithm in both directions): INT8 only and INT8 + delta (the paper's ablation rows), the
    # adaptive scheme (per page the smaller of delta and delta+RLE), and one scale per group of 8 channels
    # instead of one per page.
    extras = {}
    if args.scheme == 3 and not args.no_adaptive:
        extras = {"int8_only": 1, "int8_delta": 2,             # the other rows of the paper's compression ablation
                  "adaptive_scheme": 4, "grouped_scales": 3 | 16, "grouped_scales_adaptive": 4 | 16}
    for name, scheme in extras.items():
        b.scheme = scheme
        for _ in range(3):
            b.step()
        evx = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(5)]
        for e in evx:
            b.step(e)
        torch.cuda.synchronize()
        cx = float(np.mean([e[0].elapsed_time(e[1]) for e in evx])); gx = float(np.mean([e[1].elapsed_time(e[2]) for e in evx]))
        stx = b.ctx.stats()
        out[name] = {"scheme": scheme, "compress_uncompressed_gbs": b.pages * PAGE / (cx * 1e-3) / 1e9,
                     "gather_uncompressed_gbs": b.demand_pages * PAGE / (gx * 1e-3) / 1e9,
                     "stored_ratio": b.pages * PAGE / (64.0 * stx["granules"]), "pages_mode": stx["pages_mode"]}
    b.scheme = args.scheme
    if args.consumer:
        b.step()
        n_q_heads = args.consumer if args.consumer > 0 else (64 if w.name == "llama2-70b-gqa" else w.n_kv_heads)
        out["consumer"] = b.consumer(n_q_heads)
    if args.consumer:
        out["lifecycle"] = b.lifecycle()
    if not args.no_e2e:
        ms, h2d, d2h = b.e2e(steps=1)
        out["e2e"] = {"value": (b.pages + b.demand_pages) * PAGE / (ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": ms,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    if world == 1 and not args.no_cpu_baseline:
        # the oracle leg: sampled parity of what the timed configuration wrote (and of the extra schemes),
        # then the oracle timed on a bounded sample
        b.step()
        torch.cuda.synchronize()
        out["parity"] = b.sampled_parity()
        for name, scheme in extras.items():
            b.scheme = scheme
            b.step()
            torch.cuda.synchronize()
            out[name]["parity"] = b.sampled_parity(n_samples=16, seed=5)
        b.scheme = args.scheme
        n_pages = min(4, w.n_layers) * w.pages_per_layer   # layers 0-3: about 10 s of single-thread CPU work
        src = oracle_pages(w, n_pages, True)
        tc, td, nbytes = oracle_sample(w, src)
        out["cpu_baseline"] = {"value": 2 * nbytes / (tc + td) / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
                               "sample": f"first {n_pages} pages (layers 0-{n_pages // w.pages_per_layer - 1}, {nbytes >> 20} MiB): compress {tc:.2f} s, "
                                         f"decompress+gather {td:.2f} s",
                               "compress_gbs": nbytes / tc / 1e9, "gather_gbs": nbytes / td / 1e9}
        cores = len(os.sched_getaffinity(0))
        if cores > 1:                                      # the same oracle on every host core, the sample split evenly
            tcm, tdm, nb = oracle_sample(w, src, cores)
            out["cpu_baseline"]["all_cores"] = {"value": 2 * nb / (tcm + tdm) / 1e9, "unit": "GB/s", "cores": cores,
                                                "compress_gbs": nb / tcm / 1e9, "gather_gbs": nb / tdm / 1e9,
                                                "sample": f"the same pages, {nb >> 20} MiB split over {cores} threads, one pool each"}
    print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
