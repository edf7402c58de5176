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

from kvgen import gen, workloads  # noqa: E402

METRIC = "compress & decompress+gather GB/s (uncompressed KV)"
PAGE = 4096


# DRAM bytes per page (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture, divided by the
# pages of that launch; see profiles/), valid only for the kernel sources they were captured from.
NCU_TRAFFIC = {
    "speckv_compress": {"bytes_per_page": 6291.3, "sources": ["compress.cu", "async_ptx.cuh", "speckv_dev.cuh"], "sha1": "4186d566e6b25b3f549b206c0aac3e1138572dc4"},
    "speckv_decompress_gather": {"bytes_per_page": 5592.5, "sources": ["gather.cu", "decode.cuh", "async_ptx.cuh", "speckv_dev.cuh"], "sha1": "d11adf968f6c876b5615329d9089c0dc26f1f3e9"},
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

    def __init__(self, w, dev, scheme=3, layer0=0, n_layers=None, pool_page_bytes=4160):
        """Layers [layer0, layer0 + n_layers) of workload w (default: all); the context numbers them from 0.
        pool_page_bytes: pool capacity per page (4,160 = every page stored raw; 2,368 = the largest packed record)."""
        import torch
        from kvgen import device as gen_device
        from paper_2512_11920_b200 import Context
        self.torch, self.w, self.dev, self.scheme = torch, w, dev, scheme
        self.layer0, self.L = layer0, (w.n_layers - layer0 if n_layers is None else n_layers)
        ppl = w.pages_per_layer
        self.pages = self.L * ppl
        self.src = torch.empty(self.pages * 2048, dtype=torch.int16, device=dev)
        self.scales = torch.from_numpy(w.scales).to(dev)
        self.fill_source()
        pool_bytes = ((self.pages * pool_page_bytes + (64 << 20)) // 64) * 64
        self.ctx = Context(self.L, w.n_kv_heads, w.blocks_per_layer, w.max_blocks_per_seq, w.batch, pool_bytes)
        # compress lists a layer's pages in physical slot order (source and page table share the numbering)
        self.idx_all = torch.arange(self.pages, dtype=torch.int32, device=dev)
        self.idx = [self.idx_all[l * ppl:(l + 1) * ppl] for l in range(self.L)]
        self.bt = torch.from_numpy(w.block_table).to(dev)
        self.lens = torch.from_numpy(w.seq_lens.view(np.int32)).to(dev)
        self.tok = torch.from_numpy(w.dst_tok_off().view(np.int64)).to(dev)
        self.layer_elems = w.demand_tokens() * 2 * w.n_kv_heads * 128
        self.dst = torch.empty(self.L * self.layer_elems, dtype=torch.int16, device=dev)
        self.demand_pages = w.demand_tokens() // 16 * 2 * w.n_kv_heads * self.L
        self.raw_idx = None                 # set by mixed(): the pages that take the bypass
        torch.cuda.synchronize()

    def fill_source(self):
        """Writes the workload's pages (w.data: Gaussian, or piecewise-linear rows) into the source tensor."""
        from kvgen import device as gen_device
        w, ppl = self.w, self.w.pages_per_layer
        for l in range(self.L):
            part = self.src[l * ppl * 2048:(l + 1) * ppl * 2048]
            if w.data == "runs":
                gen_device.fill_runs(part, w.seed, (self.layer0 + l) * ppl, ppl)
            else:
                gen_device.fill(part, w.seed, (self.layer0 + l) * ppl, ppl, self.scales, ppl, w.n_kv_heads)

    def mixed(self, fraction=0.3, seed=11):
        """Splits the page list: a seeded `fraction` of the pages is stored raw by a scheme-0 call (the share of
        the traffic that bypasses the codec, Sec. 3.5.3: alpha ~ 0.3), the rest by the configured scheme."""
        torch = self.torch
        g = torch.Generator(device=self.dev).manual_seed(seed)
        take = torch.rand(self.pages, device=self.dev, generator=g) < fraction
        self.raw_take = take
        self.raw_idx = self.idx_all[take].contiguous()
        self.packed_idx = self.idx_all[~take].contiguous()

    def dst_layer(self, l):
        return self.dst[l * self.layer_elems:(l + 1) * self.layer_elems]

    def step(self, ev=None):
        """One pass of the hot path; ev = (e0, e1, e2) CUDA events recorded around the two phases."""
        c = self.ctx
        c.reset()
        if ev:
            ev[0].record()
        if self.raw_idx is None:
            c.compress(self.src, self.idx_all, self.idx_all, self.scheme)
        else:
            c.compress(self.src, self.packed_idx, self.packed_idx, self.scheme)
            c.compress(self.src, self.raw_idx, self.raw_idx, 0)
        if ev:
            ev[1].record()
        for l in range(self.L):
            c.decompress_gather(l, self.bt, self.lens, self.tok, self.dst_layer(l))
        if ev:
            ev[2].record()

    def launches_per_step(self):
        return (1 if self.raw_idx is None else 2) + self.L

    # ---- the consumer: decode-step attention per layer ---------------------------------------
    def consumer(self, n_q_heads: int, reps: int = 3):
        """Per-layer decode-step attention over the whole cache, three ways: (serial) gather a layer, then
        attend over the gathered workspace, one stream; (pipelined) the multi-layer prefetch pipeline of
        Sec. 3.4.4: gathers run up to two layers ahead on a second stream, into a ring of three workspaces;
        (fused) attention straight from the compressed pages.  Returns milliseconds per pass over all layers."""
        torch, w, c = self.torch, self.w, self.ctx
        L, B = self.L, w.batch
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

        # the multi-layer pipelined prefetch is the library's own call: gathers two layers ahead on the context's
        # fetch stream into the ring of three workspaces, attention on this stream
        ring_t = self.dst[:R * self.layer_elems]
        q_all = q.unsqueeze(0).expand(L, B, n_q_heads, 128).contiguous()
        out_all = torch.empty_like(q_all)

        def pipelined():
            c.pipeline_attend(0, L, self.bt, self.lens, self.tok, ring_t, R, q_all, out_all, ws)

        res = {"n_q_heads": n_q_heads, "layers": L,
               "gather_ms": timed(gather_only), "attend_dense_ms": timed(attend_only), "serial_ms": timed(serial),
               "pipelined_ms": timed(pipelined), "fused_ms": timed(fused)}
        kv_bytes = self.demand_pages * PAGE
        t_layer, t_pref = res["attend_dense_ms"] / L, res["gather_ms"] / L
        # Sec. 3.4.4: T_effective = T_compute + max(T_prefetch - 2 T_layer, 0) per layer, with the two stages measured
        # alone; the paper's fetch engine is a device of its own, here both stages share one GPU's HBM and SMs
        res["t_effective_model_ms"] = res["attend_dense_ms"] + L * max(t_pref - 2 * t_layer, 0.0)
        res["t_effective_measured_ms"] = res["pipelined_ms"]
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
    def e2e(self, steps: int = 3, warmup: int = 1):
        """The same step through the host-buffer entry points: every layer's own pages come from pinned host
        memory (a host copy of the whole cache) and every layer's gathered K/V goes back to pinned host memory
        of its own.  Uploads + compression run on one stream, gathers + downloads on a second one that follows
        layer by layer (an event per layer), so the two directions of the host link are busy at the same time.
        If the host cannot pin two copies of the cache, a ring of four layers is recycled instead (said in the
        result).  Afterwards every layer's host copy is compared with what the device holds."""
        torch, w, c = self.torch, self.w, self.ctx
        ppl, L = w.pages_per_layer, self.L
        ring = L
        try:
            h_in = torch.empty(L * ppl * 2048, dtype=torch.int16, pin_memory=True)
            h_out = torch.empty(L * self.layer_elems, dtype=torch.int16, pin_memory=True)
        except RuntimeError:
            ring = min(4, L)
            h_in = torch.empty(ring * ppl * 2048, dtype=torch.int16, pin_memory=True)
            h_out = torch.empty(ring * self.layer_elems, dtype=torch.int16, pin_memory=True)
        h_in.copy_(self.src[:ring * ppl * 2048])
        n_stage = min(4, L)
        staging = torch.empty(n_stage * ppl * 2048, dtype=torch.int16, device=self.dev)
        local = torch.arange(ppl, dtype=torch.int32, device=self.dev)
        up, down = torch.cuda.Stream(device=self.dev), torch.cuda.Stream(device=self.dev)
        main = torch.cuda.current_stream()

        def one_step():
            with torch.cuda.stream(up):
                up.wait_stream(down)                     # the previous step's gathers are done with the pool
                c.reset()
            for l in range(L):
                r, g = l % ring, l % n_stage
                with torch.cuda.stream(up):
                    c.compress_host(h_in[r * ppl * 2048:(r + 1) * ppl * 2048], staging[g * ppl * 2048:(g + 1) * ppl * 2048],
                                    local, self.idx[l], self.scheme)
                    done = torch.cuda.Event()
                    done.record(up)
                with torch.cuda.stream(down):
                    down.wait_event(done)
                    c.decompress_gather_host(l, self.bt, self.lens, self.tok, self.dst_layer(l),
                                             h_out[r * self.layer_elems:(r + 1) * self.layer_elems])

        torch.cuda.synchronize()
        up.wait_stream(main)
        down.wait_stream(main)
        for _ in range(warmup):
            one_step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(main)
        up.wait_event(e0)
        down.wait_event(e0)
        for _ in range(steps):
            one_step()
        main.wait_stream(up)
        main.wait_stream(down)
        e1.record(main)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        h2d = L * ppl * PAGE
        d2h = L * self.layer_elems * 2
        # every page went both ways, and what came back is what the device holds: layer by layer (the last
        # `ring` layers when a ring was recycled), compared on the device after an upload of the host copy
        stats, status = c.stats(), c.status()
        checked, same = 0, True
        for l in range(L - ring, L):
            r = l % ring
            back = h_out[r * self.layer_elems:(r + 1) * self.layer_elems].to(self.dev, non_blocking=True)
            same = same and bool(torch.equal(back, self.dst_layer(l)))
            checked += 1
        if not same or sum(status["count"]) or sum(stats["pages_mode"]) != self.pages or stats["pages_decoded"] != self.demand_pages:
            raise RuntimeError(f"end-to-end step inconsistent: {stats} {status} host copies equal: {same}")
        # what the host link gives to plain copies between the same buffers, both directions at once (no kernels):
        # the bound of this leg
        n_link = min(h_in.numel(), h_out.numel(), self.src.numel(), self.dst.numel(), 1 << 30)
        link_ms = []
        for _ in range(3):
            torch.cuda.synchronize()
            e0.record(main)
            up.wait_event(e0)
            down.wait_event(e0)
            with torch.cuda.stream(up):
                self.src[:n_link].copy_(h_in[:n_link], non_blocking=True)
            with torch.cuda.stream(down):
                h_out[:n_link].copy_(self.dst[:n_link], non_blocking=True)
            main.wait_stream(up)
            main.wait_stream(down)
            e1.record(main)
            torch.cuda.synchronize()
            link_ms.append(e0.elapsed_time(e1))
        link_gbs = 2 * n_link * 2 / (min(link_ms[1:]) * 1e-3) / 1e9
        self.fill_source()                                   # the copy above overwrote the head of the source
        return {"ms_per_step": ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps, "warmup": warmup,
                "link_gbs_plain_copies": link_gbs, "frac_of_link": (h2d + d2h) / (ms * 1e-3) / 1e9 / link_gbs,
                "host_buffers": "one pinned copy of the whole cache each way" if ring == L else f"a ring of {ring} layers, recycled",
                "layers_compared_with_device": checked}

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
            l = int(rng.integers(self.L)); b = int(rng.integers(w.batch))
            n = int(rng.integers((int(w.seq_lens[b]) + 15) // 16)); kv = int(rng.integers(2)); h = int(rng.integers(H))
            slot = ((l * w.blocks_per_layer + int(w.block_table[b][n])) * 2 + kv) * H + h
            page = w.gen_pages([self.layer0 * ppl + slot])[0]
            scheme = 0 if self.raw_idx is not None and bool(self.raw_take[slot].item()) else self.scheme
            rec = O.compress_page(page, scheme)
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


def timed_passes(b, passes: int, warmup: int = 3, sample_clocks: int = -1):
    """Runs `warmup` untimed and `passes` timed passes of b.step(); returns per-phase mean milliseconds, the
    total, the context's counters after the last pass and (if sample_clocks >= 0) the clocks seen meanwhile."""
    import torch
    for _ in range(warmup):
        b.step()
    torch.cuda.synchronize()
    sampler = ClockSampler(sample_clocks) if sample_clocks >= 0 else None
    if sampler:
        sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(passes)]
    end = torch.cuda.Event(enable_timing=True)
    for e in evs:
        b.step(e)
    end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    return {"comp_ms": float(np.mean([e[0].elapsed_time(e[1]) for e in evs])),
            "gath_ms": float(np.mean([e[1].elapsed_time(e[2]) for e in evs])),
            "total_ms": evs[0][0].elapsed_time(end), "stats": b.ctx.stats(), "status": b.ctx.status(), "clocks": clocks}


def phase_figures(b, comp_ms, gath_ms, stats, peak, clocks=None):
    """GB/s of uncompressed K/V and of algorithmic HBM traffic per phase.  Algorithmic bytes: compress reads the
    page, its two list entries, and writes the record's granules and one page-table entry; decompress+gather
    reads the granules, the entry and its share of the block-table entry, and writes the page."""
    H = b.w.n_kv_heads
    gran = stats["granules"]                                    # counters were reset at the start of the last pass
    comp_bytes = b.pages * (PAGE + 8 + 8) + 64 * gran
    gath_bytes = 64 * gran * (b.demand_pages / b.pages) + b.demand_pages * (8 + 4.0 / (2 * H) + PAGE)
    out = {}
    for name, ms, nbytes, pages in (("speckv_compress", comp_ms, comp_bytes, b.pages),
                                    ("speckv_decompress_gather", gath_ms, gath_bytes, b.demand_pages)):
        hbm = nbytes / (ms * 1e-3) / 1e9
        out[name] = {"ms_per_pass": ms, "uncompressed_gbs": pages * PAGE / (ms * 1e-3) / 1e9, "hbm_gbs": hbm,
                     "hbm_frac_of_measured": hbm / peak, "hbm_frac_of_8000": hbm / 8000.0, "algorithmic_bytes": nbytes}
        if clocks and clocks.get("sm_mhz"):
            # time x clock per page: compares runs whose power-capped clocks differ
            out[name]["gpu_cycles_per_page"] = ms * 1e-3 * clocks["sm_mhz"] * 1e6 / pages
    return out


def free_cuda(*objs):
    import gc
    import torch
    for o in objs:
        if hasattr(o, "ctx"):
            o.ctx.close()
    del objs
    gc.collect()
    torch.cuda.empty_cache()


def other_workloads(args, dev, peak):
    """Summary figures of the other configurations: 7B-shaped (whole cache resident), 13B-shaped (50 GiB,
    streamed in groups of eight layers: generate, compress, fetch back, next group), the decode-step paged
    fetch and the managed prefetch buffer.  Each with the clocks seen while it was timed."""
    import torch
    res = {}
    w = workloads.llama7b(seed=0)
    b = Bench(w, dev, args.scheme)
    t = timed_passes(b, passes=12, warmup=3, sample_clocks=dev.index or 0)
    res["llama2-7b"] = {"pages": b.pages, "kernels": phase_figures(b, t["comp_ms"], t["gath_ms"], t["stats"], peak, t["clocks"]),
                        "clocks": t["clocks"], "status_counts": t["status"]["count"], "parity": b.sampled_parity(n_samples=8, seed=7)}
    free_cuda(b)
    del b
    w = workloads.llama13b(seed=0)
    group, comp_ms, gath_ms, pages, dpages, gran, counts, bad = 8, 0.0, 0.0, 0, 0, 0, np.zeros(8, np.int64), 0
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    for l0 in range(0, w.n_layers, group):
        b = Bench(w, dev, args.scheme, layer0=l0, n_layers=min(group, w.n_layers - l0))
        t = timed_passes(b, passes=3, warmup=1)
        comp_ms += t["comp_ms"]; gath_ms += t["gath_ms"]; pages += b.pages; dpages += b.demand_pages
        gran += t["stats"]["granules"]; counts += np.array(t["status"]["count"])
        bad += b.sampled_parity(n_samples=2, seed=l0)["mismatches"]
        free_cuda(b)
        del b
    clocks = sampler.stop()
    H = w.n_kv_heads
    cb, gb = pages * (PAGE + 16) + 64 * gran, 64 * gran * (dpages / pages) + dpages * (8 + 4.0 / (2 * H) + PAGE)
    res["llama2-13b"] = {"pages": pages, "streamed": f"{w.n_layers // group} groups of {group} layers, times summed over the groups",
                         "kernels": {"speckv_compress": {"ms_per_pass": comp_ms, "uncompressed_gbs": pages * PAGE / comp_ms / 1e6,
                                                         "hbm_gbs": cb / comp_ms / 1e6, "hbm_frac_of_measured": cb / comp_ms / 1e6 / peak},
                                     "speckv_decompress_gather": {"ms_per_pass": gath_ms, "uncompressed_gbs": dpages * PAGE / gath_ms / 1e6,
                                                                  "hbm_gbs": gb / gath_ms / 1e6, "hbm_frac_of_measured": gb / gath_ms / 1e6 / peak}},
                         "clocks": clocks, "status_counts": [int(x) for x in counts], "parity": {"pages_checked": 2 * (w.n_layers // group), "mismatches": bad}}
    sub = argparse.Namespace(**vars(args))
    sub.steps, sub.warmup = 30, 3
    d = run_decode_fetch(sub, workloads.decode_fetch(seed=0), dev)
    res["decode-fetch-7b"] = {"uncompressed_gbs": d["value"], "ms_per_step": d["ms_per_step"], "per_step_demand_gbs": d["per_step_demand_gbs"],
                              "steps_timed": d["steps"], "prefetch": d["prefetch"], "clocks": d["clocks"], "status_counts": d["status_counts"]}
    torch.cuda.empty_cache()
    d = run_managed_prefetch(sub, workloads.decode_fetch(seed=0, n_layers=4), dev)
    res["managed-prefetch-7b"] = {"uncompressed_gbs": d["value"], "us_per_call": d["ms_per_step"] * 1e3, "calls_timed": d["steps"],
                                  "hit_rate": d["prefetch"]["hit_rate"], "coverage": d["prefetch"]["coverage"],
                                  "precision": d["prefetch"]["precision"], "clocks": d["clocks"], "status_counts": d["status_counts"]}
    torch.cuda.empty_cache()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="speckv", choices=["speckv", "reference"])
    ap.add_argument("--workload", default="llama2-70b-gqa", choices=["llama2-70b-gqa", "llama2-7b", "llama2-13b", "decode-fetch-7b", "managed-prefetch-7b"])
    ap.add_argument("--layers", type=int, default=0, help="use only this many layers (small cases for profiling)")
    ap.add_argument("--scheme", type=int, default=3)
    ap.add_argument("--passes-per-step", type=int, default=0, help="passes of the hot path per step (0 = enough for --min-seconds)")
    ap.add_argument("--min-seconds", type=float, default=2.2, help="shortest timed region the automatic passes-per-step aims at")
    ap.add_argument("--no-workloads", action="store_true", help="skip the summary figures of the other configurations")
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
    # A step is `passes_per_step` passes of the whole hot path (every layer compressed, every layer fetched
    # back), chosen from a first measurement so that the timed region covers at least two seconds: shorter
    # regions end before the power limit has settled the clock.
    b.step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(2):
        b.step()
    torch.cuda.synchronize()
    est_ms = (time.perf_counter() - t0) * 1e3 / 2
    pps = args.passes_per_step or max(1, int(np.ceil(args.min_seconds * 1e3 / (args.steps * est_ms))))
    if world > 1:                                             # every rank must run the same number of passes
        t = torch.tensor([pps], dtype=torch.int64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        pps = int(t.item())
    warm = max(args.warmup, 3)
    for _ in range(warm * pps):
        b.step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    n_pass = args.steps * pps
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_pass)]
    end = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    for e in evs:
        b.step(e)
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

    L, H = b.L, w.n_kv_heads
    peak, peak_kind = measured_peak_gbs()
    kern = phase_figures(b, comp_ms, gath_ms, stats, peak, clocks)
    dom = "speckv_compress" if comp_ms >= gath_ms else "speckv_decompress_gather"
    # the compressor is one launch per pass, the gather one launch per layer
    dom_pages = b.pages if dom == "speckv_compress" else b.demand_pages // L
    dom_bytes = kern[dom]["algorithmic_bytes"] / (1 if dom == "speckv_compress" else L)
    value = whole_job_gbs((b.pages + b.demand_pages) * PAGE * pps, world, ms_per_step)

    out = {"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": warm,
           "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16->i8",
           "data": "synthetic",
           "config": {"workload": w.name, "layers": L, "kv_heads": H, "batch": w.batch, "seq": int(w.seq_lens.max()),
                      "pages": b.pages, "uncompressed_gib": b.pages * PAGE / 2 ** 30, "scheme": args.scheme,
                      "passes_per_step": pps, "timed_seconds": total_ms * 1e-3,
                      "step": f"{pps} passes of the whole hot path (one compress call over the cache + one gather call per layer each); "
                              "the repeat makes the timed region long enough for the power-capped clock to settle",
                      "block_table": "seeded random permutation", "l2": "inputs larger than L2 (no flush)",
                      "parallelism": "replicas only" if world > 1 else "1 GPU", "calls_per_step": b.launches_per_step() * pps},
           "gpu_launches": b.launches_per_step() * n_pass, "clocks": clocks, "kernels": kern,
           "roofline": {"bound": "hbm", "kernel": dom, "achieved": kern[dom]["hbm_gbs"], "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                        "frac": kern[dom]["hbm_gbs"] / peak, "traffic": ncu_traffic(dom, dom_pages),
                        "algorithmic_bytes_per_launch": dom_bytes},
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
    if extras:
        extras["raw_only"] = 0                                 # the bypass of Sec. 3.5.3 for every page: a copy
    for name, scheme in extras.items():
        b.scheme = scheme
        t = timed_passes(b, passes=8, warmup=3)
        k = phase_figures(b, t["comp_ms"], t["gath_ms"], t["stats"], peak)
        out[name] = {"scheme": scheme, "compress_uncompressed_gbs": k["speckv_compress"]["uncompressed_gbs"],
                     "gather_uncompressed_gbs": k["speckv_decompress_gather"]["uncompressed_gbs"],
                     "compress_hbm_frac_of_measured": k["speckv_compress"]["hbm_frac_of_measured"],
                     "gather_hbm_frac_of_measured": k["speckv_decompress_gather"]["hbm_frac_of_measured"],
                     "stored_ratio": b.pages * PAGE / (64.0 * t["stats"]["granules"]), "pages_mode": t["stats"]["pages_mode"]}
    b.scheme = args.scheme
    if extras:
        # mixed traffic: a seeded 30 % of the pages take the bypass (a scheme-0 call over them), the rest the codec
        b.mixed(0.3)
        t = timed_passes(b, passes=20, warmup=3, sample_clocks=local)
        k = phase_figures(b, t["comp_ms"], t["gath_ms"], t["stats"], peak, t["clocks"])
        out["mixed_raw30"] = {"raw_fraction": float(b.raw_idx.numel()) / b.pages, "calls_per_pass": b.launches_per_step(),
                              "kernels": k, "clocks": t["clocks"], "pages_mode": t["stats"]["pages_mode"],
                              "stored_ratio": b.pages * PAGE / (64.0 * t["stats"]["granules"]), "status_counts": t["status"]["count"],
                              "vs_headline": {"compress_uncompressed": k["speckv_compress"]["uncompressed_gbs"] / kern["speckv_compress"]["uncompressed_gbs"],
                                              "gather_uncompressed": k["speckv_decompress_gather"]["uncompressed_gbs"] / kern["speckv_decompress_gather"]["uncompressed_gbs"],
                                              "compress_hbm": k["speckv_compress"]["hbm_gbs"] / kern["speckv_compress"]["hbm_gbs"],
                                              "gather_hbm": k["speckv_decompress_gather"]["hbm_gbs"] / kern["speckv_decompress_gather"]["hbm_gbs"]}}
        if world == 1 and not args.no_cpu_baseline:
            out["mixed_raw30"]["parity"] = b.sampled_parity(n_samples=24, seed=9)
        b.raw_idx = None
        # the codec on pages it can shrink: piecewise-linear rows (kvgen: runs_pages) whose run-length records reach
        # the ratio the paper reports for its delta + run-length stage; same shapes, same calls, other contents
        w.data = "runs"
        b.fill_source()
        out["long_runs"] = {"data": "rows piecewise linear in the channel index, a new segment per channel with probability %d/256" % gen.RUNS_P256}
        for name, scheme in (("delta_rle", 3), ("adaptive", 4)):
            b.scheme = scheme
            t = timed_passes(b, passes=8, warmup=3, sample_clocks=local)
            k = phase_figures(b, t["comp_ms"], t["gath_ms"], t["stats"], peak, t["clocks"])
            out["long_runs"][name] = {"scheme": scheme, "kernels": k, "clocks": t["clocks"], "pages_mode": t["stats"]["pages_mode"],
                                      "stored_ratio": b.pages * PAGE / (64.0 * t["stats"]["granules"]), "status_counts": t["status"]["count"]}
            if world == 1 and not args.no_cpu_baseline:
                out["long_runs"][name]["parity"] = b.sampled_parity(n_samples=16, seed=21)
        w.data = "gaussian"
        b.fill_source()
    b.scheme = args.scheme
    if args.consumer:
        b.step()
        n_q_heads = args.consumer if args.consumer > 0 else (64 if w.name == "llama2-70b-gqa" else w.n_kv_heads)
        out["consumer"] = b.consumer(n_q_heads)
    if args.consumer:
        out["lifecycle"] = b.lifecycle()
    if not args.no_e2e:
        e = b.e2e(steps=3, warmup=1)
        out["e2e"] = {"value": (b.pages + b.demand_pages) * PAGE / (e["ms_per_step"] * 1e-3) / 1e9, "unit": "GB/s", **e}
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
        n_pages = min(4, b.L) * w.pages_per_layer   # layers 0-3: about 10 s of single-thread CPU work
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
    if world == 1 and not args.no_workloads and w.name == "llama2-70b-gqa" and not args.layers:
        free_cuda(b)
        del b
        out["workloads"] = other_workloads(args, dev, peak)
    print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
