"""Shared by the GPU parity tests: run the same call sequence on the CUDA library and on the
CPU oracle, on the same seeded inputs, and compare every output."""
from __future__ import annotations

import numpy as np

from oracle import oracle as O


def ulp_distance(a_bits, b_bits):
    """Distance in binary16 steps, with +0 and -0 identified (inputs: uint16 arrays of finite values)."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7FFF), x & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


class Pair:
    """A CUDA context and an oracle pool with identical configuration."""

    def __init__(self, n_layers, n_kv_heads, blocks_per_layer, max_blocks_per_seq, max_seqs, pool_bytes):
        import torch
        from paper_2512_11920_b200 import Context
        self.torch = torch
        self.dev = torch.device("cuda:0")
        self.H = n_kv_heads
        self.max_seqs = max_seqs
        self.gpu = Context(n_layers, n_kv_heads, blocks_per_layer, max_blocks_per_seq, max_seqs, pool_bytes)
        self.cpu = O.Pool(n_layers, n_kv_heads, blocks_per_layer, max_blocks_per_seq, max_seqs, pool_bytes)

    @classmethod
    def for_workload(cls, w, pool_bytes=None):
        return cls(w.n_layers, w.n_kv_heads, w.blocks_per_layer, w.max_blocks_per_seq, w.batch,
                   pool_bytes or max(64, w.n_slots * 2368))

    def t(self, a, dtype=None):
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint32:
            a = a.view(np.int32)
        if a.dtype == np.uint64:
            a = a.view(np.int64)
        if a.dtype == np.uint16:
            a = a.view(np.int16)
        if a.dtype.fields is not None:
            a = a.view(np.uint8)
        return self.torch.from_numpy(a).to(self.dev)

    # ---- calls -------------------------------------------------------------------------
    def compress(self, src_bits, src_page, dst_slot, scheme):
        src_page = np.asarray(src_page, np.uint32)
        dst_slot = np.asarray(dst_slot, np.uint32)
        self.cpu.compress(src_bits, src_page, dst_slot, scheme)
        self.gpu.compress(self.t(np.asarray(src_bits, np.uint16)), self.t(src_page), self.t(dst_slot), scheme)

    def translate(self, block_table, va):
        want = self.cpu.translate(block_table, va)
        pa = self.torch.zeros(16 * len(va), dtype=self.torch.uint8, device=self.dev)
        self.gpu.translate(self.t(np.asarray(block_table, np.int32)), self.t(np.asarray(va, O.VADDR)), pa)
        got = pa.cpu().numpy().view(O.PADDR)
        assert got.tobytes() == want.tobytes(), "translated addresses differ"
        return got

    def gather(self, layer, block_table, seq_lens, dst_tok_off, pf=None, cap_tokens=None, fill=0xCDCD):
        torch, H = self.torch, self.H
        seq_lens = np.asarray(seq_lens, np.uint32)
        tpad = ((seq_lens.astype(np.int64) + 15) // 16) * 16
        need = int((np.asarray(dst_tok_off, np.int64) + tpad).max()) if len(seq_lens) else 0
        cap = need if cap_tokens is None else cap_tokens
        d_cpu = np.full(cap * 2 * H * 128, fill, np.uint16)
        l_cpu = np.full(self.max_seqs * 4 * 2 * H * 2048, fill, np.uint16)
        pf_np = np.zeros(0, O.PREFETCH) if pf is None else np.asarray(pf, O.PREFETCH)
        rc = self.cpu.decompress_gather(layer, block_table, seq_lens, dst_tok_off, pf_np, d_cpu, l_cpu)
        assert rc == 0
        d_gpu, l_gpu = self.t(d_cpu * 0 + fill), self.t(l_cpu * 0 + fill)
        self.gpu.decompress_gather(layer, self.t(np.asarray(block_table, np.int32)), self.t(seq_lens),
                                   self.t(np.asarray(dst_tok_off, np.uint64)), d_gpu,
                                   self.t(pf_np) if len(pf_np) else None, l_gpu)
        d_got = d_gpu.cpu().numpy().view(np.uint16)
        l_got = l_gpu.cpu().numpy().view(np.uint16)
        for name, got, want in (("demand", d_got, d_cpu), ("prefetch buffer", l_got, l_cpu)):
            if not np.array_equal(got, want):
                bad = np.nonzero(got != want)[0]
                fin = ((got[bad] & 0x7C00) != 0x7C00) & ((want[bad] & 0x7C00) != 0x7C00)
                worst = int(ulp_distance(got[bad][fin], want[bad][fin]).max()) if fin.any() else -1
                raise AssertionError(f"{name}: {bad.size} elements differ (first at {bad[0]}, page {bad[0] // 2048}); "
                                     f"worst distance {worst} ulp; tolerance is 1 ulp and bit-exact is expected")
        return d_got, l_got

    def free_slots(self, slots):
        slots = np.asarray(slots, np.uint32)
        want = self.cpu.free_slots(slots)
        freed = self.torch.zeros(2, dtype=self.torch.int64, device=self.dev)
        self.gpu.free_slots(self.t(slots), freed)
        got = [int(v) for v in freed.cpu().numpy()]
        assert got == want, f"freed {got} != {want}"
        return got

    def compact(self):
        self.cpu.compact()
        # zeroed like the oracle's: when shared records overflow the pool, the granules between the last copy
        # that fitted and the end of the pool come back from the scratch area as they were
        scratch = self.torch.zeros(self.gpu.compact_scratch_bytes(), dtype=self.torch.uint8, device=self.dev)
        self.gpu.compact(scratch)

    # ---- the consumer: decode-step attention ---------------------------------------------
    # Tolerance.  Both sides use the same binary16 K, V and q.  The CUDA path rounds the softmax
    # weights to binary16 (relative 2^-11 each, so the weighted mean of V moves by at most
    # 2^-11 max|V|), evaluates 2^x to about 2 ulp of binary32, accumulates in binary32 and rounds
    # the result to binary16 (2^-11 |o| <= 2^-11 max|V|).  Bound used: 2^-9 max|V| per KV head.
    def _attend_check(self, got, want, vmax, G, what):
        err = np.abs(got.astype(np.float64) - want)                      # [B][Hq][128]
        tol = np.repeat(vmax, G, axis=1)[:, :, None] * 2.0 ** -9 + 1e-7  # [B][Hq][1]
        if not np.all(err <= tol):
            b, hq, c = np.unravel_index(np.argmax(err / tol), err.shape)
            raise AssertionError(f"{what}: |error| {err[b, hq, c]:.3e} > {tol[b, hq, 0]:.3e} at sequence {b}, head {hq}, channel {c}")
        return float((err / tol).max())

    def _layout(self, seq_lens):
        seq_lens = np.asarray(seq_lens, np.uint32)
        tpad = ((seq_lens.astype(np.int64) + 15) // 16) * 16
        tok = np.concatenate([[0], np.cumsum(tpad)[:-1]]).astype(np.uint64)
        return seq_lens, tpad, tok

    def _vmax(self, d_bits, seq_lens, tpad, tok):
        """Largest |V| per (sequence, KV head) of a demand workspace."""
        H = self.H
        vmax = np.zeros((len(seq_lens), H))
        for b in range(len(seq_lens)):
            if seq_lens[b]:
                v = d_bits[int(tok[b]) * 2 * H * 128:][:2 * H * int(tpad[b]) * 128].view(np.float16).astype(np.float64)
                v = v.reshape(2, H, int(tpad[b]), 128)[1][:, :int(seq_lens[b])]
                vmax[b] = np.abs(np.where(np.isfinite(v), v, 0.0)).max(axis=(1, 2))
        return vmax

    def attend_dense(self, layer, block_table, seq_lens, q_bits, n_q_heads):
        """gather (both sides, compared) then attention over the gathered workspace (both sides, compared)."""
        torch, H = self.torch, self.H
        seq_lens, tpad, tok = self._layout(seq_lens)
        B = len(seq_lens)
        q = np.asarray(q_bits, np.uint16).reshape(B, n_q_heads, 128)
        d_got, _ = self.gather(layer, block_table, seq_lens, tok, fill=0)
        want = O.attend_dense(d_got, seq_lens, tok, H, q, n_q_heads)
        ws = torch.empty(self.gpu.attend_workspace_bytes(B), dtype=torch.uint8, device=self.dev)
        out = torch.full((B, n_q_heads, 128), float("nan"), dtype=torch.float16, device=self.dev)
        self.gpu.attend_dense(self.t(d_got), self.t(seq_lens), self.t(tok), self.t(q).view(torch.float16), out, ws)
        return self._attend_check(out.cpu().numpy(), want, self._vmax(d_got, seq_lens, tpad, tok), n_q_heads // H, "attend_dense")

    def attend_fused(self, layer, block_table, seq_lens, q_bits, n_q_heads):
        """Attention straight from the compressed pages (both sides, compared; statuses and counters follow)."""
        torch, H = self.torch, self.H
        seq_lens, tpad, tok = self._layout(seq_lens)
        B = len(seq_lens)
        q = np.asarray(q_bits, np.uint16).reshape(B, n_q_heads, 128)
        want = self.cpu.attend(layer, block_table, seq_lens, q, n_q_heads)
        # bound: from a gather on a scratch copy of the oracle's bookkeeping (same pool and page table)
        scratch = O.Pool.__new__(O.Pool)
        scratch.__dict__.update(self.cpu.__dict__)
        scratch.status, scratch.stats, scratch.l2_tag = O.Status(), O.Stats(), self.cpu.l2_tag.copy()
        d = np.zeros(max(1, int(tpad.sum())) * 2 * H * 128, np.uint16)
        scratch.decompress_gather(layer, block_table, seq_lens, tok, None, d, np.zeros(self.max_seqs * 4 * 2 * H * 2048, np.uint16))
        ws = torch.empty(self.gpu.attend_workspace_bytes(B), dtype=torch.uint8, device=self.dev)
        out = torch.full((B, n_q_heads, 128), float("nan"), dtype=torch.float16, device=self.dev)
        self.gpu.decompress_attend(layer, self.t(np.asarray(block_table, np.int32)), self.t(seq_lens),
                                   self.t(q).view(torch.float16), out, ws)
        return self._attend_check(out.cpu().numpy(), want, self._vmax(d, seq_lens, tpad, tok), n_q_heads // H, "decompress_attend")

    # ---- state comparison ----------------------------------------------------------------
    def check_state(self, pool_defined_bytes=None):
        """pool_defined_bytes: compare the pool only up to there (after a compaction whose copies did not all fit,
        the bytes behind the last copy that did are unspecified)."""
        cur = self.gpu.cursor()
        assert cur == self.cpu.cursor.value, f"cursor {cur} != {self.cpu.cursor.value}"
        pte = self.gpu.pte_view().cpu().numpy().view(np.uint64)
        if not np.array_equal(pte, self.cpu.pte):
            bad = np.nonzero(pte != self.cpu.pte)[0]
            raise AssertionError(f"{bad.size} page-table entries differ, first slot {bad[0]}: "
                                 f"{int(pte[bad[0]]):#x} != {int(self.cpu.pte[bad[0]]):#x}")
        # The whole pool, not only the log up to the cursor: bytes behind the cursor are a canary (nothing may be
        # written there; after a compaction they keep what the old log held, on both sides alike).  Pools too
        # large to copy whole are compared up to the cursor and on 64 MiB behind it.
        total = self.cpu.cfg.pool_bytes
        used = min(cur * 64, total)
        upto = total if total <= (1 << 28) else min(total, used + (64 << 20))
        if pool_defined_bytes is not None:
            upto = used = min(upto, pool_defined_bytes)
        pool = self.gpu.pool_view(upto).cpu().numpy()
        if not np.array_equal(pool, self.cpu.pool[:upto]):
            bad = np.nonzero(pool != self.cpu.pool[:upto])[0]
            where = "compressed bytestream" if bad[0] < used else "pool bytes behind the cursor (nothing may be written there)"
            raise AssertionError(f"{where}: {bad.size} bytes differ, first at byte {bad[0]} (cursor at byte {used})")
        tags = self.gpu.l2_tag_view().cpu().numpy().view(np.uint64)
        assert np.array_equal(tags, self.cpu.l2_tag), "prefetch tags differ"
        assert self.gpu.stats() == self.cpu.stats.as_dict(), f"{self.gpu.stats()} != {self.cpu.stats.as_dict()}"
        assert self.gpu.status() == self.cpu.status_dict(), f"{self.gpu.status()} != {self.cpu.status_dict()}"

    def close(self):
        self.gpu.close()
