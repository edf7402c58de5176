"""The five seeded workloads (shapes, block tables, sequence lengths, prefetch lists).

They stand in for the KV caches of the paper's LLaMA-2 7B/13B/70B serving runs:
same tensor shapes, 16-token pages, fp16, K with a few large-magnitude channels
and Gaussian V.  Only index structures and distribution parameters live here;
page contents come from gen.py / gen.cu.

Page numbering inside the source tensor and inside the page table is the same:
slot = ((layer * blocks_per_layer + physical_block) * 2 + kv) * H + head.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import gen

L2_SLOTS = 4
PREFETCH = np.dtype([("seq", "<u4"), ("block", "<u4"), ("l2_slot", "<u4")])


@dataclass
class Workload:
    name: str
    seed: int
    n_layers: int
    n_kv_heads: int
    batch: int
    blocks_per_layer: int
    max_blocks_per_seq: int
    seq_lens: np.ndarray            # [batch] tokens
    block_table: np.ndarray         # [batch][max_blocks_per_seq] int32, -1 = unmapped
    scales: np.ndarray              # [n_layers][2][128] float32
    steps: int = 1
    extra: dict = field(default_factory=dict)
    data: str = "gaussian"          # page contents: "gaussian" (gen.gen_pages) or "runs" (gen.runs_pages)

    @property
    def pages_per_layer(self) -> int:
        return self.blocks_per_layer * 2 * self.n_kv_heads

    @property
    def n_slots(self) -> int:
        return self.n_layers * self.pages_per_layer

    def mapped_blocks(self) -> np.ndarray:
        """Physical blocks that hold data, ascending."""
        bt = self.block_table
        return np.unique(bt[bt >= 0]).astype(np.int64)

    def layer_slots(self, layer: int, blocks=None) -> np.ndarray:
        """Global page slots of `layer` for the given physical blocks, in physical order."""
        blocks = self.mapped_blocks() if blocks is None else np.asarray(blocks, np.int64)
        per = 2 * self.n_kv_heads
        base = (layer * self.blocks_per_layer + blocks) * per
        return (base[:, None] + np.arange(per)[None, :]).reshape(-1).astype(np.uint32)

    def dst_tok_off(self, seq_lens=None) -> np.ndarray:
        sl = self.seq_lens if seq_lens is None else np.asarray(seq_lens)
        tpad = ((sl.astype(np.int64) + 15) // 16) * 16
        return np.concatenate([[0], np.cumsum(tpad)[:-1]]).astype(np.uint64)

    def demand_tokens(self, seq_lens=None) -> int:
        sl = self.seq_lens if seq_lens is None else np.asarray(seq_lens)
        return int((((sl.astype(np.int64) + 15) // 16) * 16).sum())

    def gen_pages(self, slots) -> np.ndarray:
        if self.data == "runs":
            return gen.runs_pages(self.seed, slots)
        return gen.gen_pages(self.seed, slots, self.scales, self.pages_per_layer, self.n_kv_heads)


def _contiguous_table(batch, blocks_per_seq):
    return (np.arange(batch)[:, None] * blocks_per_seq + np.arange(blocks_per_seq)[None, :]).astype(np.int32)


def tiny(seed: int = 0) -> Workload:
    """1 layer, 8 KV heads, 256 tokens: 256 pages."""
    L, H, B, S = 1, 8, 1, 256
    return Workload("tiny", seed, L, H, B, S // 16, S // 16, np.full(B, S, np.uint32),
                    _contiguous_table(B, S // 16), gen.channel_scales(seed, L, "fixed4"))


def llama7b(seed: int = 0, n_layers: int = 32) -> Workload:
    """32 layers, 32 KV heads, batch 8, seq 2048, contiguous block table."""
    H, B, S = 32, 8, 2048
    return Workload("llama2-7b", seed, n_layers, H, B, B * S // 16, S // 16, np.full(B, S, np.uint32),
                    _contiguous_table(B, S // 16), gen.channel_scales(seed, n_layers, "fixed4"))


def llama13b(seed: int = 0, n_layers: int = 40) -> Workload:
    """40 layers, 40 KV heads, batch 16, seq 4096, per-layer outlier channels."""
    H, B, S = 40, 16, 4096
    return Workload("llama2-13b", seed, n_layers, H, B, B * S // 16, S // 16, np.full(B, S, np.uint32),
                    _contiguous_table(B, S // 16), gen.channel_scales(seed, n_layers, "perlayer"))


def llama70b(seed: int = 0, n_layers: int = 80, batch: int = 32, seq: int = 2048) -> Workload:
    """80 layers, 8 KV heads (GQA), batch 32, seq 2048; the block table is one seeded random
    permutation of the physical pool, shared by all layers."""
    H = 8
    nblk = seq // 16
    rng = np.random.Generator(np.random.PCG64(seed ^ 0x70B))
    perm = rng.permutation(batch * nblk).astype(np.int32)
    return Workload("llama2-70b-gqa", seed, n_layers, H, batch, batch * nblk, nblk,
                    np.full(batch, seq, np.uint32), perm.reshape(batch, nblk),
                    gen.channel_scales(seed, n_layers, "fixed4"))


def decode_fetch(seed: int = 0, n_layers: int = 32, batch: int = 64, steps: int = 100,
                 max_blocks_per_seq: int = 512, len_lo: int = 512, len_hi: int = 8192) -> Workload:
    """7B shape, ragged lognormal lengths, block table a random permutation of a pool with
    batch * max_blocks_per_seq blocks per layer (2M page slots per layer at full size)."""
    H = 32
    rng = np.random.Generator(np.random.PCG64(seed ^ 0xDEC0DE))
    ln = np.exp(rng.normal(np.log(2048.0), 0.6, size=batch))
    lens = np.clip(np.rint(ln), len_lo, min(len_hi, 16 * max_blocks_per_seq)).astype(np.uint32)
    bpl = batch * max_blocks_per_seq
    perm = rng.permutation(bpl).astype(np.int32).reshape(batch, max_blocks_per_seq)
    # blocks that are populated: up to len + steps + 4 prefetched blocks, capped by the table
    pop_tokens = np.minimum(lens.astype(np.int64) + steps + 4 * 16, 16 * max_blocks_per_seq)
    pop_blocks = (pop_tokens + 15) // 16
    bt = np.where(np.arange(max_blocks_per_seq)[None, :] < pop_blocks[:, None], perm, -1).astype(np.int32)
    w = Workload("decode-fetch-7b", seed, n_layers, H, batch, bpl, max_blocks_per_seq, lens, bt,
                 gen.channel_scales(seed, n_layers, "fixed4"), steps=steps)
    w.extra["pf_depth"] = rng.integers(1, 5, size=(steps, batch)).astype(np.uint32)
    return w


def decode_step(w: Workload, step: int):
    """(layer, seq_lens, prefetch list) of decode step `step`: the demand part covers every block
    below the current length, the prefetch list the next 1..4 blocks of each sequence."""
    layer = step % w.n_layers
    lens = np.minimum(w.seq_lens.astype(np.int64) + step, 16 * w.max_blocks_per_seq).astype(np.uint32)
    nblk = (lens.astype(np.int64) + 15) // 16
    depth = w.extra["pf_depth"][step]
    ent = []
    for b in range(w.batch):
        for i in range(int(depth[b])):
            blk = int(nblk[b]) + i
            if blk < w.max_blocks_per_seq:
                ent.append((b, blk, i))
    pf = np.array(ent, dtype=PREFETCH) if ent else np.zeros(0, PREFETCH)
    return layer, lens, pf


def prefetch_trace(w: Workload, steps: int, seed: int = 0, accuracy: float = 0.95, p_repeat: float = 0.5):
    """Inputs of the managed prefetch buffer, standing in for a sparse decode read pattern and for
    the token predictor's output: (access [steps][batch][4], cand [steps][batch][4]), int32, -1 = none.
    Step t of sequence b reads 1..4 logical blocks below its length; each read repeats the block
    the same position read in the previous step with probability p_repeat, else it is uniform over
    the sequence's blocks.  cand[t] is what a predictor of the given accuracy would say about step
    t + 1: the blocks really read then, each replaced by a uniformly drawn block with probability
    1 - accuracy, in the order of the reads."""
    rng = np.random.Generator(np.random.PCG64(seed ^ 0x9F37C4))
    nblk = np.maximum((w.seq_lens.astype(np.int64) + 15) // 16, 1)
    B = w.batch
    access = np.full((steps + 1, B, 4), -1, np.int32)
    for t in range(steps + 1):
        n_acc = rng.integers(1, 5, size=B)
        fresh = (rng.random((B, 4)) * nblk[:, None]).astype(np.int32)
        repeat = rng.random((B, 4)) < p_repeat
        prev = access[t - 1] if t else np.full((B, 4), -1, np.int32)
        blk = np.where(repeat & (prev >= 0), prev, fresh)
        access[t] = np.where(np.arange(4)[None, :] < n_acc[:, None], blk, -1)
    wrong = rng.random((steps, B, 4)) >= accuracy
    noise = (rng.random((steps, B, 4)) * nblk[None, :, None]).astype(np.int32)
    cand = np.where(access[1:] >= 0, np.where(wrong, noise, access[1:]), -1).astype(np.int32)
    return access[:steps].copy(), cand


BY_NAME = {"tiny": tiny, "llama2-7b": llama7b, "llama2-13b": llama13b, "llama2-70b-gqa": llama70b,
           "decode-fetch-7b": decode_fetch}
