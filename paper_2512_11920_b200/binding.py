"""ctypes binding of the speckv C ABI (include/speckv.h).

Argument marshalling only: torch supplies device memory and the current stream, every step
of the codec runs inside libspeckv.so.  Names and argument order follow the C header.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspeckv.so")

RAW, INT8, INT8_DELTA, INT8_DELTA_RLE, AUTO = 0, 1, 2, 3, 4
GROUPED = 16     # OR-ed into a scheme: one scale per group of 8 channels instead of one per page
N_STATUS = 8
L2_SLOTS = 4
STATUS_NAMES = ["", "unmapped", "bad_pte", "bad_record", "pool_full", "bad_index", "timeout", "bad_dst"]

VADDR_DTYPE = np.dtype([("seq", "<u4"), ("layer", "<u2"), ("kv", "u1"), ("head", "u1"), ("pos", "<u4"), ("rsvd", "<u4")])
PADDR_DTYPE = np.dtype([("byte_off", "<u8"), ("rec_len", "<u4"), ("mode", "u1"), ("status", "u1"), ("rsvd", "<u2")])
PREFETCH_DTYPE = np.dtype([("seq", "<u4"), ("block", "<u4"), ("l2_slot", "<u4")])
# managed prefetch buffer: per-sequence state (80 bytes) and the counters of speckv_prefetch_step (10 x uint64)
PF_SEQ_DTYPE = np.dtype([("tag", "<u4", (2, 4)), ("used", "u1", (2, 4)), ("depth", "u1", (2,)), ("fill", "u1"), ("rsvd", "u1"),
                         ("steps", "<u4"), ("plays", "<u4", (4,)), ("reward", "<i4", (4,))])
PF_COUNTER_NAMES = ("accesses", "hits", "late", "misses", "fetched", "kept", "evicted", "evicted_used", "pages", "rsvd")

EXPORTS = ["speckv_create", "speckv_destroy", "speckv_reset", "speckv_compress", "speckv_translate",
           "speckv_decompress_gather", "speckv_compress_host", "speckv_decompress_gather_host", "speckv_compress_static",
           "speckv_attend_workspace_bytes", "speckv_attend_dense", "speckv_decompress_attend",
           "speckv_compact_scratch_bytes", "speckv_compact", "speckv_prefetch_step", "speckv_get_status", "speckv_get_stats", "speckv_clear_status", "speckv_pool_ptr",
           "speckv_pte_ptr", "speckv_l2_tag_ptr", "speckv_get_cursor", "speckv_version",
           "speckv_set_wait_limits", "speckv_inject_missing_tiles", "speckv_set_gather_chaining", "speckv_free_slots",
           "speckv_pipeline_layers", "speckv_pipeline_attend", "speckv_probe_pages", "speckv_select_scheme"]


# speckv_layer_fn: int consume(void *user, uint32_t layer, const void *kv, void *stream)
LAYER_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p)


class SpeckvError(RuntimeError):
    pass


class _Config(C.Structure):
    _fields_ = [("n_layers", C.c_uint32), ("n_kv_heads", C.c_uint32), ("blocks_per_layer", C.c_uint32),
                ("max_blocks_per_seq", C.c_uint32), ("max_seqs", C.c_uint32), ("reserved", C.c_uint32),
                ("pool_bytes", C.c_uint64)]


class _Status(C.Structure):
    _fields_ = [("count", C.c_uint32 * N_STATUS), ("first", C.c_uint32 * N_STATUS)]


class _Stats(C.Structure):
    _fields_ = [("pages_mode", C.c_uint64 * 4), ("granules", C.c_uint64), ("payload_bytes", C.c_uint64),
                ("n_runs", C.c_uint64), ("nonfinite", C.c_uint64), ("pages_decoded", C.c_uint64),
                ("pf_issued", C.c_uint64), ("pf_skipped", C.c_uint64)]


_lib = None


def load_library(path: str = LIB_PATH):
    """Loads libspeckv.so and declares the prototypes.  Raises if the library is not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise SpeckvError(f"{path} is missing: build it with __graft_entry__.build() "
                          "(python -m paper_2512_11920_b200.build); there is no CPU fallback")
    lib = C.CDLL(path)
    vp, u32, u64, i32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int
    lib.speckv_create.argtypes = [C.POINTER(vp), C.POINTER(_Config)]
    lib.speckv_destroy.argtypes = [vp]
    lib.speckv_reset.argtypes = [vp, vp]
    lib.speckv_compress.argtypes = [vp, vp, u32, vp, vp, u32, i32, vp]
    lib.speckv_translate.argtypes = [vp, vp, vp, vp, u32, vp]
    lib.speckv_decompress_gather.argtypes = [vp, u32, vp, vp, vp, u32, vp, u32, vp, u64, vp, vp]
    lib.speckv_compress_host.argtypes = [vp, vp, u32, vp, vp, vp, u32, i32, vp]
    lib.speckv_decompress_gather_host.argtypes = [vp, u32, vp, vp, vp, u32, vp, u32, vp, u64, vp, vp, u64, vp]
    lib.speckv_compress_static.argtypes = [vp, u32, vp, vp, u32, i32, vp, u64, vp, u64, vp, vp]
    lib.speckv_compact_scratch_bytes.argtypes = [vp]
    lib.speckv_compact.argtypes = [vp, vp, u64, vp]
    lib.speckv_prefetch_step.argtypes = [vp, u32, u32, vp, vp, vp, u32, C.c_double, vp, vp, vp, vp, vp, vp]
    lib.speckv_attend_workspace_bytes.argtypes = [u32, u32]
    lib.speckv_attend_dense.argtypes = [vp, vp, vp, vp, u32, vp, u32, vp, vp, u64, vp]
    lib.speckv_decompress_attend.argtypes = [vp, u32, vp, vp, u32, vp, u32, vp, vp, u64, vp]
    lib.speckv_get_status.argtypes = [vp, C.POINTER(_Status), vp]
    lib.speckv_get_stats.argtypes = [vp, C.POINTER(_Stats), vp]
    lib.speckv_clear_status.argtypes = [vp, vp]
    lib.speckv_set_wait_limits.argtypes = [vp, u32, u64]
    lib.speckv_inject_missing_tiles.argtypes = [vp, u32]
    lib.speckv_set_gather_chaining.argtypes = [vp, i32]
    lib.speckv_free_slots.argtypes = [vp, vp, u32, vp, vp]
    lib.speckv_probe_pages.argtypes = [vp, u32, vp, u32, vp, vp]
    lib.speckv_select_scheme.argtypes = [vp, vp, vp]
    lib.speckv_pipeline_layers.argtypes = [vp, u32, u32, vp, vp, vp, u32, vp, u32, u64, LAYER_FN, vp, vp]
    lib.speckv_pipeline_attend.argtypes = [vp, u32, u32, vp, vp, vp, u32, vp, u32, u64, vp, u32, vp, vp, u64, vp]
    lib.speckv_get_cursor.argtypes = [vp, C.POINTER(u64), vp]
    for name in ("speckv_pool_ptr", "speckv_pte_ptr", "speckv_l2_tag_ptr"):
        getattr(lib, name).argtypes = [vp]
        getattr(lib, name).restype = vp
    lib.speckv_version.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("speckv_pool_ptr", "speckv_pte_ptr", "speckv_l2_tag_ptr", "speckv_version"):
            getattr(lib, name).restype = C.c_int
    lib.speckv_attend_workspace_bytes.restype = u64
    lib.speckv_compact_scratch_bytes.restype = u64
    _lib = lib
    return lib


def _check(rc: int, what: str):
    if rc != 0:
        why = {-1: "invalid argument", -2: "CUDA runtime error", -3: "device is not compute capability 10.x",
               -4: "too many pages for a fixed-capacity entry point"}.get(rc, "?")
        raise SpeckvError(f"{what} failed: {rc} ({why})")


def _stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


def _ptr(t, dtypes=None, what="tensor"):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise SpeckvError(f"{what} must be a contiguous CUDA tensor")
    if dtypes is not None and t.dtype not in dtypes:
        raise SpeckvError(f"{what} has dtype {t.dtype}, expected one of {dtypes}")
    return t.data_ptr()


STATIC_MAX_PAGES = 524288
CTL_BLOCK_BYTES = 160


def compress_static(src, src_page, dst_slot, scheme, pool, pte, ctl):
    """speckv_compress_static: the compressor for callers that may not allocate device memory.

    Every buffer is the caller's: `pool` (uint8, 64-byte aligned, multiple of 64 bytes), `pte`
    (int64, one entry per slot, zeroed before first use) and `ctl` (CTL_BLOCK_BYTES bytes: zero,
    with bytes 40..71 set to 0xFF, before first use).  The library's own scan scratch is a fixed
    array, so one call takes at most STATIC_MAX_PAGES pages and calls must not overlap on the GPU.
    """
    import torch
    lib = load_library()
    n = int(src_page.numel())
    if int(dst_slot.numel()) != n:
        raise SpeckvError("src_page and dst_slot differ in length")
    if ctl.numel() * ctl.element_size() < CTL_BLOCK_BYTES:
        raise SpeckvError("ctl too small")
    _check(lib.speckv_compress_static(_ptr(src, None, "src"), src.numel() * src.element_size() // 4096,
                                      _ptr(src_page, (torch.int32,), "src_page"), _ptr(dst_slot, (torch.int32,), "dst_slot"),
                                      n, scheme, _ptr(pool, (torch.uint8,), "pool"), pool.numel(),
                                      _ptr(pte, (torch.int64,), "pte"), pte.numel(), _ptr(ctl), _stream()),
           "speckv_compress_static")


PROBE_DTYPE = np.dtype([("pages", "<u8"), ("nonfinite", "<u8"), ("bad_index", "<u8"), ("granules", "<u8", (8,)),
                        ("sq_err", "<f8", (2,)), ("sq_sum", "<f8")])
POLICY_DTYPE = np.dtype([("w_r", "<f8"), ("w_q", "<f8"), ("w_c", "<f8"), ("q_min", "<f8"), ("cost", "<f8", (8,))])
CANDIDATE_SCHEMES = (1, 2, 3, 4, 17, 18, 19, 20)


def probe_pages(src, src_page, probe):
    """speckv_probe_pages: adds the measurements of the listed pages to `probe`, a zeroed uint8 CUDA tensor of
    PROBE_DTYPE.itemsize bytes (one layer's accumulator)."""
    import torch
    lib = load_library()
    if probe.numel() * probe.element_size() < PROBE_DTYPE.itemsize:
        raise SpeckvError("probe too small")
    _check(lib.speckv_probe_pages(_ptr(src, None, "src"), src.numel() * src.element_size() // 4096,
                                  _ptr(src_page, (torch.int32,), "src_page"), int(src_page.numel()), _ptr(probe), _stream()),
           "speckv_probe_pages")


def select_scheme(probe, w_r: float, w_q: float, w_c: float, q_min: float, cost):
    """speckv_select_scheme: probe = a PROBE_DTYPE record on the host (numpy); returns (scheme, objective[8])."""
    lib = load_library()
    pr = np.ascontiguousarray(probe, dtype=PROBE_DTYPE).reshape(1)
    pol = np.zeros(1, POLICY_DTYPE)
    pol["w_r"], pol["w_q"], pol["w_c"], pol["q_min"] = w_r, w_q, w_c, q_min
    pol["cost"][0] = cost
    obj = np.zeros(8, np.float64)
    rc = lib.speckv_select_scheme(pr.ctypes.data_as(C.c_void_p), pol.ctypes.data_as(C.c_void_p), obj.ctypes.data_as(C.c_void_p))
    if rc < 0:
        _check(rc, "speckv_select_scheme")
    return int(rc), obj


class Context:
    """Owns one speckv context (pool, page table, cursor, prefetch tags) on the current device."""

    def __init__(self, n_layers: int, n_kv_heads: int, blocks_per_layer: int, max_blocks_per_seq: int, max_seqs: int,
                 pool_bytes: int):
        import torch
        if not torch.cuda.is_available():
            raise SpeckvError("speckv needs a CUDA device (sm_100a); there is no CPU fallback")
        self._lib = load_library()
        self.cfg = _Config(n_layers, n_kv_heads, blocks_per_layer, max_blocks_per_seq, max_seqs, 0, pool_bytes)
        self.n_slots = n_layers * blocks_per_layer * 2 * n_kv_heads
        self._h = C.c_void_p()
        _check(self._lib.speckv_create(C.byref(self._h), C.byref(self.cfg)), "speckv_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.speckv_destroy(self._h)
            self._h = None

    __del__ = close

    # -- the three calls of the hot path -------------------------------------------------
    def compress(self, src, src_page, dst_slot, scheme: int = INT8_DELTA_RLE):
        """speckv_compress: src fp16/int16/uint8 pages, src_page/dst_slot int32 tensors (read as uint32)."""
        import torch
        n = int(src_page.numel())
        if int(dst_slot.numel()) != n:
            raise SpeckvError("src_page and dst_slot differ in length")
        n_src = src.numel() * src.element_size() // 4096
        _check(self._lib.speckv_compress(self._h, _ptr(src, None, "src"), n_src,
                                         _ptr(src_page, (torch.int32,), "src_page"),
                                         _ptr(dst_slot, (torch.int32,), "dst_slot"), n, scheme, _stream()), "speckv_compress")

    def translate(self, block_table, va, pa):
        """speckv_translate: va/pa are uint8 CUDA tensors holding VADDR_DTYPE / PADDR_DTYPE records."""
        import torch
        n = va.numel() * va.element_size() // 16
        if pa.numel() * pa.element_size() < 16 * n:
            raise SpeckvError("pa too small")
        _check(self._lib.speckv_translate(self._h, _ptr(block_table, (torch.int32,), "block_table"), _ptr(va), _ptr(pa), n,
                                          _stream()), "speckv_translate")

    def decompress_gather(self, layer: int, block_table, seq_lens, dst_tok_off, dst_demand, pf=None, dst_l2=None):
        """speckv_decompress_gather: seq_lens int32, dst_tok_off int64, pf uint8 tensor of PREFETCH_DTYPE records."""
        import torch
        B = int(seq_lens.numel()) if seq_lens is not None else 0
        n_pf = (pf.numel() * pf.element_size() // 12) if pf is not None else 0
        H = self.cfg.n_kv_heads
        cap = (dst_demand.numel() * dst_demand.element_size() // (2 * H * 256)) if dst_demand is not None else 0
        if n_pf and dst_l2.numel() * dst_l2.element_size() < self.cfg.max_seqs * L2_SLOTS * 2 * H * 4096:
            raise SpeckvError("dst_l2 too small")
        _check(self._lib.speckv_decompress_gather(
            self._h, layer, _ptr(block_table, (torch.int32,), "block_table"), _ptr(seq_lens, (torch.int32,), "seq_lens"),
            _ptr(dst_tok_off, (torch.int64,), "dst_tok_off"), B, _ptr(pf), n_pf, _ptr(dst_demand), cap, _ptr(dst_l2),
            _stream()), "speckv_decompress_gather")

    def free_slots(self, slots, freed=None):
        """speckv_free_slots: slots int32 tensor (read as uint32); freed int64[2] tensor or None (added to)."""
        import torch
        _check(self._lib.speckv_free_slots(self._h, _ptr(slots, (torch.int32,), "slots"), int(slots.numel()),
                                           _ptr(freed, (torch.int64,), "freed"), _stream()), "speckv_free_slots")

    def compact_scratch_bytes(self) -> int:
        return int(self._lib.speckv_compact_scratch_bytes(self._h))

    def compact(self, scratch):
        """speckv_compact: drop the records no page-table entry points at, pack the rest in slot order."""
        _check(self._lib.speckv_compact(self._h, _ptr(scratch), scratch.numel() * scratch.element_size(), _stream()),
               "speckv_compact")

    def prefetch_step(self, layer: int, back: int, block_table, access, cand, beta: float, state, counters, l2, miss_dst,
                      where):
        """speckv_prefetch_step: one decode step of the managed prefetch buffer.  access, cand, where int32 [B][4];
        state uint8 tensor of PF_SEQ_DTYPE records; counters int64 [10]; l2, miss_dst fp16/int16 buffers."""
        import torch
        B = int(access.numel()) // 4
        H = self.cfg.n_kv_heads
        if cand.numel() != 4 * B or where.numel() != 4 * B or state.numel() * state.element_size() < 80 * B:
            raise SpeckvError("access, cand, where and state must cover the same sequences")
        if l2.numel() * l2.element_size() < 2 * self.cfg.max_seqs * L2_SLOTS * 2 * H * 4096 or \
                miss_dst.numel() * miss_dst.element_size() < B * 4 * 2 * H * 4096 or counters.numel() * counters.element_size() < 80:
            raise SpeckvError("l2, miss_dst or counters too small")
        _check(self._lib.speckv_prefetch_step(
            self._h, layer, back, _ptr(block_table, (torch.int32,), "block_table"), _ptr(access, (torch.int32,), "access"),
            _ptr(cand, (torch.int32,), "cand"), B, float(beta), _ptr(state), _ptr(counters, (torch.int64,), "counters"),
            _ptr(l2), _ptr(miss_dst), _ptr(where, (torch.int32,), "where"), _stream()), "speckv_prefetch_step")

    def attend_workspace_bytes(self, B: int) -> int:
        return int(self._lib.speckv_attend_workspace_bytes(B, self.cfg.n_kv_heads))

    def attend_dense(self, kv, seq_lens, dst_tok_off, q, out, workspace):
        """speckv_attend_dense: q, out fp16 [B][n_q_heads][128]; kv = the demand workspace of decompress_gather."""
        import torch
        B = int(seq_lens.numel())
        n_q_heads = q.numel() // (B * 128) if B else self.cfg.n_kv_heads
        _check(self._lib.speckv_attend_dense(
            self._h, _ptr(kv), _ptr(seq_lens, (torch.int32,), "seq_lens"), _ptr(dst_tok_off, (torch.int64,), "dst_tok_off"),
            B, _ptr(q, (torch.float16,), "q"), n_q_heads, _ptr(out, (torch.float16,), "out"),
            _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()), "speckv_attend_dense")

    def decompress_attend(self, layer: int, block_table, seq_lens, q, out, workspace):
        """speckv_decompress_attend: attention straight from the compressed pages of `layer`."""
        import torch
        B = int(seq_lens.numel())
        n_q_heads = q.numel() // (B * 128) if B else self.cfg.n_kv_heads
        _check(self._lib.speckv_decompress_attend(
            self._h, layer, _ptr(block_table, (torch.int32,), "block_table"), _ptr(seq_lens, (torch.int32,), "seq_lens"),
            B, _ptr(q, (torch.float16,), "q"), n_q_heads, _ptr(out, (torch.float16,), "out"),
            _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()), "speckv_decompress_attend")

    def _ring_args(self, ring, ring_slots):
        H = self.cfg.n_kv_heads
        slot_tokens = ring.numel() * ring.element_size() // ring_slots // (2 * H * 256)
        if slot_tokens == 0:
            raise SpeckvError("ring too small")
        return slot_tokens

    def pipeline_layers(self, layer0: int, n_layers: int, block_table, seq_lens, dst_tok_off, ring, ring_slots: int, consume):
        """speckv_pipeline_layers: gathers run up to ring_slots - 1 layers ahead on the context's fetch stream;
        consume(layer, kv_ptr, stream_ptr) is called per layer and enqueues that layer's work on the current stream."""
        import torch
        failed = []

        def trampoline(_user, layer, kv, stream):
            try:
                consume(int(layer), int(kv), int(stream or 0))
                return 0
            except Exception as exc:                      # an exception must not cross the C frames
                failed.append(exc)
                return -1

        fn = LAYER_FN(trampoline)
        rc = self._lib.speckv_pipeline_layers(
            self._h, layer0, n_layers, _ptr(block_table, (torch.int32,), "block_table"), _ptr(seq_lens, (torch.int32,), "seq_lens"),
            _ptr(dst_tok_off, (torch.int64,), "dst_tok_off"), int(seq_lens.numel()), _ptr(ring), ring_slots,
            self._ring_args(ring, ring_slots), fn, None, _stream())
        if failed:
            raise failed[0]
        _check(rc, "speckv_pipeline_layers")

    def pipeline_attend(self, layer0: int, n_layers: int, block_table, seq_lens, dst_tok_off, ring, ring_slots: int, q, out,
                        workspace):
        """speckv_pipeline_attend: q, out fp16 [n_layers][B][n_q_heads][128]."""
        import torch
        B = int(seq_lens.numel())
        n_q_heads = q.numel() // (n_layers * B * 128)
        _check(self._lib.speckv_pipeline_attend(
            self._h, layer0, n_layers, _ptr(block_table, (torch.int32,), "block_table"), _ptr(seq_lens, (torch.int32,), "seq_lens"),
            _ptr(dst_tok_off, (torch.int64,), "dst_tok_off"), B, _ptr(ring), ring_slots, self._ring_args(ring, ring_slots),
            _ptr(q, (torch.float16,), "q"), n_q_heads, _ptr(out, (torch.float16,), "out"), _ptr(workspace),
            workspace.numel() * workspace.element_size(), _stream()), "speckv_pipeline_attend")

    def compress_host(self, src_host, staging, src_page, dst_slot, scheme: int = INT8_DELTA_RLE):
        """speckv_compress_host: src_host is a (pinned) CPU tensor of pages, staging a CUDA tensor of the same size."""
        import torch
        n = int(src_page.numel())
        n_src = src_host.numel() * src_host.element_size() // 4096
        if src_host.is_cuda or not src_host.is_contiguous() or staging.numel() * staging.element_size() < n_src * 4096:
            raise SpeckvError("src_host must be a contiguous CPU tensor and staging at least as large")
        _check(self._lib.speckv_compress_host(self._h, src_host.data_ptr(), n_src, _ptr(staging, None, "staging"),
                                              _ptr(src_page, (torch.int32,), "src_page"),
                                              _ptr(dst_slot, (torch.int32,), "dst_slot"), n, scheme, _stream()),
               "speckv_compress_host")

    def decompress_gather_host(self, layer: int, block_table, seq_lens, dst_tok_off, dst_demand, dst_host):
        """speckv_decompress_gather_host: demand gather into dst_demand, then copy to the (pinned) CPU tensor dst_host."""
        import torch
        H = self.cfg.n_kv_heads
        cap = dst_demand.numel() * dst_demand.element_size() // (2 * H * 256)
        nbytes = dst_host.numel() * dst_host.element_size()
        if dst_host.is_cuda or not dst_host.is_contiguous():
            raise SpeckvError("dst_host must be a contiguous CPU tensor")
        _check(self._lib.speckv_decompress_gather_host(
            self._h, layer, _ptr(block_table, (torch.int32,), "block_table"), _ptr(seq_lens, (torch.int32,), "seq_lens"),
            _ptr(dst_tok_off, (torch.int64,), "dst_tok_off"), int(seq_lens.numel()), None, 0, _ptr(dst_demand), cap, None,
            dst_host.data_ptr(), nbytes, _stream()), "speckv_decompress_gather_host")

    # -- state ---------------------------------------------------------------------------
    def reset(self):
        _check(self._lib.speckv_reset(self._h, _stream()), "speckv_reset")

    def clear_status(self):
        _check(self._lib.speckv_clear_status(self._h, _stream()), "speckv_clear_status")

    def set_wait_limits(self, lookback_polls: int = 0, wait_ns: int = 0):
        """speckv_set_wait_limits: bounds of the compressor's internal waits (0 = default)."""
        _check(self._lib.speckv_set_wait_limits(self._h, lookback_polls, wait_ns), "speckv_set_wait_limits")

    def set_gather_chaining(self, enabled: bool):
        """speckv_set_gather_chaining: allow consecutive gathers on one stream to overlap (default on)."""
        _check(self._lib.speckv_set_gather_chaining(self._h, int(bool(enabled))), "speckv_set_gather_chaining")

    def inject_missing_tiles(self, n_tiles: int):
        """speckv_inject_missing_tiles: the next compress call never hands out its first n_tiles tiles."""
        _check(self._lib.speckv_inject_missing_tiles(self._h, n_tiles), "speckv_inject_missing_tiles")

    def status(self) -> dict:
        s = _Status()
        _check(self._lib.speckv_get_status(self._h, C.byref(s), _stream()), "speckv_get_status")
        return {"count": [int(v) for v in s.count], "first": [int(v) for v in s.first]}

    def stats(self) -> dict:
        s = _Stats()
        _check(self._lib.speckv_get_stats(self._h, C.byref(s), _stream()), "speckv_get_stats")
        d = {k: int(getattr(s, k)) for k, _ in s._fields_ if k != "pages_mode"}
        d["pages_mode"] = [int(v) for v in s.pages_mode]
        return d

    def cursor(self) -> int:
        v = C.c_uint64(0)
        _check(self._lib.speckv_get_cursor(self._h, C.byref(v), _stream()), "speckv_get_cursor")
        return int(v.value)

    def _view(self, ptr: int, nbytes: int):
        """uint8 torch view of context-owned device memory (valid while the context lives)."""
        import torch
        iface = {"shape": (nbytes,), "typestr": "|u1", "data": (int(ptr), False), "version": 2, "strides": None}
        holder = type("DevMem", (), {"__cuda_array_interface__": iface})()
        return torch.as_tensor(holder, device="cuda")

    def pool_view(self, nbytes=None):
        return self._view(self._lib.speckv_pool_ptr(self._h), nbytes or self.cfg.pool_bytes)

    def pte_view(self):
        return self._view(self._lib.speckv_pte_ptr(self._h), self.n_slots * 8)

    def l2_tag_view(self):
        return self._view(self._lib.speckv_l2_tag_ptr(self._h), self.cfg.max_seqs * L2_SLOTS * 8)
