"""ctypes/numpy front end of the CPU oracle (speckv_oracle.c).

TEST INFRASTRUCTURE ONLY.  Imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark; the CUDA library and its binding never
import it.  It holds no arithmetic of its own: every result comes from the C
file next to it, which follows the paper's compression algorithm, its
decompression pipeline, its address translation unit and its prefetch loop.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "speckv_oracle.c")
_HDR = os.path.join(_HERE, "speckv_oracle.h")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB = os.path.join(_OUT_DIR, "libspeckv_oracle.so")

PAGE_N, PAGE_D = 16, 128
PAGE_ELEMS = PAGE_N * PAGE_D
HDR_BYTES, GRANULE, L2_SLOTS = 16, 64, 4
N_STATUS = 8
GROUPED, GROUP_CHANNELS = 16, 8      # scheme / mode flag: one scale per group of 8 channels
ST_UNMAPPED, ST_BAD_PTE, ST_BAD_RECORD, ST_POOL_FULL, ST_BAD_INDEX, ST_TIMEOUT, ST_BAD_DST = range(1, 8)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved) and return the library path."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        os.makedirs(_OUT_DIR, exist_ok=True)
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O1", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class Status(C.Structure):
    _fields_ = [("count", C.c_uint32 * N_STATUS), ("first", C.c_uint32 * N_STATUS)]


class Stats(C.Structure):
    _fields_ = [("pages_mode", C.c_uint64 * 4), ("granules", C.c_uint64), ("payload_bytes", C.c_uint64),
                ("n_runs", C.c_uint64), ("nonfinite", C.c_uint64), ("pages_decoded", C.c_uint64),
                ("pf_issued", C.c_uint64), ("pf_skipped", C.c_uint64)]

    def as_dict(self):
        d = {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "pages_mode"}
        d["pages_mode"] = [int(v) for v in self.pages_mode]
        return d


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_uint32), ("n_kv_heads", C.c_uint32), ("blocks_per_layer", C.c_uint32),
                ("max_blocks_per_seq", C.c_uint32), ("max_seqs", C.c_uint32), ("reserved", C.c_uint32),
                ("pool_bytes", C.c_uint64)]


VADDR = np.dtype([("seq", "<u4"), ("layer", "<u2"), ("kv", "u1"), ("head", "u1"), ("pos", "<u4"), ("rsvd", "<u4")])
PADDR = np.dtype([("byte_off", "<u8"), ("rec_len", "<u4"), ("mode", "u1"), ("status", "u1"), ("rsvd", "<u2")])
PREFETCH = np.dtype([("seq", "<u4"), ("block", "<u4"), ("l2_slot", "<u4")])
# managed prefetch buffer: per-sequence state and the counters of the step calls
PF_SLOTS, PF_ACCESSES = 4, 4
PF_SEQ = np.dtype([("tag", "<u4", (2, 4)), ("used", "u1", (2, 4)), ("depth", "u1", (2,)), ("fill", "u1"), ("rsvd", "u1"),
                   ("steps", "<u4"), ("plays", "<u4", (4,)), ("reward", "<i4", (4,))])
PF_COUNTERS = ("accesses", "hits", "late", "misses", "fetched", "kept", "evicted", "evicted_used", "pages", "rsvd")

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.okv_half_to_float.restype = C.c_float
        _lib.okv_half_to_float.argtypes = [C.c_uint16]
        _lib.okv_float_to_half.restype = C.c_uint16
        _lib.okv_float_to_half.argtypes = [C.c_float]
        _lib.okv_compress_page.restype = C.c_uint32
        _lib.okv_decompress_record.restype = C.c_int
        _lib.okv_pf_score.restype = C.c_double
        _lib.okv_pf_score.argtypes = [C.c_int32, C.c_uint32, C.c_uint32, C.c_double]
        _lib.okv_pf_choose_depth.restype = C.c_uint32
        _lib.okv_pf_choose_depth.argtypes = [C.c_void_p, C.c_double]
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def half_to_float(h: int) -> float:
    return float(lib().okv_half_to_float(int(h)))


def float_to_half(f) -> int:
    return int(lib().okv_float_to_half(C.c_float(float(f))))


def compress_page(x_bits, scheme: int, N: int = PAGE_N, d: int = PAGE_D) -> bytes:
    """One page of binary16 bit patterns -> record bytes (header + payload, unpadded)."""
    x = _arr(x_bits, np.uint16).reshape(-1)
    assert x.size == N * d and (N * d) % 8 == 0 and N * d <= 2048
    rec = np.zeros(HDR_BYTES + 2 * N * d + GRANULE, np.uint8)
    n = lib().okv_compress_page(_p(x), C.c_uint32(N), C.c_uint32(d), C.c_int(scheme), _p(rec))
    return rec[:n].tobytes()


def page_stages(x_bits, N: int = PAGE_N, d: int = PAGE_D) -> dict:
    """Intermediate results of the compression algorithm for one page."""
    x = _arr(x_bits, np.uint16).reshape(-1)
    assert x.size == N * d
    amax = C.c_uint16(0)
    s, inv, n_runs = C.c_float(0), C.c_float(0), C.c_uint32(0)
    q = np.zeros(N * d, np.int8)
    sym = np.zeros(N * d, np.uint8)
    bitmap = np.zeros(N * d // 8, np.uint8)
    values = np.zeros(N * d, np.uint8)
    lib().okv_page_stages(_p(x), C.c_uint32(N), C.c_uint32(d), C.byref(amax), C.byref(s), C.byref(inv),
                          _p(q), _p(sym), _p(bitmap), _p(values), C.byref(n_runs))
    return dict(amax_bits=int(amax.value), s=np.float32(s.value), inv=np.float32(inv.value), q=q, sym=sym,
                bitmap=bitmap, values=values[:n_runs.value].copy(), n_runs=int(n_runs.value))


def page_stages_grouped(x_bits, N: int = PAGE_N, d: int = PAGE_D) -> dict:
    """Intermediate results with one scale per group of 8 adjacent channels."""
    x = _arr(x_bits, np.uint16).reshape(-1)
    assert x.size == N * d and d % GROUP_CHANNELS == 0
    n_runs = C.c_uint32(0)
    group_amax = np.zeros(d // GROUP_CHANNELS, np.uint16)
    q = np.zeros(N * d, np.int8)
    sym = np.zeros(N * d, np.uint8)
    bitmap = np.zeros(N * d // 8, np.uint8)
    values = np.zeros(N * d, np.uint8)
    lib().okv_page_stages_grouped(_p(x), C.c_uint32(N), C.c_uint32(d), _p(group_amax), _p(q), _p(sym), _p(bitmap),
                                  _p(values), C.byref(n_runs))
    return dict(group_amax=group_amax, q=q, sym=sym, bitmap=bitmap, values=values[:n_runs.value].copy(),
                n_runs=int(n_runs.value))


def decompress_record(rec: bytes, N: int = PAGE_N, d: int = PAGE_D):
    """Record bytes -> (status, page of binary16 bit patterns)."""
    r = np.frombuffer(bytes(rec), np.uint8).copy()
    out = np.zeros(N * d, np.uint16)
    rc = lib().okv_decompress_record(_p(r), C.c_uint32(r.size), C.c_uint32(N), C.c_uint32(d), _p(out))
    return int(rc), out


class Pool:
    """The oracle's state: record log, page table, cursor, prefetch tags, status and counters."""

    def __init__(self, n_layers, n_kv_heads, blocks_per_layer, max_blocks_per_seq, max_seqs, pool_bytes):
        self.cfg = Config(n_layers, n_kv_heads, blocks_per_layer, max_blocks_per_seq, max_seqs, 0, pool_bytes)
        self.n_slots = n_layers * blocks_per_layer * 2 * n_kv_heads
        self.pool = np.zeros(pool_bytes, np.uint8)
        self.pte = np.zeros(self.n_slots, np.uint64)
        self.cursor = C.c_uint64(0)
        self.l2_tag = np.zeros(max_seqs * L2_SLOTS, np.uint64)
        self.epoch = 0
        self.status = Status()
        self.stats = Stats()
        lib().okv_status_clear(C.byref(self.status))

    def clear_status(self):
        lib().okv_status_clear(C.byref(self.status))

    def status_dict(self):
        return {"count": [int(v) for v in self.status.count], "first": [int(v) for v in self.status.first]}

    def compress(self, src_bits, src_page, dst_slot, scheme: int) -> int:
        src = _arr(src_bits, np.uint16).reshape(-1, PAGE_ELEMS)
        sp, ds = _arr(src_page, np.uint32), _arr(dst_slot, np.uint32)
        assert sp.size == ds.size
        return lib().okv_compress(C.byref(self.cfg), _p(self.pool), _p(self.pte), C.byref(self.cursor), _p(src),
                                  C.c_uint32(src.shape[0]), _p(sp), _p(ds), C.c_uint32(sp.size), C.c_int(scheme),
                                  C.byref(self.status), C.byref(self.stats))

    def compact(self) -> int:
        scratch = np.zeros(self.cfg.pool_bytes, np.uint8)
        return lib().okv_compact(C.byref(self.cfg), _p(self.pool), _p(self.pte), C.byref(self.cursor), _p(scratch),
                                 C.byref(self.status))

    def free_slots(self, slots):
        """Clears the listed entries; returns [entries freed, granules released] of this call."""
        sl = _arr(slots, np.uint32)
        freed = np.zeros(2, np.uint64)
        rc = lib().okv_free_slots(C.byref(self.cfg), _p(self.pte), _p(sl), C.c_uint32(sl.size), _p(freed), C.byref(self.status))
        assert rc == 0
        return [int(freed[0]), int(freed[1])]

    def translate(self, block_table, va):
        bt = _arr(block_table, np.int32)
        va = np.ascontiguousarray(va, dtype=VADDR)
        pa = np.zeros(va.size, PADDR)
        lib().okv_translate(C.byref(self.cfg), _p(self.pte), _p(bt), _p(va), _p(pa), C.c_uint32(va.size),
                            C.byref(self.status))
        return pa

    def decompress_gather(self, layer, block_table, seq_lens, dst_tok_off, pf, dst_demand, dst_l2) -> int:
        bt = _arr(block_table, np.int32)
        sl, off = _arr(seq_lens, np.uint32), _arr(dst_tok_off, np.uint64)
        pf = np.ascontiguousarray(pf if pf is not None else np.zeros(0, PREFETCH), dtype=PREFETCH)
        assert dst_demand.dtype == np.uint16 and dst_demand.flags.c_contiguous
        assert dst_l2.dtype == np.uint16 and dst_l2.flags.c_contiguous
        H = self.cfg.n_kv_heads
        assert dst_l2.size >= self.cfg.max_seqs * L2_SLOTS * 2 * H * PAGE_ELEMS
        cap_tokens = dst_demand.size // (2 * H * PAGE_D)
        self.epoch += 1
        return lib().okv_decompress_gather(
            C.byref(self.cfg), _p(self.pool), _p(self.pte), _p(self.l2_tag), C.c_uint32(self.epoch),
            C.c_uint32(layer), _p(bt), _p(sl), _p(off), C.c_uint32(sl.size), _p(pf), C.c_uint32(pf.size),
            _p(dst_demand), C.c_uint64(cap_tokens), _p(dst_l2), C.byref(self.status), C.byref(self.stats))

    def attend(self, layer, block_table, seq_lens, q_bits, n_q_heads):
        """Decode-step attention over the pool's pages: [B][Hq][128] float64, pages fetched through translation."""
        bt = _arr(block_table, np.int32)
        sl = _arr(seq_lens, np.uint32)
        q = _arr(q_bits, np.uint16).reshape(sl.size, n_q_heads, PAGE_D)
        out = np.zeros((sl.size, n_q_heads, PAGE_D), np.float64)
        rc = lib().okv_attend(C.byref(self.cfg), _p(self.pool), _p(self.pte), C.c_uint32(layer), _p(bt), _p(sl),
                              C.c_uint32(sl.size), _p(q), C.c_uint32(n_q_heads), _p(out), C.byref(self.status), C.byref(self.stats))
        assert rc == 0
        return out


N_CANDIDATES = 8
CANDIDATE_SCHEMES = (1, 2, 3, 4, 17, 18, 19, 20)
PROBE = np.dtype([("pages", "<u8"), ("nonfinite", "<u8"), ("bad_index", "<u8"), ("granules", "<u8", (8,)),
                  ("sq_err", "<f8", (2,)), ("sq_sum", "<f8")])
POLICY = np.dtype([("w_r", "<f8"), ("w_q", "<f8"), ("w_c", "<f8"), ("q_min", "<f8"), ("cost", "<f8", (8,))])


def probe_pages(src_bits, src_page, probe=None):
    """Adds what the listed pages cost and lose under every candidate scheme to `probe` (a PROBE record)."""
    src = _arr(src_bits, np.uint16).reshape(-1, PAGE_ELEMS)
    sp = _arr(src_page, np.uint32)
    out = np.zeros(1, PROBE) if probe is None else np.ascontiguousarray(probe, dtype=PROBE).reshape(1)
    rc = lib().okv_probe_pages(_p(src), C.c_uint32(src.shape[0]), _p(sp), C.c_uint32(sp.size), _p(out))
    assert rc == 0
    return out


def make_policy(w_r, w_q, w_c, q_min, cost):
    pol = np.zeros(1, POLICY)
    pol["w_r"], pol["w_q"], pol["w_c"], pol["q_min"] = w_r, w_q, w_c, q_min
    pol["cost"][0] = cost
    return pol


def probe_quality(probe, grouped: bool) -> float:
    lib().okv_probe_quality.restype = C.c_double
    pr = np.ascontiguousarray(probe, dtype=PROBE).reshape(1)
    return float(lib().okv_probe_quality(_p(pr), C.c_int(int(grouped))))


def select_scheme(probe, policy):
    """(scheme, J of the 8 candidates) for one layer's probe and a policy."""
    pr = np.ascontiguousarray(probe, dtype=PROBE).reshape(1)
    pol = np.ascontiguousarray(policy, dtype=POLICY).reshape(1)
    obj = np.zeros(N_CANDIDATES, np.float64)
    return int(lib().okv_select_scheme(_p(pr), _p(pol), _p(obj))), obj


def pf_score(reward: int, plays: int, steps: int, beta: float) -> float:
    """The depth rule's score of one arm: mean reward + exploration bonus."""
    return float(lib().okv_pf_score(int(reward), int(plays), int(steps), float(beta)))


def pf_choose_depth(seq_state, beta: float) -> int:
    """Depth (1..4) the rule picks for one sequence's statistics (a PF_SEQ record)."""
    s = np.ascontiguousarray(seq_state, dtype=PF_SEQ).reshape(1)
    return int(lib().okv_pf_choose_depth(_p(s), float(beta)))


class PrefetchBuffer:
    """State of the managed prefetch buffer next to a Pool: two banks of 4 slots per sequence, per-sequence
    depth statistics, counters.  step() fills bank `back` and reads from the other one."""

    def __init__(self, pool: "Pool"):
        self.pool = pool
        cfg = pool.cfg
        self.state = np.zeros(cfg.max_seqs, PF_SEQ)
        self.counters = np.zeros(len(PF_COUNTERS), np.uint64)
        self.l2 = np.zeros(2 * cfg.max_seqs * PF_SLOTS * 2 * cfg.n_kv_heads * PAGE_ELEMS, np.uint16)

    def counters_dict(self):
        return {k: int(v) for k, v in zip(PF_COUNTERS, self.counters) if k != "rsvd"}

    def step(self, layer, back, block_table, access, cand, beta):
        """Returns (where [B][4], miss_dst [B][4][2][H][2048])."""
        pool, cfg = self.pool, self.pool.cfg
        bt = _arr(block_table, np.int32)
        acc = _arr(access, np.int32).reshape(-1, PF_ACCESSES)
        cd = _arr(cand, np.int32).reshape(-1, PF_SLOTS)
        B = acc.shape[0]
        assert cd.shape[0] == B
        where = np.zeros((B, PF_ACCESSES), np.int32)
        miss = np.zeros((B, PF_ACCESSES, 2, cfg.n_kv_heads, PAGE_ELEMS), np.uint16)
        rc = lib().okv_prefetch_step(C.byref(cfg), _p(pool.pool), _p(pool.pte), C.c_uint32(layer), C.c_uint32(back),
                                     _p(bt), _p(acc), _p(cd), C.c_uint32(B), C.c_double(beta), _p(self.state),
                                     _p(self.counters), _p(self.l2), _p(miss), _p(where), C.byref(pool.status),
                                     C.byref(pool.stats))
        assert rc == 0
        return where, miss

    def slot_pages(self, bank, seq, slot):
        """The 2*H pages of one buffer slot: [2][H][2048] binary16 patterns."""
        cfg = self.pool.cfg
        return self.l2.reshape(2, cfg.max_seqs, PF_SLOTS, 2, cfg.n_kv_heads, PAGE_ELEMS)[bank, seq, slot]


def attend_dense(kv_bits, seq_lens, dst_tok_off, n_kv_heads, q_bits, n_q_heads):
    """Decode-step attention over a demand workspace ([K|V][head][token][channel] per sequence)."""
    sl, off = _arr(seq_lens, np.uint32), _arr(dst_tok_off, np.uint64)
    kv = _arr(kv_bits, np.uint16).reshape(-1)
    q = _arr(q_bits, np.uint16).reshape(sl.size, n_q_heads, PAGE_D)
    out = np.zeros((sl.size, n_q_heads, PAGE_D), np.float64)
    rc = lib().okv_attend_dense(_p(kv), _p(sl), _p(off), C.c_uint32(sl.size), C.c_uint32(n_kv_heads), _p(q),
                                C.c_uint32(n_q_heads), _p(out))
    assert rc == 0
    return out
