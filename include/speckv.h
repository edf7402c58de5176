/*
 * speckv — KV-cache page codec for one NVIDIA B200 (sm_100a), after the cache engine of
 * CXL-SpecKV (Sec. 3.5: compression, decompression, address translation, scatter-gather)
 * and the prefetch loop of its Algorithm "Speculative KV-Cache Prefetching".
 *
 * C ABI.  No C++ or framework types cross it.  Unless marked HOST, every pointer is DEVICE
 * memory owned by the caller; the library neither frees it nor touches it after the work
 * it enqueued has completed.  `stream` is a cudaStream_t passed as void* (NULL = default
 * stream).  Calls enqueue work and return; they do not synchronise unless stated.
 *
 * Return value of every call: 0 = enqueued/OK, negative = rejected on the host (see
 * SPECKV_E_*), nothing enqueued.  Conditions found on the device for individual pages
 * (unmapped block, empty slot, damaged record, pool full, index out of range, ...) never
 * fault: the page is skipped, its destination (or page-table entry) is left untouched and
 * the condition is counted in the context's status block (speckv_get_status).
 *
 * Data model
 *   page      16 tokens x 128 channels of IEEE binary16 = 4,096 bytes, row-major
 *             (Sec. 3.3.1: 4 KB pages; Algorithm "KV-Cache Compression": X in R^{N x d}).
 *   slot      physical page number: ((layer*blocks_per_layer + block)*2 + kv)*n_kv_heads + head
 *             (layer-separated regions, Sec. 3.3.3).
 *   record    16-byte header + payload, zero-padded to a multiple of 64 bytes, appended to
 *             the pool at the cursor in list order (64 B = one 512-bit beat, Sec. 3.5.1).
 *             header: +0 s (binary32 bits) +4 payload_len u16 +6 mode u8 +7 version u8 (=1)
 *                     +8 n_runs u16 +10 amax bits u16 +12 reserved u32 (=0); little-endian.
 *             mode 0: raw fp16 page (4,096 B)            — bypass of Sec. 3.5.3
 *             mode 1: int8 q[2048]                       — "INT8 only"
 *             mode 2: int8 deltas along channels, mod 256 — "INT8 + Delta"
 *             mode 3: 256-byte run-head bitmap (bit k, LSB first, set iff symbol k differs
 *                     from symbol k-1 or k = 0) + one byte per run — "INT8 + Delta + RLE"
 *             modes 17, 18, 19 (= 1, 2, 3 | SPECKV_GROUPED): the payload starts with 16 u16
 *                     values, the largest |x| (binary16 pattern) of each group of 8 adjacent
 *                     channels over the page's 16 tokens; group g is quantised and dequantised
 *                     with s_g = fl32(max_g/127), fl32(127/max_g) in place of the page's.  The
 *                     header's s and amax stay the page's.  Not in the paper, which has one scale.
 *   PTE       8 bytes per slot: bits 0-31 record offset in 64-byte units, 32-47 record
 *             length, 48-55 mode, bit 56 valid.  All-zero = never written.
 */
#ifndef SPECKV_H
#define SPECKV_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECKV_PAGE_TOKENS 16
#define SPECKV_HEAD_DIM 128
#define SPECKV_PAGE_BYTES 4096
#define SPECKV_L2_SLOTS 4 /* prefetch-buffer slots per sequence (prefetch depth k <= 4) */

/* host-side errors */
#define SPECKV_E_ARG (-1)    /* null pointer, size or index out of range, bad scheme */
#define SPECKV_E_CUDA (-2)   /* a CUDA runtime call failed (allocation, launch)      */
#define SPECKV_E_DEVICE (-3) /* the current device is not compute capability 10.x    */
#define SPECKV_E_TOO_LARGE (-4) /* more pages than a fixed-capacity entry point takes */

/* storage schemes / record modes */
enum { SPECKV_RAW = 0, SPECKV_INT8 = 1, SPECKV_INT8_DELTA = 2, SPECKV_INT8_DELTA_RLE = 3,
       /* scheme only, never a stored mode: adaptive selection (Sec. 3.6.3, compression selection, taken
        * per page): mode 3 where run-length coding makes the record smaller than mode 2, else mode 2 */
       SPECKV_AUTO = 4,
       /* flag, OR-ed into a scheme 1..4 (ignored with SPECKV_RAW) and into the stored mode: one scale
        * per group of 8 adjacent channels instead of one per page.  The paper's scaling step takes the
        * maximum over the whole block; a finer granularity keeps a few large channels from setting
        * the quantisation step of all the others. */
       SPECKV_GROUPED = 16 };

/* per-page conditions (index into speckv_status arrays) */
enum {
    SPECKV_ST_UNMAPPED = 1,   /* block-table entry -1 / out of range, or coordinates out of range */
    SPECKV_ST_BAD_PTE = 2,    /* slot has no valid page-table entry                               */
    SPECKV_ST_BAD_RECORD = 3, /* header inconsistent with the PTE / format, or outside the pool   */
    SPECKV_ST_POOL_FULL = 4,  /* record would end beyond pool_bytes; not written                  */
    SPECKV_ST_BAD_INDEX = 5,  /* src_page >= n_src_pages or dst_slot >= number of slots           */
    SPECKV_ST_TIMEOUT = 6,    /* an internal bounded wait gave up; the call's results are partial */
    SPECKV_ST_BAD_DST = 7,    /* destination page would lie outside dst_demand                    */
    SPECKV_N_STATUS = 8
};

typedef struct speckv_ctx speckv_ctx; /* opaque: pool, page table, cursor, prefetch tags, status, counters */

typedef struct {
    uint32_t n_layers, n_kv_heads, blocks_per_layer, max_blocks_per_seq, max_seqs;
    uint32_t reserved;   /* 0 */
    uint64_t pool_bytes; /* capacity of the record pool, multiple of 64 */
} speckv_config;

typedef struct { uint32_t seq; uint16_t layer; uint8_t kv /*0=K,1=V*/, head; uint32_t pos /*token*/; uint32_t rsvd; } speckv_vaddr;
typedef struct { uint64_t byte_off; uint32_t rec_len; uint8_t mode, status; uint16_t rsvd; } speckv_paddr;
typedef struct { uint32_t seq, block /*logical 16-token block*/, l2_slot /* < SPECKV_L2_SLOTS */; } speckv_prefetch;

typedef struct {
    uint32_t count[SPECKV_N_STATUS]; /* pages affected since the last clear, per condition   */
    uint32_t first[SPECKV_N_STATUS]; /* smallest page index affected (0xFFFFFFFF if none)    */
} speckv_status;

typedef struct {
    uint64_t pages_mode[4]; /* records written, per stored mode (without the GROUPED flag) */
    uint64_t granules;      /* 64-byte units appended to the pool                  */
    uint64_t payload_bytes; /* sum of payload_len of the records written           */
    uint64_t n_runs;        /* sum of n_runs of the mode-3 records written         */
    uint64_t nonfinite;     /* pages stored raw because they hold Inf or NaN       */
    uint64_t pages_decoded; /* pages delivered by speckv_decompress_gather         */
    uint64_t pf_issued;     /* prefetch entries fetched                            */
    uint64_t pf_skipped;    /* prefetch entries skipped because already resident   */
} speckv_stats;

/* Creates a context on the current device: allocates (cudaMalloc) and zeroes the pool
 * (pool_bytes), the page table (8 B per slot), the prefetch tags and small control blocks.
 * Synchronises the device.  cfg is HOST memory.  Limits (SPECKV_E_ARG beyond): n_kv_heads <= 255,
 * n_layers <= 4095, blocks_per_layer and max_blocks_per_seq < 2^20, max_seqs <= 4096,
 * max_seqs*max_blocks_per_seq*2*n_kv_heads < 2^31 (page indices are 32-bit), pool_bytes a multiple of 64
 * below 2^38.  Fails with SPECKV_E_DEVICE on a GPU that is
 * not sm_100.  speckv_destroy frees everything the context allocated. */
int speckv_create(speckv_ctx **out, const speckv_config *cfg);
int speckv_destroy(speckv_ctx *ctx);

/* Empties the context: cursor = 0, all PTEs and prefetch tags cleared, status and counters
 * cleared.  The pool bytes themselves are not rewritten.  Asynchronous on `stream`. */
int speckv_reset(speckv_ctx *ctx, void *stream);

/* Algorithm "KV-Cache Compression" (scale s = max|X|/127, INT8 quantisation with round to
 * nearest even of x*fl(127/max|X|), per-row delta mod 256, run-length coding) over a list of
 * pages.  Page i is read from src + 4096*src_page[i]; its record is appended at
 * cursor + sum of the sizes of records 0..i-1 of this call (list order, whatever the
 * scheduling), and PTE[dst_slot[i]] is overwritten.  The cursor advances by the size of all
 * records of the call, including those that did not fit (SPECKV_ST_POOL_FULL).  A page that
 * holds Inf or NaN is stored with mode 0 whatever the scheme.  dst_slot values in one call
 * should be distinct (otherwise the surviving PTE is unspecified).
 *   src          fp16 pages, 16-byte aligned          src_page, dst_slot   uint32[n]
 *   n_src_pages  number of pages readable at src      scheme  SPECKV_RAW .. SPECKV_AUTO,
 *                                                              optionally | SPECKV_GROUPED
 * n = 0 is a no-op; n may not exceed the context's number of slots (SPECKV_E_TOO_LARGE: the scan scratch
 * is sized once, at speckv_create, and the call never allocates or synchronises).
 * Calls on one context must be issued on one stream, or be ordered by
 * the caller, with these exceptions: reading calls (speckv_decompress_gather, speckv_translate,
 * speckv_attend_dense, speckv_decompress_attend) may run on other streams at the same time as
 * each other — provided their outputs do not overlap and at most one of them carries a prefetch
 * list — and at the same time as a speckv_compress whose dst_slot list shares no slot with what
 * they read: the compressor only appends behind the cursor and writes the entries of its own
 * slots.  (The host side of a context is not thread-safe: issue the calls from one thread.) */
int speckv_compress(speckv_ctx *ctx, const void *src, uint32_t n_src_pages, const uint32_t *src_page,
                    const uint32_t *dst_slot, uint32_t n, int scheme, void *stream);

/* Address translation unit (Sec. 3.5.1; Algorithm "Speculative KV-Cache Prefetching", the
 * TranslateAddress step): virtual (seq, layer, kv, head, pos) -> block = pos/16 ->
 * physical block = block_table[seq][block] -> slot -> PTE -> byte offset, length and mode of
 * the record.  pa[i].status = 0 or a SPECKV_ST_* code (then the other fields are 0).
 * Changes nothing but pa and the status block.
 *   block_table  int32 [max_seqs][max_blocks_per_seq], -1 = unmapped */
int speckv_translate(speckv_ctx *ctx, const int32_t *block_table, const speckv_vaddr *va, speckv_paddr *pa,
                     uint32_t n, void *stream);

/* Decompression (Sec. 3.5.3: run expansion, running sum of deltas, x = fp16(q*s); mode 0
 * bypasses) fused with the paged gather, for one layer.
 * Demand part: for every sequence b < B, every block n < ceil(seq_lens[b]/16), K and V, every
 * head: the page is written to dst_demand at element offset
 *   dst_tok_off[b]*2*H*128 + ((kv*H + head)*Tpad_b + 16*n)*128,  Tpad_b = 16*ceil(seq_lens[b]/16)
 * i.e. each sequence is a dense [2][H][Tpad_b][128] fp16 tensor starting at token row
 * dst_tok_off[b] (the caller normally passes the exclusive prefix sum of Tpad).  A sequence
 * whose rows would pass dst_cap_tokens is skipped (SPECKV_ST_BAD_DST).  A sequence longer than the
 * block table can describe (more than max_blocks_per_seq blocks) is reported once as
 * SPECKV_ST_UNMAPPED, at the page index its first page would have had, and left out altogether: none of
 * its pages is fetched and it takes no place in the page numbering (speckv_decompress_attend likewise:
 * its output rows are zero).
 * Prefetch part (the loop of the prefetching algorithm after token prediction): entry e
 * names logical block pf[e].block of sequence pf[e].seq; if the prefetch-buffer slot
 * (seq, l2_slot) is already tagged with this (layer, block) the entry is skipped, otherwise
 * its 2*H pages are written to dst_l2[seq][l2_slot][kv][head][16][128] and the slot is
 * retagged; a stale slot is simply overwritten.  (seq, l2_slot) pairs in one call must be
 * distinct.  The tag names the block, not the bytes: it does not notice that the block's slots were
 * compressed again since (a tail block that decode keeps filling), nor that dst_l2 is another buffer than
 * last time.  Pass the same dst_l2 for the life of the tags, and after rewriting a block that may sit in
 * the buffer clear its tag (speckv_l2_tag_ptr: a zero word = empty) or all tags (speckv_reset) — the lazy
 * invalidation of Sec. 3.4.3 is the overwrite by the next different block, nothing more.  dst_l2 must hold max_seqs*4*2*H pages; it may be NULL when n_pf = 0.
 * Page indices reported in the status block count demand pages first (sequence, block, kv,
 * head order) and then 2*H per prefetch entry.
 *   seq_lens uint32[B] tokens   dst_tok_off uint64[B] token rows   B <= max_seqs
 *
 * Ordering.  Work enqueued on `stream` after this call finds all pages of this call and of every earlier
 * call written, as stream order promises.  Consecutive calls on one stream overlap, though: the library
 * launches a gather so that it may start while the previous gather's last CTAs are still running
 * (programmatic dependent launch); it then reads its inputs and fetches records at once, and waits for
 * the previous gather before it writes a page or touches a residency tag — or, when the host has seen that
 * destinations are disjoint and there is no prefetch list, only before it ends.  Consequence for the caller:
 * block_table, seq_lens, dst_tok_off and pf of a call that directly follows another gather on the same
 * stream must not be produced by a kernel or copy enqueued between the two calls.  If they are, make any
 * other speckv call in between (speckv_clear_status will do: the next gather is then an ordinary launch),
 * or switch the overlap off for the context with speckv_set_gather_chaining(ctx, 0). */
int speckv_set_gather_chaining(speckv_ctx *ctx, int enabled); /* default 1; host-side setting */
int speckv_decompress_gather(speckv_ctx *ctx, uint32_t layer, const int32_t *block_table,
                             const uint32_t *seq_lens, const uint64_t *dst_tok_off, uint32_t B,
                             const speckv_prefetch *pf, uint32_t n_pf, void *dst_demand,
                             uint64_t dst_cap_tokens, void *dst_l2, void *stream);

/* End-to-end variants for callers whose K/V lives in HOST memory (pinned memory recommended).
 * speckv_compress_host copies n_src_pages pages from src_host (HOST) into staging (DEVICE,
 * >= n_src_pages*4096 bytes, 16-byte aligned) on `stream`, then runs speckv_compress on the
 * staged pages.  speckv_decompress_gather_host runs speckv_decompress_gather and then copies
 * the first copy_bytes bytes of dst_demand to dst_host (HOST).  Both are asynchronous with
 * respect to the host when the host buffers are pinned; the caller synchronises the stream
 * before reusing or reading the host buffers.  No counterpart in the paper, whose pool sits
 * behind the device interconnect; these exist so that transfers can be timed inside the call. */
int speckv_compress_host(speckv_ctx *ctx, const void *src_host, uint32_t n_src_pages, void *staging,
                         const uint32_t *src_page, const uint32_t *dst_slot, uint32_t n, int scheme, void *stream);
int speckv_decompress_gather_host(speckv_ctx *ctx, uint32_t layer, const int32_t *block_table,
                                  const uint32_t *seq_lens, const uint64_t *dst_tok_off, uint32_t B,
                                  const speckv_prefetch *pf, uint32_t n_pf, void *dst_demand,
                                  uint64_t dst_cap_tokens, void *dst_l2, void *dst_host, uint64_t copy_bytes,
                                  void *stream);

/* Pool lifecycle (no counterpart in the paper, whose pool is managed by its allocator plug-in): the
 * record log only grows, and a slot that is written again — a tail page rewritten as decode fills it —
 * leaves its old record behind.  speckv_compact rewrites the pool so that it holds exactly the
 * records that page-table entries point at, in slot order, each with its padding, from byte 0 on;
 * every entry gets its new offset and the cursor becomes the number of 64-byte units kept.  An
 * entry whose record is not inside the pool is reported (SPECKV_ST_BAD_RECORD, index = slot) and
 * cleared.  scratch: DEVICE memory, 256-byte aligned, at least speckv_compact_scratch_bytes(ctx)
 * bytes (pool_bytes + 8 bytes per slot + one bit per 64 bytes of pool + a little), contents undefined
 * afterwards.  Pool bytes behind the last record kept are unspecified.  Prefetch residency tags stay valid
 * (they name blocks, not offsets).
 *
 * speckv_free_slots gives slots back (a finished request's blocks): the listed page-table entries are
 * cleared, so the slots read as never written and their records are garbage that the next speckv_compact
 * drops.  freed (DEVICE uint64[2], optional, added to): [0] entries that were valid, [1] the 64-byte units
 * their records occupy.  A slot listed twice counts once; slots[i] beyond the table is reported as
 * SPECKV_ST_BAD_INDEX with index i.  Prefetch-buffer tags of the freed blocks are the caller's to clear. */
int speckv_free_slots(speckv_ctx *ctx, const uint32_t *slots, uint32_t n, uint64_t *freed, void *stream);
uint64_t speckv_compact_scratch_bytes(speckv_ctx *ctx);
int speckv_compact(speckv_ctx *ctx, void *scratch, uint64_t scratch_bytes, void *stream);

/* The per-layer computation that consumes the fetched pages: decode-step attention, one query
 * token per sequence (the T_layer stage that the multi-layer prefetch pipeline of Sec. 3.4.4
 * overlaps with the fetches of layers l+1 and l+2; the paper does not describe the computation
 * itself, this is the standard one):
 *   out[b][hq][:] = sum_t softmax_t(q[b][hq] . K[t] / sqrt(128)) V[t],   t < seq_lens[b],
 * query head hq reading KV head hq / (n_q_heads / n_kv_heads).  Scores and softmax in binary32,
 * probabilities rounded to binary16 for the weighted sum, result rounded to binary16.
 *   q, out        fp16 [B][n_q_heads][128], 16-byte aligned; n_q_heads a multiple of n_kv_heads,
 *                 at most 8 query heads per KV head; B <= 512
 *   workspace     at least speckv_attend_workspace_bytes(B, n_kv_heads) bytes (about 35 MB plus
 *                 4 KB per sequence and KV head), 256-byte aligned; scratch for the call,
 *                 contents undefined afterwards
 * A sequence of length 0 gives zero output rows.
 *
 * speckv_attend_dense reads K and V from kv = the dst_demand workspace that
 * speckv_decompress_gather wrote with the same seq_lens and dst_tok_off.
 *
 * speckv_decompress_attend fetches the pages itself — block table -> PTE -> record ->
 * decompression pipeline of Sec. 3.5.3 into shared memory — so the decompressed K/V never reach
 * device memory.  A page that cannot be delivered is counted in the status block exactly as
 * speckv_decompress_gather would count it (same page numbering), and the 16 tokens of its block
 * take no part in the softmax.  Pages decoded are added to the pages_decoded counter. */
uint64_t speckv_attend_workspace_bytes(uint32_t B, uint32_t n_kv_heads);
int speckv_attend_dense(speckv_ctx *ctx, const void *kv, const uint32_t *seq_lens, const uint64_t *dst_tok_off,
                        uint32_t B, const void *q, uint32_t n_q_heads, void *out, void *workspace,
                        uint64_t workspace_bytes, void *stream);
int speckv_decompress_attend(speckv_ctx *ctx, uint32_t layer, const int32_t *block_table, const uint32_t *seq_lens,
                             uint32_t B, const void *q, uint32_t n_q_heads, void *out, void *workspace,
                             uint64_t workspace_bytes, void *stream);

/* Compression selection per layer (Sec. 3.6.3, policy engine):
 *     C*(l,t) = argmax_{C in CC}  w_r R_c(C,l) + w_q Q(C,l) - w_c L_comp(C)    subject to  Q(C,l) >= Q_min.
 * The paper leaves CC, Q and L_comp open.  Here CC = the schemes 1, 2, 3, 4 with one scale per page followed
 * by the same four with SPECKV_GROUPED (candidate index 0..7, the order that breaks ties); R_c = uncompressed
 * bytes / stored bytes (64-byte units) of a sample of the layer's pages; Q = signal-to-quantisation-noise
 * ratio of that sample in decibels, 10 log10(sum x^2 / sum (x - decoded x)^2), capped at 200; L_comp(C) and
 * the weights are the caller's numbers (the paper updates its weights by gradient steps on a throughput
 * reward that only a serving system has).
 *
 * speckv_probe_pages measures the sample on the GPU: page i of the list is read from src + 4096*src_page[i],
 * quantised with both scale granularities, its delta symbols' run heads are counted, and `out` (DEVICE, zeroed
 * by the caller before the first call for a layer, added to by every call) receives what the pages would
 * occupy under each candidate and the squared errors.  Pages holding Inf or NaN (stored raw by every scheme)
 * and list entries >= n_src_pages are only counted.  Stateless: needs no context.  Integer fields are exact;
 * the three sums are binary64 sums of exact terms in an unspecified order.
 *
 * speckv_select_scheme (HOST arithmetic, binary64; probe and policy in HOST memory) returns the scheme to
 * pass to speckv_compress for that layer: the candidate with the largest objective among those with
 * Q >= q_min, the earlier one on a tie; if none qualifies, the earliest candidate of the best quality.
 * objective (optional, HOST double[8]) receives every candidate's value.  SPECKV_E_ARG for an empty sample. */
#define SPECKV_N_CANDIDATES 8
typedef struct {
    uint64_t pages, nonfinite, bad_index;    /* measured / skipped for Inf, NaN / list entries out of range */
    uint64_t granules[SPECKV_N_CANDIDATES];  /* 64-byte units the measured pages take under each candidate  */
    double sq_err[2];                        /* sum (x - decoded x)^2: one scale per page, per channel group */
    double sq_sum;                           /* sum x^2                                                     */
} speckv_probe;
typedef struct { double w_r, w_q, w_c, q_min; double cost[SPECKV_N_CANDIDATES]; } speckv_policy;
int speckv_probe_pages(const void *src, uint32_t n_src_pages, const uint32_t *src_page, uint32_t n, speckv_probe *out,
                       void *stream);
int speckv_select_scheme(const speckv_probe *probe, const speckv_policy *policy, double *objective);

/* Multi-layer pipelined prefetch (Sec. 3.4.4: "while computing layer l, prefetch for layers l+1 and l+2",
 * T_effective = T_compute + max(T_prefetch - 2 T_layer, 0)).  The call owns the schedule: a fetch stream
 * of the context runs speckv_decompress_gather for layers layer0 .. layer0+n_layers-1 into a ring of
 * ring_slots demand workspaces (slot r = ring + r*slot_tokens*2*H*128*2 bytes, each with room for
 * slot_tokens token rows; 3 slots = the layer in use and two ahead), and for each layer, once its pages
 * are there, calls consume(user, layer, slot, stream), which enqueues that layer's computation on `stream`
 * and returns 0 (anything else ends the call and is returned).  A slot is refilled only after the
 * computation that read it has finished; the first gather starts after the work already enqueued on
 * `stream`.  Everything is enqueued; the call returns without synchronising.  On return, work enqueued on
 * `stream` follows all of it.  The first call on a context creates the fetch stream and its events (no
 * device memory) and should come before any stream capture.  seq_lens, dst_tok_off, block_table as for
 * speckv_decompress_gather (one set for all layers); no prefetch list.
 *
 * speckv_pipeline_attend is the same with the library's own per-layer computation, decode-step attention
 * over the fetched workspace:  q, out  fp16 [n_layers][B][n_q_heads][128]; workspace as for
 * speckv_attend_dense (shared by the layers, which run one after the other on `stream`). */
typedef int (*speckv_layer_fn)(void *user, uint32_t layer, const void *kv, void *stream);
int speckv_pipeline_layers(speckv_ctx *ctx, uint32_t layer0, uint32_t n_layers, const int32_t *block_table,
                           const uint32_t *seq_lens, const uint64_t *dst_tok_off, uint32_t B, void *ring,
                           uint32_t ring_slots, uint64_t slot_tokens, speckv_layer_fn consume, void *user, void *stream);
int speckv_pipeline_attend(speckv_ctx *ctx, uint32_t layer0, uint32_t n_layers, const int32_t *block_table,
                           const uint32_t *seq_lens, const uint64_t *dst_tok_off, uint32_t B, void *ring,
                           uint32_t ring_slots, uint64_t slot_tokens, const void *q, uint32_t n_q_heads, void *out,
                           void *workspace, uint64_t workspace_bytes, void *stream);

/* Managed prefetch buffer: the paper's tier L2 with its double buffering (Sec. 3.3.1), its handling
 * of mispredictions (Sec. 3.4.3: lazy invalidation, fallback to a synchronous fetch, prefetch depth
 * adapted per request) and the depth rule of Sec. 3.6.3,
 *     k* = argmax_k  mu_k + beta * sqrt(2 ln T / N_k),
 * one decode step of one layer per call.  The buffer has two banks of 4 slots per sequence; a slot
 * holds the 2*H decompressed pages of one logical block.  A call fills bank `back` and serves reads
 * only from the other bank, which the previous call filled — so the pages a call writes are never the
 * pages its caller is reading, and the caller alternates back = 0, 1, 0, ...
 * Per sequence b < B, in this order:
 *   1. reads: for each block access[b][a] >= 0, where[b][a] = bank*4 + slot if the readable bank holds
 *      it (the slot is marked used), else -1 and its 2*H pages are fetched from the pool into
 *      miss_dst[b][a] (the fallback path); -2 where there was nothing to read.
 *   2. the fill that bank `back` received two calls ago is scored for the depth d it used:
 *      reward[d] += 2 per requested block that was read, -1 per requested block that was not
 *      (the paper leaves the reward open); plays[d] += 1, steps += 1.
 *   3. depth k: the smallest depth not yet scored, else the rule above with mu_k = reward_k/(8*plays_k),
 *      T = steps, ln T rounded to 20 fractional bits, binary64 with one rounding per operation,
 *      ties to the smaller depth.
 *   4. refill: the first k predictions cand[b][j] (best first, -1 = none) go to slots j < k of bank
 *      `back`.  A slot that already holds the predicted block is kept (no transfer); anything else is
 *      overwritten, which is the only form of invalidation; slots from k on stay as they are.  A
 *      prediction whose block is not mapped leaves its slot alone (2*H pages SPECKV_ST_UNMAPPED).
 * Page numbers in the status block: (b*4 + a)*2H + r for reads, ((B + b)*4 + j)*2H + r for refills.
 *   access, cand  int32 [B][4]           state   speckv_pf_seq [>= B], zeroed by the caller before first use
 *   where         int32 [B][4]           cnt     speckv_pf_counters, zeroed by the caller; the call adds
 *   l2            fp16 [2][max_seqs][4][2][H][16][128]     miss_dst  fp16 [B][4][2][H][16][128]
 *   B <= 512; every pointer 16-byte aligned; one state array per layer if layers are to keep separate depths.
 *   Calls that share state, cnt, where, miss_dst or a bank of l2 must be ordered (one stream); the caller reads
 *   the hit slots named by `where` from bank back^1 and must be done with them before the next call but one
 *   refills that bank.
 * hit rate = hits/accesses, coverage = (hits + late)/accesses, precision = evicted_used/evicted
 * (the rows of the paper's prefetch-statistics table; its latencies are those of its own link). */
typedef struct {
    uint32_t tag[2][SPECKV_L2_SLOTS];  /* [bank][slot]: layer*2^20 + block + 1; 0 = empty             */
    uint8_t used[2][SPECKV_L2_SLOTS];  /* read since the slot was last requested                     */
    uint8_t depth[2];                  /* depth the bank was last filled with; 0 = never             */
    uint8_t fill;                      /* bit j: slot j of bank `back` was transferred by the last call */
    uint8_t rsvd;
    uint32_t steps;                    /* T: fills scored so far                                     */
    uint32_t plays[SPECKV_L2_SLOTS];   /* N_k                                                        */
    int32_t reward[SPECKV_L2_SLOTS];   /* reward sum of depth k                                      */
} speckv_pf_seq;
typedef struct {
    uint64_t accesses, hits, late, misses; /* late: missed although the bank being written holds the block */
    uint64_t fetched, kept;                /* refill: transferred / already in its slot                    */
    uint64_t evicted, evicted_used;        /* slots overwritten / of those, read before                    */
    uint64_t pages;                        /* pages delivered (reads that missed + refills)                */
    uint64_t rsvd;
} speckv_pf_counters;
int speckv_prefetch_step(speckv_ctx *ctx, uint32_t layer, uint32_t back, const int32_t *block_table,
                         const int32_t *access, const int32_t *cand, uint32_t B, double beta,
                         speckv_pf_seq *state, speckv_pf_counters *cnt, void *l2, void *miss_dst,
                         int32_t *where, void *stream);

/* Compression for callers that must not allocate device memory.  (No counterpart in the paper:
 * its engine owns fixed on-chip buffers; this is the same compressor with a fixed scratch area.)
 *
 * Who needs it: code that runs where cudaMalloc/cudaFree are off limits — inside a serving
 * engine that has handed all device memory to its own pool allocator at start-up, inside a
 * region where an allocation would synchronise the device or fragment a carefully sized heap,
 * or in a plug-in that is only ever given buffers.  speckv_create allocates the pool, the page
 * table and the scan scratch; this call allocates nothing and needs no context: the caller
 * passes every buffer, and the scan scratch (a ticket counter and one 8-byte word per tile of 16 or
 * 20 pages) is a fixed array inside the library, 256 KiB, present on every GPU that loads the
 * library until the process ends.
 *
 * Same operation, record format, placement rule and status reporting as speckv_compress.
 *   pool, pool_bytes  DEVICE record log (64-byte aligned; multiple of 64 bytes)
 *   pte, n_slots      DEVICE page table, uint64[n_slots]; the caller zeroes it before first use
 *   ctl               DEVICE control block (cursor, status, counters), read and updated by the call;
 *                     before first use the caller sets it to zero and status `first` words to
 *                     0xFFFFFFFF (cudaMemset calls on its own buffer)
 *   n                 at most SPECKV_STATIC_MAX_PAGES pages per call, else SPECKV_E_TOO_LARGE
 * The first call on a device looks up the address of the fixed array (no allocation) and should
 * therefore be made before any stream capture begins; that look-up is serialised, so first calls from
 * several host threads are safe.  ctl and pte must be 8-byte aligned, src_page and dst_slot 4-byte
 * aligned (SPECKV_E_ARG otherwise).  All calls on a device share the array: each
 * call clears the part it uses, and two calls whose kernels could overlap on the GPU (different
 * streams without ordering, several host threads) would corrupt each other's scan — issue them on
 * one stream or order them. */
#define SPECKV_STATIC_MAX_PAGES 524288u
typedef struct {
    uint64_t cursor64;                 /* next free 64-byte unit of the pool */
    uint32_t count[SPECKV_N_STATUS];   /* as speckv_status.count             */
    uint32_t first[SPECKV_N_STATUS];   /* as speckv_status.first             */
    uint64_t stats[11];                /* as speckv_stats, in field order    */
} speckv_ctl_block;
int speckv_compress_static(const void *src, uint32_t n_src_pages, const uint32_t *src_page,
                           const uint32_t *dst_slot, uint32_t n, int scheme, void *pool, uint64_t pool_bytes,
                           uint64_t *pte, uint64_t n_slots, speckv_ctl_block *ctl, void *stream);

/* Status block and counters (HOST out).  Both synchronise `stream` first. */
int speckv_get_status(speckv_ctx *ctx, speckv_status *out, void *stream);
int speckv_get_stats(speckv_ctx *ctx, speckv_stats *out, void *stream);
int speckv_clear_status(speckv_ctx *ctx, void *stream); /* status and counters; asynchronous */

/* Every wait inside the kernels is bounded (the engine's failure mode "a request that never completes"
 * must come back as a status, never as a kernel that does not end): the compressor's scan polls the
 * sizes of earlier tiles at most lookback_polls times per window of 64 tiles (>= 200 ns per poll), and
 * a warp waits at most wait_ns nanoseconds on a shared-memory barrier.  A wait that runs out is counted
 * as SPECKV_ST_TIMEOUT (index = first page of the tile whose place in the log could not be computed,
 * or 0xFFFFFFF0..0xFFFFFFF3 for a barrier wait of an encoder, a record stage, the loader, the scanner);
 * the tiles behind it in list order are not placed, their page-table entries and the cursor stay as they
 * were, and the call still ends.  Defaults: 4,194,304 polls and 2 s; 0 selects the default.  Host-side
 * setting of the context, applies to later speckv_compress calls.  No counterpart in the paper. */
int speckv_set_wait_limits(speckv_ctx *ctx, uint32_t lookback_polls, uint64_t wait_ns);

/* Fault injection for tests of those limits, made on the host: the next speckv_compress call (only)
 * never hands out its first n_tiles tiles (20 pages each; 16 with SPECKV_RAW), as if the CTAs that drew them had stalled.
 * Every later tile then waits for sizes that are never published, until its limit runs out.  Nothing
 * faults or traps; combine with short limits.  n_tiles = 0 cancels. */
int speckv_inject_missing_tiles(speckv_ctx *ctx, uint32_t n_tiles);

/* Introspection for tools and tests.  Device pointers stay owned by the context. */
void *speckv_pool_ptr(speckv_ctx *ctx);       /* uint8  [pool_bytes]                       */
void *speckv_pte_ptr(speckv_ctx *ctx);        /* uint64 [n_layers*blocks_per_layer*2*H]    */
void *speckv_l2_tag_ptr(speckv_ctx *ctx);     /* uint64 [max_seqs*4]: epoch<<32 | tag      */
int speckv_get_cursor(speckv_ctx *ctx, uint64_t *cursor64 /*HOST*/, void *stream); /* synchronises */
const char *speckv_version(void);

#ifdef __cplusplus
}
#endif
#endif
