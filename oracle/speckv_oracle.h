/*
 * CPU oracle for the KV page codec of CXL-SpecKV (compression Algorithm
 * "KV-Cache Compression", the decompression pipeline of Sec. 3.5.3, the
 * address translation unit of Sec. 3.5.1 and the prefetch loop of Algorithm
 * "Speculative KV-Cache Prefetching").
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, single-threaded C that follows the
 * paper's steps one by one.  It shares no code, header, table or constant
 * with the CUDA library; only tests, the smoke check and the CPU-baseline
 * leg of the benchmark may call it.
 *
 * Parity pins: every function below is pinned by the CPU tests against
 * closed forms, brute force and a hand-worked page, EXCEPT the compression
 * ratios the paper reports for real KV tensors (2.73x with delta, 3.21x with
 * RLE, range 2.5-4.0): those depend on data that is not available and are
 * "parity unpinned".
 */
#ifndef SPECKV_ORACLE_H
#define SPECKV_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* record modes = the four rows of the paper's compression ablation table */
enum { OKV_RAW = 0, OKV_INT8 = 1, OKV_INT8_DELTA = 2, OKV_INT8_DELTA_RLE = 3,
       OKV_AUTO = 4 /* a scheme, never a stored mode: per page the smaller of modes 2 and 3 */ };

/* Scale granularity (not in the paper, which has one scale per page): OR-ed into a scheme or a
 * stored mode 1-3, it gives every group of 8 adjacent channels (over the 16 tokens of the page)
 * its own scale.  The groups' largest magnitudes (binary16 patterns, d/8 of them) then precede
 * the mode's payload, and each group's scale is derived from its magnitude like the page's. */
enum { OKV_GROUPED = 16, OKV_GROUP_CHANNELS = 8 };

/* per-page conditions a call can report (index into okv_status arrays) */
enum {
    OKV_ST_UNMAPPED = 1,   /* block table entry missing or out of range      */
    OKV_ST_BAD_PTE = 2,    /* page slot never written                        */
    OKV_ST_BAD_RECORD = 3, /* header inconsistent or record outside the pool */
    OKV_ST_POOL_FULL = 4,  /* record does not fit behind the cursor          */
    OKV_ST_BAD_INDEX = 5,  /* source page / destination slot out of range    */
    OKV_ST_TIMEOUT = 6,    /* never raised by the oracle                     */
    OKV_ST_BAD_DST = 7,    /* destination page outside the output buffer     */
    OKV_N_STATUS = 8
};

typedef struct {
    uint32_t count[OKV_N_STATUS]; /* pages affected, per condition   */
    uint32_t first[OKV_N_STATUS]; /* smallest index affected, or ~0u */
} okv_status;

typedef struct {
    uint64_t pages_mode[4]; /* records written, per stored mode          */
    uint64_t granules;      /* 64-byte granules appended to the pool     */
    uint64_t payload_bytes; /* sum of payload_len over records written   */
    uint64_t n_runs;        /* sum of n_runs over mode-3 records written */
    uint64_t nonfinite;     /* pages stored raw because of Inf/NaN       */
    uint64_t pages_decoded; /* pages written by decompress_gather        */
    uint64_t pf_issued;     /* prefetch entries fetched                  */
    uint64_t pf_skipped;    /* prefetch entries already resident         */
} okv_stats;

typedef struct {
    uint32_t n_layers, n_kv_heads, blocks_per_layer, max_blocks_per_seq, max_seqs;
    uint32_t reserved;
    uint64_t pool_bytes;
} okv_config;

typedef struct { uint32_t seq; uint16_t layer; uint8_t kv, head; uint32_t pos; uint32_t rsvd; } okv_vaddr;
typedef struct { uint64_t byte_off; uint32_t rec_len; uint8_t mode, status; uint16_t rsvd; } okv_paddr;
typedef struct { uint32_t seq, block, l2_slot; } okv_prefetch;

/* ---- scalar building blocks ------------------------------------------- */
float    okv_half_to_float(uint16_t h);
uint16_t okv_float_to_half(float f);

/* ---- one page (N tokens x d channels, N*d a multiple of 8, <= 2048) ---- */
/* Writes header + payload (no padding) to rec, returns rec_len in bytes.  */
uint32_t okv_compress_page(const uint16_t *x, uint32_t N, uint32_t d, int scheme, uint8_t *rec);
/* Intermediate results of the same algorithm, for tests (any may be NULL). */
void okv_page_stages(const uint16_t *x, uint32_t N, uint32_t d, uint16_t *amax_bits, float *s,
                     float *inv, int8_t *q, uint8_t *sym, uint8_t *bitmap, uint8_t *values,
                     uint32_t *n_runs);
/* The same with one scale per channel group (d a multiple of 8); group_amax gets d/8 entries. */
void okv_page_stages_grouped(const uint16_t *x, uint32_t N, uint32_t d, uint16_t *group_amax,
                             int8_t *q, uint8_t *sym, uint8_t *bitmap, uint8_t *values,
                             uint32_t *n_runs);
/* Returns 0, or OKV_ST_BAD_RECORD if the header is inconsistent. */
int okv_decompress_record(const uint8_t *rec, uint32_t avail, uint32_t N, uint32_t d, uint16_t *out);

/* ---- pool level (pages are 16 x 128) ----------------------------------- */
void okv_status_clear(okv_status *st);
int okv_compress(const okv_config *cfg, uint8_t *pool, uint64_t *pte, uint64_t *cursor64,
                 const uint16_t *src, uint32_t n_src_pages, const uint32_t *src_page,
                 const uint32_t *dst_slot, uint32_t n, int scheme, okv_status *st, okv_stats *stats);
/* Pool lifecycle, not in the paper (whose pool is managed by its allocator): drops the records that
 * no page-table entry points at and packs the rest in slot order.  scratch: pool_bytes bytes. */
int okv_compact(const okv_config *cfg, uint8_t *pool, uint64_t *pte, uint64_t *cursor64,
                uint8_t *scratch, okv_status *st);
/* ---- compression selection per layer (Sec. 3.6.3) ----------------------- */
/* The paper gives the form  C*(l,t) = argmax_C  w_r R_c(C,l) + w_q Q(C,l) - w_c L_comp(C)  s.t. Q >= Q_min
 * and leaves the candidate set, Q and L_comp open.  Here: candidates = schemes 1-4 with one scale per
 * page, then the same four with one scale per channel group; R_c = stored ratio on a sample of the
 * layer's pages; Q = signal-to-quantisation-noise ratio of the sample in dB; L_comp and the weights are
 * the caller's numbers. */
enum { OKV_N_CANDIDATES = 8 };
typedef struct {
    uint64_t pages, nonfinite, bad_index; /* pages measured / skipped (Inf, NaN) / list entries out of range */
    uint64_t granules[OKV_N_CANDIDATES];  /* 64-byte granules the measured pages take under each candidate */
    double sq_err[2];                     /* sum of (x - decoded x)^2: page scale, grouped scales */
    double sq_sum;                        /* sum of x^2 */
} okv_probe;
typedef struct { double w_r, w_q, w_c, q_min; double cost[OKV_N_CANDIDATES]; } okv_policy;
int okv_probe_pages(const uint16_t *src, uint32_t n_src_pages, const uint32_t *src_page, uint32_t n,
                    okv_probe *out);
double okv_probe_quality(const okv_probe *p, int grouped);
int okv_select_scheme(const okv_probe *p, const okv_policy *pol, double *objective);

int okv_free_slots(const okv_config *cfg, uint64_t *pte, const uint32_t *slots, uint32_t n,
                   uint64_t *freed, okv_status *st);
int okv_translate(const okv_config *cfg, const uint64_t *pte, const int32_t *block_table,
                  const okv_vaddr *va, okv_paddr *pa, uint32_t n, okv_status *st);
int okv_decompress_gather(const okv_config *cfg, const uint8_t *pool, const uint64_t *pte,
                          uint64_t *l2_tag, uint32_t epoch, uint32_t layer,
                          const int32_t *block_table, const uint32_t *seq_lens,
                          const uint64_t *dst_tok_off, uint32_t B, const okv_prefetch *pf,
                          uint32_t n_pf, uint16_t *dst_demand, uint64_t dst_cap_tokens,
                          uint16_t *dst_l2, okv_status *st, okv_stats *stats);


/* ---- the per-layer computation that consumes the fetched pages --------- */
/* Decode-step attention (the T_layer stage of the multi-layer prefetch pipeline, Sec. 3.4.4), one
 * query token per sequence, binary64 arithmetic on the binary16 inputs:
 *   out[b][hq][:] = sum_t softmax_t(q[b][hq] . K[t] / sqrt(128)) V[t],  t < seq_lens[b],
 * query head hq reading KV head hq / (Hq / H).  q: [B][Hq][128] binary16; out: [B][Hq][128] double.
 * okv_attend_dense reads K/V from the demand workspace written by okv_decompress_gather;
 * okv_attend fetches the pages itself (translate, decompress), reports pages it cannot deliver with
 * the demand fetch's page numbering and leaves their blocks out of the softmax; every page it
 * delivers is counted in pages_decoded. */
int okv_attend_dense(const uint16_t *kv, const uint32_t *seq_lens, const uint64_t *tok_off, uint32_t B,
                     uint32_t H, const uint16_t *q, uint32_t Hq, double *out);
int okv_attend(const okv_config *cfg, const uint8_t *pool, const uint64_t *pte, uint32_t layer,
               const int32_t *block_table, const uint32_t *seq_lens, uint32_t B, const uint16_t *q,
               uint32_t Hq, double *out, okv_status *st, okv_stats *stats);

/* ---- managed prefetch buffer ------------------------------------------- */
/* The paper's tier L2 with its double buffering (Sec. 3.3.1), the misprediction handling of
 * Sec. 3.4.3 (lazy invalidation, fallback fetch, depth adapted per request) and the depth rule of
 * Sec. 3.6.3, k* = argmax_k mu_k + beta*sqrt(2 ln T / N_k).  The buffer has two banks of
 * OKV_PF_SLOTS slots per sequence; a step fills one bank (`back`) while the other one, filled
 * during the previous step, is the only one that may be read.  The paper defines neither the
 * reward nor the bank discipline; both are spelled out at the implementation.
 *   access [B][4]   logical blocks sequence b reads in this step (-1 = none)
 *   cand   [B][4]   blocks predicted for the next step, best first (-1 = none)
 *   l2     fp16 [2][max_seqs][4][2][H][16][128]     miss_dst fp16 [B][4][2][H][16][128]
 *   where  [B][4]   bank*4 + slot if the read is served from the buffer, -1 if it was fetched into
 *                   miss_dst, -2 if there was nothing to read
 * Page numbering of the status block: ((b*4 + a)*2H + r) for reads, ((B + b)*4 + j)*2H + r for
 * refills. */
enum { OKV_PF_SLOTS = 4, OKV_PF_ACCESSES = 4 };
typedef struct {
    uint32_t tag[2][OKV_PF_SLOTS];   /* layer*2^20 + block + 1; 0 = empty                  */
    uint8_t used[2][OKV_PF_SLOTS];   /* read since the slot was last requested             */
    uint8_t depth[2];                /* depth the bank was last filled with; 0 = never     */
    uint8_t fill;                    /* bit j: slot j of the back bank was transferred in the last step */
    uint8_t rsvd;
    uint32_t steps;                  /* T: fills scored so far                             */
    uint32_t plays[OKV_PF_SLOTS];    /* N_k                                                */
    int32_t reward[OKV_PF_SLOTS];    /* reward sum of depth k                              */
} okv_pf_seq;
typedef struct {
    uint64_t accesses, hits, late, misses; /* late: missed, although the other bank holds it */
    uint64_t fetched, kept;                /* refill: transferred / already in its slot      */
    uint64_t evicted, evicted_used;        /* overwritten slots / of those, read before      */
    uint64_t pages;                        /* pages delivered by the step calls              */
    uint64_t rsvd;
} okv_pf_counters;
double okv_pf_score(int32_t reward, uint32_t plays, uint32_t steps, double beta);
uint32_t okv_pf_choose_depth(const okv_pf_seq *s, double beta);
int okv_prefetch_step(const okv_config *cfg, const uint8_t *pool, const uint64_t *pte, uint32_t layer,
                      uint32_t back, const int32_t *block_table, const int32_t *access,
                      const int32_t *cand, uint32_t B, double beta, okv_pf_seq *state,
                      okv_pf_counters *cnt, uint16_t *l2, uint16_t *miss_dst, int32_t *where,
                      okv_status *st, okv_stats *stats);

#ifdef __cplusplus
}
#endif
#endif
