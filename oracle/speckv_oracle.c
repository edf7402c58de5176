/*
 * CPU oracle for the CXL-SpecKV page codec.  TEST INFRASTRUCTURE ONLY: see
 * speckv_oracle.h.  Build: gcc -O1 -std=c11 -ffp-contract=off -fPIC -shared.
 *
 * Every step is written the way the paper states it, with the readings that
 * the paper leaves open spelled out next to the step.  Nothing here is
 * blocked, fused or reordered.
 */
#include "speckv_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#define PAGE_N 16u
#define PAGE_D 128u
#define PAGE_ELEMS (PAGE_N * PAGE_D)
#define PAGE_BYTES (PAGE_ELEMS * 2u)
#define HDR_BYTES 16u
#define GRANULE 64u
#define FORMAT_VERSION 1u
#define L2_SLOTS 4u
#define MAX_ELEMS 2048u

/* ---------------------------------------------------------------------- */
/* IEEE binary16 <-> binary32, by the format's definition                  */
/* ---------------------------------------------------------------------- */

float okv_half_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    uint32_t e = (uint32_t)(h >> 10) & 0x1Fu;
    uint32_t m = (uint32_t)h & 0x3FFu;
    double v;
    if (e == 31u) {
        uint32_t bits = (sign << 31) | 0x7F800000u | (m << 13);
        float f;
        memcpy(&f, &bits, 4);
        return f;
    }
    if (e == 0u)
        v = ldexp((double)m, -24); /* subnormal: m * 2^-24 */
    else
        v = ldexp((double)(1024u + m), (int)e - 25); /* (1 + m/1024) * 2^(e-15) */
    return (float)(sign ? -v : v); /* exact: every binary16 value is a binary32 value */
}

uint16_t okv_float_to_half(float f)
{
    /* round to nearest, ties to even */
    uint32_t x;
    memcpy(&x, &f, 4);
    uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
    uint32_t a = x & 0x7FFFFFFFu;
    if (a > 0x7F800000u) return (uint16_t)(sign | 0x7E00u | ((a >> 13) & 0x3FFu)); /* NaN */
    if (a >= 0x47800000u) return (uint16_t)(sign | 0x7C00u); /* >= 65536 or Inf -> Inf */
    uint32_t e = a >> 23;
    uint32_t m = a & 0x7FFFFFu;
    uint32_t h, rem, half;
    if (e >= 113u) { /* result is normal (or rounds up to Inf): keep 10 of 23 fraction bits */
        h = ((e - 112u) << 10) | (m >> 13);
        rem = m & 0x1FFFu;
        half = 0x1000u;
    } else { /* result is subnormal: units of 2^-24 */
        uint32_t shift = 126u - e;
        if (shift > 24u) return sign;
        m |= 0x800000u;
        h = m >> shift;
        rem = m & ((1u << shift) - 1u);
        half = 1u << (shift - 1u);
    }
    if (rem > half || (rem == half && (h & 1u))) h += 1u; /* a carry into the exponent is correct */
    return (uint16_t)(sign | h);
}

/* ---------------------------------------------------------------------- */
/* Algorithm "KV-Cache Compression", one page                              */
/* ---------------------------------------------------------------------- */

static void put16(uint8_t *p, uint32_t v) { p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8); }
static void put32(uint8_t *p, uint32_t v) { put16(p, v & 0xFFFFu); put16(p + 2, v >> 16); }
static uint32_t get16(const uint8_t *p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8); }
static uint32_t get32(const uint8_t *p) { return get16(p) | (get16(p + 2) << 16); }

/* Scale of one quantisation group from its largest magnitude (a finite binary16 pattern). */
static void group_scale(uint16_t amax_bits, float *s_out, float *inv_out)
{
    volatile float amax = okv_half_to_float(amax_bits);
    volatile float s = 0.0f, inv = 0.0f;
    if (amax_bits != 0 && amax_bits < 0x7C00u) {
        s = amax / 127.0f;   /* binary32 division */
        inv = 127.0f / amax; /* the quantiser multiplies by fl(127/amax) instead of dividing by s */
    }
    *s_out = s;
    *inv_out = inv;
}

/* All stages of the algorithm.  group_amax == NULL: one scale for the page (the paper's
 * scaling step).  Otherwise one scale per group of OKV_GROUP_CHANNELS adjacent channels, taken
 * over all token rows of the page, and group_amax[g] receives the group's largest magnitude. */
static void page_stages(const uint16_t *x, uint32_t N, uint32_t d, uint16_t *amax_bits_out,
                        float *s_out, float *inv_out, uint16_t *group_amax, int8_t *q, uint8_t *sym,
                        uint8_t *bitmap, uint8_t *values, uint32_t *n_runs_out)
{
    uint32_t n_el = N * d;
    /* Scaling step: s = max|X| / 127.  |x| ordering of finite binary16 values is the
     * ordering of their bit patterns with the sign cleared. */
    uint16_t amax_bits = 0;
    for (uint32_t k = 0; k < n_el; ++k) {
        uint16_t a = x[k] & 0x7FFFu;
        if (a > amax_bits) amax_bits = a;
    }
    float s, inv;
    group_scale(amax_bits, &s, &inv);
    if (amax_bits_out) *amax_bits_out = amax_bits;
    if (s_out) *s_out = s;
    if (inv_out) *inv_out = inv;
    if (amax_bits >= 0x7C00u) { /* Inf/NaN present: page is stored uncompressed, no later stage */
        if (n_runs_out) *n_runs_out = 0;
        return;
    }

    /* Scale per element: the page's, or that of the element's channel group. */
    float inv_of_channel[MAX_ELEMS];
    for (uint32_t i = 0; i < d; ++i) inv_of_channel[i] = inv;
    if (group_amax) {
        for (uint32_t g = 0; g < d / OKV_GROUP_CHANNELS; ++g) {
            uint16_t ga = 0;
            for (uint32_t j = 0; j < N; ++j)
                for (uint32_t c = 0; c < OKV_GROUP_CHANNELS; ++c) {
                    uint16_t a = x[j * d + g * OKV_GROUP_CHANNELS + c] & 0x7FFFu;
                    if (a > ga) ga = a;
                }
            group_amax[g] = ga;
            float gs, ginv;
            group_scale(ga, &gs, &ginv);
            for (uint32_t c = 0; c < OKV_GROUP_CHANNELS; ++c) inv_of_channel[g * OKV_GROUP_CHANNELS + c] = ginv;
        }
    }

    /* Quantisation loop: x_int8 = round(x * 127 / max|X|), nearest with ties to even, taken
     * on the exact product x * inv (11-bit by 24-bit significands: exact in binary64). */
    int8_t qbuf[MAX_ELEMS];
    for (uint32_t j = 0; j < N; ++j)
        for (uint32_t i = 0; i < d; ++i) {
            double p = (double)okv_half_to_float(x[j * d + i]) * (double)inv_of_channel[i];
            double r = rint(p); /* default rounding mode: ties to even */
            if (r > 127.0) r = 127.0;
            if (r < -127.0) r = -127.0;
            qbuf[j * d + i] = (int8_t)r;
        }
    if (q) memcpy(q, qbuf, n_el);

    /* Delta loop: along the channel axis, restarting on every token row; the first channel
     * of a row is kept as it is.  Differences wrap modulo 256. */
    uint8_t sbuf[MAX_ELEMS];
    for (uint32_t j = 0; j < N; ++j) {
        sbuf[j * d] = (uint8_t)qbuf[j * d];
        for (uint32_t i = 1; i < d; ++i)
            sbuf[j * d + i] = (uint8_t)((int)qbuf[j * d + i] - (int)qbuf[j * d + i - 1]);
    }
    if (sym) memcpy(sym, sbuf, n_el);

    /* Run-length step over the row-major symbol stream: one stored value per run; run lengths
     * are the gaps between set bits of a head bitmap (bit k set <=> symbol k starts a run). */
    uint32_t n_runs = 0;
    if (bitmap) memset(bitmap, 0, n_el / 8u);
    for (uint32_t k = 0; k < n_el; ++k) {
        if (k == 0 || sbuf[k] != sbuf[k - 1]) {
            if (bitmap) bitmap[k >> 3] |= (uint8_t)(1u << (k & 7u));
            if (values) values[n_runs] = sbuf[k];
            ++n_runs;
        }
    }
    if (n_runs_out) *n_runs_out = n_runs;
}

void okv_page_stages(const uint16_t *x, uint32_t N, uint32_t d, uint16_t *amax_bits_out,
                     float *s_out, float *inv_out, int8_t *q, uint8_t *sym, uint8_t *bitmap,
                     uint8_t *values, uint32_t *n_runs_out)
{
    page_stages(x, N, d, amax_bits_out, s_out, inv_out, NULL, q, sym, bitmap, values, n_runs_out);
}

void okv_page_stages_grouped(const uint16_t *x, uint32_t N, uint32_t d, uint16_t *group_amax,
                             int8_t *q, uint8_t *sym, uint8_t *bitmap, uint8_t *values,
                             uint32_t *n_runs_out)
{
    uint16_t scratch[MAX_ELEMS / OKV_GROUP_CHANNELS];
    page_stages(x, N, d, NULL, NULL, NULL, group_amax ? group_amax : scratch, q, sym, bitmap, values, n_runs_out);
}

uint32_t okv_compress_page(const uint16_t *x, uint32_t N, uint32_t d, int scheme, uint8_t *rec)
{
    uint32_t n_el = N * d;
    uint16_t amax_bits;
    float s, inv;
    int8_t q[MAX_ELEMS];
    uint8_t sym[MAX_ELEMS], bitmap[MAX_ELEMS / 8], values[MAX_ELEMS];
    uint16_t group_amax[MAX_ELEMS / OKV_GROUP_CHANNELS];
    uint32_t n_runs = 0, payload_len;
    int grouped = (scheme & OKV_GROUPED) != 0;
    int mode = scheme & ~OKV_GROUPED;
    uint32_t n_groups = grouped ? d / OKV_GROUP_CHANNELS : 0u;

    page_stages(x, N, d, &amax_bits, &s, &inv, grouped ? group_amax : NULL, q, sym, bitmap, values, &n_runs);
    if (amax_bits >= 0x7C00u) mode = OKV_RAW;
    /* Adaptive selection (the per-layer compression choice of Sec. 3.6.3, taken per page): keep the
     * run-length stage only where it makes the record smaller than the plain delta stream. */
    if (mode == OKV_AUTO) mode = (n_el / 8u + n_runs < n_el) ? OKV_INT8_DELTA_RLE : OKV_INT8_DELTA;

    uint8_t *pay = rec + HDR_BYTES;
    if (mode == OKV_RAW) {
        for (uint32_t k = 0; k < n_el; ++k) put16(pay + 2 * k, x[k]);
        payload_len = 2 * n_el;
        s = 0.0f; amax_bits = 0; n_runs = 0;
    } else {
        /* grouped scales: the groups' largest magnitudes come first in the payload */
        for (uint32_t g = 0; g < n_groups; ++g) put16(pay + 2 * g, group_amax[g]);
        pay += 2 * n_groups;
        if (grouped) mode |= OKV_GROUPED;
        if ((mode & 3) == OKV_INT8) {
            memcpy(pay, q, n_el);
            payload_len = n_el; n_runs = 0;
        } else if ((mode & 3) == OKV_INT8_DELTA) {
            memcpy(pay, sym, n_el);
            payload_len = n_el; n_runs = 0;
        } else {
            memcpy(pay, bitmap, n_el / 8u);
            memcpy(pay + n_el / 8u, values, n_runs);
            payload_len = n_el / 8u + n_runs;
        }
        payload_len += 2 * n_groups;
    }
    uint32_t sbits;
    memcpy(&sbits, &s, 4);
    put32(rec + 0, sbits);
    put16(rec + 4, payload_len);
    rec[6] = (uint8_t)mode;
    rec[7] = (uint8_t)FORMAT_VERSION;
    put16(rec + 8, n_runs);
    put16(rec + 10, amax_bits);
    put32(rec + 12, 0);
    return HDR_BYTES + payload_len;
}

/* ---------------------------------------------------------------------- */
/* Decompression pipeline (inverse mapping), one record                    */
/* ---------------------------------------------------------------------- */

int okv_decompress_record(const uint8_t *rec, uint32_t avail, uint32_t N, uint32_t d, uint16_t *out)
{
    uint32_t n_el = N * d;
    if (avail < HDR_BYTES) return OKV_ST_BAD_RECORD;
    uint32_t sbits = get32(rec + 0);
    uint32_t payload_len = get16(rec + 4);
    uint32_t mode = rec[6], version = rec[7], n_runs = get16(rec + 8);
    uint32_t grouped = mode & OKV_GROUPED;
    mode &= ~(uint32_t)OKV_GROUPED;
    if (version != FORMAT_VERSION || mode > 3u || (grouped && mode == OKV_RAW)) return OKV_ST_BAD_RECORD;
    if (HDR_BYTES + payload_len > avail) return OKV_ST_BAD_RECORD;
    const uint8_t *pay = rec + HDR_BYTES;

    if (mode == OKV_RAW) { /* early exit: uncompressed data bypasses the pipeline */
        if (payload_len != 2 * n_el) return OKV_ST_BAD_RECORD;
        for (uint32_t k = 0; k < n_el; ++k) out[k] = (uint16_t)get16(pay + 2 * k);
        return 0;
    }

    /* scale per channel: the header's, or the one derived from the group's stored magnitude */
    float s_of_channel[MAX_ELEMS];
    {
        float s;
        memcpy(&s, &sbits, 4);
        for (uint32_t i = 0; i < d; ++i) s_of_channel[i] = s;
    }
    if (grouped) {
        uint32_t n_groups = d / OKV_GROUP_CHANNELS;
        if (payload_len < 2 * n_groups) return OKV_ST_BAD_RECORD;
        for (uint32_t g = 0; g < n_groups; ++g) {
            uint32_t ga = get16(pay + 2 * g);
            if (ga >= 0x7C00u) return OKV_ST_BAD_RECORD; /* not a finite magnitude */
            float gs, ginv;
            group_scale((uint16_t)ga, &gs, &ginv);
            for (uint32_t c = 0; c < OKV_GROUP_CHANNELS; ++c) s_of_channel[g * OKV_GROUP_CHANNELS + c] = gs;
        }
        pay += 2 * n_groups;
        payload_len -= 2 * n_groups;
    }

    uint8_t sym[MAX_ELEMS];
    int8_t q[MAX_ELEMS];
    if (mode == OKV_INT8_DELTA_RLE) {
        /* expand runs: symbol k takes the value of the last run head at or before k */
        if (n_runs < 1u || n_runs > n_el || payload_len != n_el / 8u + n_runs) return OKV_ST_BAD_RECORD;
        const uint8_t *bitmap = pay, *values = pay + n_el / 8u;
        if (!(bitmap[0] & 1u)) return OKV_ST_BAD_RECORD;
        uint32_t run = 0;
        for (uint32_t k = 0; k < n_el; ++k) {
            if ((bitmap[k >> 3] >> (k & 7u)) & 1u) ++run;
            if (run > n_runs) return OKV_ST_BAD_RECORD;
            sym[k] = values[run - 1u];
        }
        if (run != n_runs) return OKV_ST_BAD_RECORD;
    } else {
        if (payload_len != n_el) return OKV_ST_BAD_RECORD;
        memcpy(sym, pay, n_el);
    }
    if (mode == OKV_INT8) {
        memcpy(q, sym, n_el);
    } else { /* undo the delta: running sum modulo 256 along each token row */
        for (uint32_t j = 0; j < N; ++j) {
            uint8_t acc = 0;
            for (uint32_t i = 0; i < d; ++i) {
                acc = (uint8_t)(acc + sym[j * d + i]);
                q[j * d + i] = (int8_t)acc;
            }
        }
    }
    /* dequantise: x = q * s in binary32, then round to binary16 (nearest even) */
    for (uint32_t j = 0; j < N; ++j)
        for (uint32_t i = 0; i < d; ++i) {
            volatile float p = (float)q[j * d + i] * s_of_channel[i];
            out[j * d + i] = okv_float_to_half(p);
        }
    return 0;
}

/* ---------------------------------------------------------------------- */
/* Pool level: append-only log of records in 64-byte granules + page table */
/* ---------------------------------------------------------------------- */

void okv_status_clear(okv_status *st)
{
    for (int c = 0; c < OKV_N_STATUS; ++c) { st->count[c] = 0; st->first[c] = 0xFFFFFFFFu; }
}

static void raise_status(okv_status *st, int code, uint32_t index)
{
    st->count[code] += 1u;
    if (index < st->first[code]) st->first[code] = index;
}

static uint64_t n_slots(const okv_config *cfg)
{
    return (uint64_t)cfg->n_layers * cfg->blocks_per_layer * 2u * cfg->n_kv_heads;
}

/* page-table entry: offset in granules | rec_len << 32 | mode << 48 | valid << 56 */
static uint64_t make_pte(uint64_t off64, uint32_t rec_len, uint32_t mode)
{
    return off64 | ((uint64_t)rec_len << 32) | ((uint64_t)mode << 48) | (1ull << 56);
}

int okv_compress(const okv_config *cfg, uint8_t *pool, uint64_t *pte, uint64_t *cursor64,
                 const uint16_t *src, uint32_t n_src_pages, const uint32_t *src_page,
                 const uint32_t *dst_slot, uint32_t n, int scheme, okv_status *st, okv_stats *stats)
{
    if (scheme < 0 || (scheme & ~OKV_GROUPED) > OKV_AUTO) return -1;
    uint64_t pool_gran = cfg->pool_bytes / GRANULE;
    uint8_t rec[HDR_BYTES + PAGE_BYTES + GRANULE];
    for (uint32_t i = 0; i < n; ++i) {
        if (src_page[i] >= n_src_pages || dst_slot[i] >= n_slots(cfg)) {
            raise_status(st, OKV_ST_BAD_INDEX, i); /* takes no space in the log */
            continue;
        }
        const uint16_t *x = src + (uint64_t)src_page[i] * PAGE_ELEMS;
        uint32_t rec_len = okv_compress_page(x, PAGE_N, PAGE_D, scheme, rec);
        uint32_t gran = (rec_len + GRANULE - 1u) / GRANULE;
        uint64_t off64 = *cursor64;
        *cursor64 += gran; /* the cursor advances whether or not the record fits */
        if (off64 + gran > pool_gran) {
            raise_status(st, OKV_ST_POOL_FULL, i);
            continue;
        }
        memset(rec + rec_len, 0, gran * GRANULE - rec_len);
        memcpy(pool + off64 * GRANULE, rec, gran * GRANULE);
        pte[dst_slot[i]] = make_pte(off64, rec_len, rec[6]);
        if (stats) {
            stats->pages_mode[rec[6] & 3u] += 1; /* grouped records count under their base mode */
            stats->granules += gran;
            stats->payload_bytes += rec_len - HDR_BYTES;
            stats->n_runs += get16(rec + 8);
            if (rec[6] == OKV_RAW && (scheme & ~OKV_GROUPED) != OKV_RAW) stats->nonfinite += 1;
        }
    }
    return 0;
}

/* Log compaction (pool lifecycle): the log only grows, and a slot that is written again leaves its
 * old record behind.  Rewrites the pool so that it holds exactly the records that page-table entries
 * point at, in slot order, each with its padding, from granule 0 on; every entry gets its new offset
 * and the cursor becomes the number of granules kept.  An entry whose record is not inside the pool
 * is reported (BAD_RECORD, index = slot) and cleared.  scratch: at least pool_bytes. */
int okv_compact(const okv_config *cfg, uint8_t *pool, uint64_t *pte, uint64_t *cursor64,
                uint8_t *scratch, okv_status *st)
{
    uint64_t kept = 0;
    for (uint64_t slot = 0; slot < n_slots(cfg); ++slot) {
        uint64_t e = pte[slot];
        if (!((e >> 56) & 1u)) continue;
        uint64_t off = (e & 0xFFFFFFFFull) * GRANULE;
        uint32_t rec_len = (uint32_t)((e >> 32) & 0xFFFFu), mode = (uint32_t)((e >> 48) & 0xFFu);
        uint64_t gran = (rec_len + GRANULE - 1u) / GRANULE;
        if (rec_len < HDR_BYTES || off + gran * GRANULE > cfg->pool_bytes) {
            raise_status(st, OKV_ST_BAD_RECORD, (uint32_t)slot);
            pte[slot] = 0;
            continue;
        }
        if (kept + gran > cfg->pool_bytes / GRANULE) { /* possible only if entries share a record */
            raise_status(st, OKV_ST_POOL_FULL, (uint32_t)slot);
            pte[slot] = 0;
            kept += gran; /* like the compressor's cursor: advances whether or not the record fits */
            continue;
        }
        memcpy(scratch + kept * GRANULE, pool + off, gran * GRANULE);
        pte[slot] = make_pte(kept, rec_len, mode);
        kept += gran;
    }
    uint64_t fits = kept < cfg->pool_bytes / GRANULE ? kept : cfg->pool_bytes / GRANULE;
    memcpy(pool, scratch, fits * GRANULE);
    *cursor64 = kept;
    return 0;
}

/* Slot free (pool lifecycle): the listed slots' page-table entries are cleared; their records stay in
 * the log as garbage until the next compaction.  freed[0] += entries that were valid, freed[1] += the
 * granules their records occupy.  A slot named twice counts once; a slot beyond the table is reported
 * (BAD_INDEX, index = position in the list). */
int okv_free_slots(const okv_config *cfg, uint64_t *pte, const uint32_t *slots, uint32_t n,
                   uint64_t *freed, okv_status *st)
{
    for (uint32_t i = 0; i < n; ++i) {
        if (slots[i] >= n_slots(cfg)) { raise_status(st, OKV_ST_BAD_INDEX, i); continue; }
        uint64_t e = pte[slots[i]];
        pte[slots[i]] = 0;
        if (!((e >> 56) & 1u)) continue;
        uint32_t rec_len = (uint32_t)((e >> 32) & 0xFFFFu);
        freed[0] += 1;
        freed[1] += (rec_len + GRANULE - 1u) / GRANULE;
    }
    return 0;
}

/* ---------------------------------------------------------------------- */
/* Compression selection per layer (Sec. 3.6.3):                            */
/*   C*(l,t) = argmax_{C in CC} J,  J = w_r R_c(C,l) + w_q Q(C,l) - w_c L_comp(C),  s.t. Q >= Q_min */
/* ---------------------------------------------------------------------- */

/* The candidate set CC, in the order that breaks ties (simpler first). */
static const int probe_schemes[OKV_N_CANDIDATES] = {
    OKV_INT8, OKV_INT8_DELTA, OKV_INT8_DELTA_RLE, OKV_AUTO,
    OKV_INT8 | OKV_GROUPED, OKV_INT8_DELTA | OKV_GROUPED, OKV_INT8_DELTA_RLE | OKV_GROUPED, OKV_AUTO | OKV_GROUPED};

/* What a sample of a layer's pages would cost and lose under every candidate: each page is really
 * compressed with each scheme (size) and the two quantisers' records are really decompressed (error).
 * Pages holding Inf/NaN are stored raw whatever the scheme and are only counted. */
int okv_probe_pages(const uint16_t *src, uint32_t n_src_pages, const uint32_t *src_page, uint32_t n,
                    okv_probe *out)
{
    uint8_t rec[HDR_BYTES + PAGE_BYTES + GRANULE];
    uint16_t back[PAGE_ELEMS];
    for (uint32_t i = 0; i < n; ++i) {
        if (src_page[i] >= n_src_pages) { out->bad_index += 1; continue; }
        const uint16_t *x = src + (uint64_t)src_page[i] * PAGE_ELEMS;
        uint32_t len = okv_compress_page(x, PAGE_N, PAGE_D, OKV_INT8, rec);
        if (rec[6] == OKV_RAW) { out->nonfinite += 1; continue; }
        out->pages += 1;
        for (int c = 0; c < OKV_N_CANDIDATES; ++c) {
            len = okv_compress_page(x, PAGE_N, PAGE_D, probe_schemes[c], rec);
            out->granules[c] += (len + GRANULE - 1u) / GRANULE;
        }
        for (int g = 0; g < 2; ++g) {   /* the lossy step is the quantiser: one scale per page, or per group */
            len = okv_compress_page(x, PAGE_N, PAGE_D, g ? (OKV_INT8 | OKV_GROUPED) : OKV_INT8, rec);
            okv_decompress_record(rec, len, PAGE_N, PAGE_D, back);
            for (uint32_t k = 0; k < PAGE_ELEMS; ++k) {
                double e = (double)okv_half_to_float(x[k]) - (double)okv_half_to_float(back[k]);
                out->sq_err[g] += e * e;
            }
        }
        for (uint32_t k = 0; k < PAGE_ELEMS; ++k) {
            double v = (double)okv_half_to_float(x[k]);
            out->sq_sum += v * v;
        }
    }
    return 0;
}

/* Quality Q of a quantiser on the sample: signal-to-noise ratio in decibels, capped at 200 (also
 * when there is no error at all). */
double okv_probe_quality(const okv_probe *p, int grouped)
{
    double err = p->sq_err[grouped ? 1 : 0];
    if (!(err > 0.0) || !(p->sq_sum > 0.0)) return 200.0;
    double q = 10.0 * log10(p->sq_sum / err);
    return q > 200.0 ? 200.0 : q;
}

/* The selection itself.  R_c = uncompressed bytes / stored bytes of the sample.  Among the candidates
 * with Q >= q_min the largest J wins, the earlier candidate on a tie; if no candidate reaches q_min, the
 * one with the best quality does (earlier on a tie).  objective (optional): J of every candidate.
 * Returns the scheme, or -1 if the sample is empty. */
int okv_select_scheme(const okv_probe *p, const okv_policy *pol, double *objective)
{
    if (p->pages == 0) return -1;
    int best = -1, best_q = 0;
    double best_j = 0.0;
    for (int c = 0; c < OKV_N_CANDIDATES; ++c) {
        double ratio = (double)p->pages * (double)(PAGE_BYTES / GRANULE) / (double)p->granules[c];
        double q = okv_probe_quality(p, c >= 4);
        double j = pol->w_r * ratio + pol->w_q * q - pol->w_c * pol->cost[c];
        if (objective) objective[c] = j;
        if (q >= pol->q_min && (best < 0 || j > best_j)) { best = c; best_j = j; }
        if (q > okv_probe_quality(p, best_q >= 4)) best_q = c;
    }
    return probe_schemes[best >= 0 ? best : best_q];
}

/* Address translation: (seq, layer, K|V, head, token position) -> page slot -> record.
 * Layer-major regions; inside a layer the 2*H pages of one physical block are adjacent. */
static int walk(const okv_config *cfg, const uint64_t *pte, const int32_t *block_table,
                uint32_t seq, uint32_t layer, uint32_t kv, uint32_t head, uint32_t block,
                uint64_t *byte_off, uint32_t *rec_len, uint32_t *mode)
{
    if (seq >= cfg->max_seqs || block >= cfg->max_blocks_per_seq || layer >= cfg->n_layers ||
        kv > 1u || head >= cfg->n_kv_heads)
        return OKV_ST_UNMAPPED;
    int32_t p = block_table[(uint64_t)seq * cfg->max_blocks_per_seq + block];
    if (p < 0 || (uint32_t)p >= cfg->blocks_per_layer) return OKV_ST_UNMAPPED;
    uint64_t slot = (((uint64_t)layer * cfg->blocks_per_layer + (uint32_t)p) * 2u + kv) * cfg->n_kv_heads + head;
    uint64_t e = pte[slot];
    if (!((e >> 56) & 1u)) return OKV_ST_BAD_PTE;
    *byte_off = (e & 0xFFFFFFFFull) * GRANULE;
    *rec_len = (uint32_t)((e >> 32) & 0xFFFFu);
    *mode = (uint32_t)((e >> 48) & 0xFFu);
    if (*rec_len < HDR_BYTES || *byte_off + *rec_len > cfg->pool_bytes) return OKV_ST_BAD_RECORD;
    return 0;
}

int okv_translate(const okv_config *cfg, const uint64_t *pte, const int32_t *block_table,
                  const okv_vaddr *va, okv_paddr *pa, uint32_t n, okv_status *st)
{
    for (uint32_t i = 0; i < n; ++i) {
        uint64_t off = 0; uint32_t len = 0, mode = 0;
        int rc = walk(cfg, pte, block_table, va[i].seq, va[i].layer, va[i].kv, va[i].head,
                      va[i].pos >> 4, &off, &len, &mode);
        if (rc) { raise_status(st, rc, i); off = 0; len = 0; mode = 0; }
        pa[i].byte_off = off; pa[i].rec_len = len; pa[i].mode = (uint8_t)mode;
        pa[i].status = (uint8_t)rc; pa[i].rsvd = 0;
    }
    return 0;
}

/* ---------------------------------------------------------------------- */
/* Demand fetch + prefetch loop: translate, fetch, decompress, place       */
/* ---------------------------------------------------------------------- */

/* Fetch one page through the translation unit and write it at dst. */
static void fetch_page(const okv_config *cfg, const uint8_t *pool, const uint64_t *pte,
                       const int32_t *block_table, uint32_t seq, uint32_t layer, uint32_t kv,
                       uint32_t head, uint32_t block, uint16_t *dst, uint32_t index,
                       okv_status *st, okv_stats *stats)
{
    uint64_t off = 0; uint32_t len = 0, mode = 0;
    int rc = walk(cfg, pte, block_table, seq, layer, kv, head, block, &off, &len, &mode);
    if (rc) { raise_status(st, rc, index); return; }
    uint16_t page[PAGE_ELEMS];
    const uint8_t *rec = pool + off;
    if (rec[6] != mode || HDR_BYTES + get16(rec + 4) != len) { raise_status(st, OKV_ST_BAD_RECORD, index); return; }
    rc = okv_decompress_record(rec, len, PAGE_N, PAGE_D, page);
    if (rc) { raise_status(st, rc, index); return; } /* destination left untouched */
    memcpy(dst, page, PAGE_BYTES);
    if (stats) stats->pages_decoded += 1;
}

int okv_decompress_gather(const okv_config *cfg, const uint8_t *pool, const uint64_t *pte,
                          uint64_t *l2_tag, uint32_t epoch, uint32_t layer,
                          const int32_t *block_table, const uint32_t *seq_lens,
                          const uint64_t *dst_tok_off, uint32_t B, const okv_prefetch *pf,
                          uint32_t n_pf, uint16_t *dst_demand, uint64_t dst_cap_tokens,
                          uint16_t *dst_l2, okv_status *st, okv_stats *stats)
{
    uint32_t H = cfg->n_kv_heads;
    if (layer >= cfg->n_layers || B > cfg->max_seqs) return -1;
    uint32_t index = 0; /* running page index: demand pages first, then prefetch pages */

    /* Demand (fallback/synchronous) path: every block below the sequence length, K and V, all
     * heads.  Sequence b owns Tpad_b = 16*ceil(len_b/16) token rows starting at dst_tok_off[b];
     * inside it the layout is [K|V][head][token][channel]. */
    for (uint32_t b = 0; b < B; ++b) {
        uint32_t nblk = (uint32_t)(((uint64_t)seq_lens[b] + PAGE_N - 1u) / PAGE_N);
        /* a length the block table cannot describe: the sequence is reported once, at the index its
         * first page would have had, and takes no part (no pages, no place in the numbering) */
        if (nblk > cfg->max_blocks_per_seq) { raise_status(st, OKV_ST_UNMAPPED, index); continue; }
        uint64_t tpad = (uint64_t)nblk * PAGE_N;
        for (uint32_t n = 0; n < nblk; ++n)
            for (uint32_t kv = 0; kv < 2u; ++kv)
                for (uint32_t h = 0; h < H; ++h, ++index) {
                    if (dst_tok_off[b] + tpad > dst_cap_tokens) { raise_status(st, OKV_ST_BAD_DST, index); continue; }
                    uint64_t el = dst_tok_off[b] * 2u * H * PAGE_D +
                                  (((uint64_t)kv * H + h) * tpad + (uint64_t)PAGE_N * n) * PAGE_D;
                    fetch_page(cfg, pool, pte, block_table, b, layer, kv, h, n, dst_demand + el, index, st, stats);
                }
    }

    /* Prefetch loop: for each predicted block, translate, skip it if the prefetch buffer slot
     * already holds that block, otherwise fetch it into the slot and retag the slot (a stale
     * slot is simply overwritten). */
    for (uint32_t e = 0; e < n_pf; ++e) {
        uint32_t seq = pf[e].seq, blk = pf[e].block, slot = pf[e].l2_slot;
        int mapped = seq < cfg->max_seqs && slot < L2_SLOTS && blk < cfg->max_blocks_per_seq;
        if (mapped) {
            int32_t p = block_table[(uint64_t)seq * cfg->max_blocks_per_seq + blk];
            mapped = p >= 0 && (uint32_t)p < cfg->blocks_per_layer;
        }
        if (!mapped) {
            for (uint32_t r = 0; r < 2u * H; ++r, ++index) raise_status(st, OKV_ST_UNMAPPED, index);
            continue;
        }
        uint32_t tag = layer * (1u << 20) + blk + 1u;
        uint64_t *t = &l2_tag[(uint64_t)seq * L2_SLOTS + slot];
        if ((uint32_t)(*t & 0xFFFFFFFFull) == tag) {
            if (stats) stats->pf_skipped += 1;
            index += 2u * H;
            continue;
        }
        *t = ((uint64_t)epoch << 32) | tag;
        if (stats) stats->pf_issued += 1;
        for (uint32_t kv = 0; kv < 2u; ++kv)
            for (uint32_t h = 0; h < H; ++h, ++index) {
                uint64_t el = (((((uint64_t)seq * L2_SLOTS + slot) * 2u + kv) * H + h) * PAGE_N) * PAGE_D;
                fetch_page(cfg, pool, pte, block_table, seq, layer, kv, h, blk, dst_l2 + el, index, st, stats);
            }
    }
    return 0;
}

/* ---------------------------------------------------------------------- */
/* Per-layer computation that consumes the fetched pages (Sec. 3.4.4, the   */
/* T_layer stage of the multi-layer prefetch pipeline): decode-step         */
/* attention of one query token per sequence, in binary64.                  */
/* ---------------------------------------------------------------------- */

/* out[c] = sum_t softmax_t(q . k_t / sqrt(d)) * v_t[c] over the rows marked valid.
 * k, v: n_tok rows of PAGE_D binary16 values.  No valid row: out = 0. */
static void attend_rows(const uint16_t *q, const uint16_t *const *k_rows, const uint16_t *const *v_rows,
                        uint32_t n_tok, double *out)
{
    double best = -INFINITY;
    for (uint32_t c = 0; c < PAGE_D; ++c) out[c] = 0.0;
    if (n_tok == 0) return;
    double *score = (double *)malloc(n_tok * sizeof(double));
    for (uint32_t t = 0; t < n_tok; ++t) {
        double dot = 0.0;
        for (uint32_t c = 0; c < PAGE_D; ++c)
            dot += (double)okv_half_to_float(q[c]) * (double)okv_half_to_float(k_rows[t][c]);
        score[t] = dot / sqrt((double)PAGE_D);
        if (score[t] > best) best = score[t];
    }
    double denom = 0.0;
    for (uint32_t t = 0; t < n_tok; ++t) {
        double p = exp(score[t] - best);
        denom += p;
        for (uint32_t c = 0; c < PAGE_D; ++c) out[c] += p * (double)okv_half_to_float(v_rows[t][c]);
    }
    for (uint32_t c = 0; c < PAGE_D; ++c) out[c] /= denom;
    free(score);
}

int okv_attend_dense(const uint16_t *kv, const uint32_t *seq_lens, const uint64_t *tok_off, uint32_t B,
                     uint32_t H, const uint16_t *q, uint32_t Hq, double *out)
{
    if (H == 0 || Hq == 0 || Hq % H) return -1;
    uint32_t G = Hq / H; /* query heads g*G .. g*G + G-1 read KV head g */
    for (uint32_t b = 0; b < B; ++b) {
        uint32_t len = seq_lens[b];
        uint64_t tpad = (uint64_t)((len + PAGE_N - 1u) / PAGE_N) * PAGE_N;
        const uint16_t **kr = (const uint16_t **)malloc((len + 1u) * sizeof(*kr));
        const uint16_t **vr = (const uint16_t **)malloc((len + 1u) * sizeof(*vr));
        for (uint32_t hq = 0; hq < Hq; ++hq) {
            uint32_t h = hq / G;
            /* workspace layout of the demand path: [K|V][head][token][channel] per sequence */
            const uint16_t *base = kv + tok_off[b] * 2u * H * PAGE_D;
            for (uint32_t t = 0; t < len; ++t) {
                kr[t] = base + (((uint64_t)0 * H + h) * tpad + t) * PAGE_D;
                vr[t] = base + (((uint64_t)1 * H + h) * tpad + t) * PAGE_D;
            }
            attend_rows(q + ((uint64_t)b * Hq + hq) * PAGE_D, kr, vr, len, out + ((uint64_t)b * Hq + hq) * PAGE_D);
        }
        free(kr); free(vr);
    }
    return 0;
}

int okv_attend(const okv_config *cfg, const uint8_t *pool, const uint64_t *pte, uint32_t layer,
               const int32_t *block_table, const uint32_t *seq_lens, uint32_t B, const uint16_t *q,
               uint32_t Hq, double *out, okv_status *st, okv_stats *stats)
{
    uint32_t H = cfg->n_kv_heads;
    if (layer >= cfg->n_layers || B > cfg->max_seqs || Hq == 0 || Hq % H) return -1;
    uint32_t G = Hq / H;
    uint32_t index0 = 0; /* page index of the sequence's first page, numbered as in the demand fetch */
    for (uint32_t b = 0; b < B; ++b) {
        uint32_t len = seq_lens[b];
        uint32_t nblk = (uint32_t)(((uint64_t)len + PAGE_N - 1u) / PAGE_N);
        if (nblk > cfg->max_blocks_per_seq) { /* as in the demand fetch: reported once, left out, zero output */
            raise_status(st, OKV_ST_UNMAPPED, index0);
            for (uint64_t i = 0; i < (uint64_t)Hq * PAGE_D; ++i) out[(uint64_t)b * Hq * PAGE_D + i] = 0.0;
            continue;
        }
        uint16_t *kpage = (uint16_t *)malloc((size_t)(nblk + 1u) * PAGE_BYTES);
        uint16_t *vpage = (uint16_t *)malloc((size_t)(nblk + 1u) * PAGE_BYTES);
        const uint16_t **kr = (const uint16_t **)malloc((len + 1u) * sizeof(*kr));
        const uint16_t **vr = (const uint16_t **)malloc((len + 1u) * sizeof(*vr));
        for (uint32_t h = 0; h < H; ++h) {
            /* fetch the head's pages through the translation unit; a block whose K or V page cannot
             * be delivered is reported and takes no part in the attention */
            uint32_t n_tok = 0;
            for (uint32_t n = 0; n < nblk; ++n) {
                int ok = 1;
                for (uint32_t kv = 0; kv < 2u; ++kv) {
                    uint32_t index = index0 + (n * 2u + kv) * H + h;
                    uint64_t off = 0; uint32_t rlen = 0, mode = 0;
                    uint16_t *dst = (kv ? vpage : kpage) + (size_t)n * PAGE_ELEMS;
                    int rc = walk(cfg, pte, block_table, b, layer, kv, h, n, &off, &rlen, &mode);
                    if (!rc) {
                        const uint8_t *rec = pool + off;
                        if (rec[6] != mode || HDR_BYTES + get16(rec + 4) != rlen) rc = OKV_ST_BAD_RECORD;
                        else rc = okv_decompress_record(rec, rlen, PAGE_N, PAGE_D, dst);
                    }
                    if (rc) { raise_status(st, rc, index); ok = 0; }
                    else if (stats) stats->pages_decoded += 1;
                }
                if (!ok) continue;
                for (uint32_t t = 0; t < PAGE_N && n * PAGE_N + t < len; ++t, ++n_tok) {
                    kr[n_tok] = kpage + (size_t)n * PAGE_ELEMS + t * PAGE_D;
                    vr[n_tok] = vpage + (size_t)n * PAGE_ELEMS + t * PAGE_D;
                }
            }
            for (uint32_t g = 0; g < G; ++g) {
                uint32_t hq = h * G + g;
                attend_rows(q + ((uint64_t)b * Hq + hq) * PAGE_D, kr, vr, n_tok, out + ((uint64_t)b * Hq + hq) * PAGE_D);
            }
        }
        free(kpage); free(vpage); free(kr); free(vr);
        index0 += nblk * 2u * H;
    }
    return 0;
}

/* ---------------------------------------------------------------------- */
/* Managed prefetch buffer: double buffering (Sec. 3.3.1, tier L2), lazy    */
/* invalidation / fallback fetch / per-request adaptive depth (Sec. 3.4.3), */
/* depth chosen by the UCB rule of Sec. 3.6.3, and the counters behind the  */
/* paper's prefetch-statistics table.                                       */
/* ---------------------------------------------------------------------- */

/* ln T kept to 20 fractional bits, so that the depth decision does not hang on the last
 * bits of a logarithm routine. */
static double ln_steps(uint32_t steps)
{
    return rint(log((double)steps) * 1048576.0) / 1048576.0;
}

/* mu_k + beta * sqrt(2 ln T / N_k); mu_k = mean reward scaled to at most 1 (8 = the reward of a
 * fill whose four slots were all used).  One rounding per operation, binary64. */
double okv_pf_score(int32_t reward, uint32_t plays, uint32_t steps, double beta)
{
    double mean = (double)reward / (8.0 * (double)plays);
    double ratio = (2.0 * ln_steps(steps)) / (double)plays;
    double bonus = beta * sqrt(ratio);
    return mean + bonus;
}

uint32_t okv_pf_choose_depth(const okv_pf_seq *s, double beta)
{
    for (uint32_t k = 1; k <= OKV_PF_SLOTS; ++k)
        if (s->plays[k - 1] == 0) return k; /* every depth is tried once first */
    uint32_t best = 1;
    double best_score = okv_pf_score(s->reward[0], s->plays[0], s->steps, beta);
    for (uint32_t k = 2; k <= OKV_PF_SLOTS; ++k) {
        double sc = okv_pf_score(s->reward[k - 1], s->plays[k - 1], s->steps, beta);
        if (sc > best_score) { best_score = sc; best = k; } /* ties: the smaller depth */
    }
    return best;
}

int okv_prefetch_step(const okv_config *cfg, const uint8_t *pool, const uint64_t *pte, uint32_t layer,
                      uint32_t back, const int32_t *block_table, const int32_t *access,
                      const int32_t *cand, uint32_t B, double beta, okv_pf_seq *state,
                      okv_pf_counters *cnt, uint16_t *l2, uint16_t *miss_dst, int32_t *where,
                      okv_status *st, okv_stats *stats)
{
    uint32_t H = cfg->n_kv_heads, twoH = 2u * H;
    if (layer >= cfg->n_layers || B > cfg->max_seqs || back > 1u) return -1;
    uint32_t front = back ^ 1u;
    uint64_t set_elems = (uint64_t)twoH * PAGE_ELEMS; /* the 2*H pages of one block */

    for (uint32_t b = 0; b < B; ++b) {
        okv_pf_seq *s = &state[b];

        /* 1. This step's reads.  Only the front bank (filled during the previous step) may be
         *    read; a block found there is served from the buffer, any other block takes the
         *    fallback path: a synchronous fetch from the pool. */
        for (uint32_t a = 0; a < OKV_PF_ACCESSES; ++a) {
            int32_t blk = access[b * OKV_PF_ACCESSES + a];
            int32_t *w = &where[b * OKV_PF_ACCESSES + a];
            *w = -2;
            if (blk < 0) continue;
            uint32_t index = (b * OKV_PF_ACCESSES + a) * twoH;
            if ((uint32_t)blk >= cfg->max_blocks_per_seq) {
                for (uint32_t r = 0; r < twoH; ++r) raise_status(st, OKV_ST_UNMAPPED, index + r);
                continue;
            }
            uint32_t tag = layer * (1u << 20) + (uint32_t)blk + 1u;
            cnt->accesses += 1;
            int hit = -1, late = 0;
            for (uint32_t j = 0; j < OKV_PF_SLOTS; ++j) {
                if (hit < 0 && s->tag[front][j] == tag) hit = (int)j;
                if (s->tag[back][j] == tag) late = 1;
            }
            if (hit >= 0) {
                s->used[front][hit] = 1;
                cnt->hits += 1;
                *w = (int32_t)(front * OKV_PF_SLOTS + (uint32_t)hit);
                continue;
            }
            cnt->misses += 1;
            if (late) cnt->late += 1; /* requested earlier, but its bank cannot be read in this step */
            *w = -1;
            uint16_t *dst = miss_dst + (uint64_t)(b * OKV_PF_ACCESSES + a) * set_elems;
            for (uint32_t kv = 0; kv < 2u; ++kv)
                for (uint32_t h = 0; h < H; ++h) {
                    uint64_t before = stats ? stats->pages_decoded : 0;
                    fetch_page(cfg, pool, pte, block_table, b, layer, kv, h, (uint32_t)blk,
                               dst + (uint64_t)(kv * H + h) * PAGE_ELEMS, index + kv * H + h, st, stats);
                    if (stats) cnt->pages += stats->pages_decoded - before;
                }
        }

        /* 2. The back bank is about to be refilled: score the depth it was filled with two steps
         *    ago (it was the readable bank during the previous step, so its used marks are final).
         *    reward = 2 per requested block that was read, -1 per requested block that was not. */
        uint32_t d = s->depth[back];
        if (d > 0) {
            int32_t valid = 0, useful = 0;
            for (uint32_t j = 0; j < d; ++j)
                if (s->tag[back][j] != 0) { valid += 1; useful += s->used[back][j] ? 1 : 0; }
            s->reward[d - 1] += 3 * useful - valid;
            s->plays[d - 1] += 1;
            s->steps += 1;
        }

        /* 3. Depth for this fill. */
        uint32_t k = okv_pf_choose_depth(s, beta);

        /* 4. Refill: the first k predicted blocks go to slots 0..k-1 of the back bank.  A slot that
         *    already holds the predicted block is kept (no transfer); any other content is simply
         *    overwritten.  Slots from k on are left as they are. */
        s->fill = 0;
        for (uint32_t j = 0; j < k; ++j) {
            int32_t c = cand[b * OKV_PF_SLOTS + j];
            if (c < 0 || (uint32_t)c >= cfg->max_blocks_per_seq) continue; /* no prediction */
            uint32_t index = ((B + b) * OKV_PF_SLOTS + j) * twoH;
            int32_t p = block_table[(uint64_t)b * cfg->max_blocks_per_seq + (uint32_t)c];
            if (p < 0 || (uint32_t)p >= cfg->blocks_per_layer) {
                for (uint32_t r = 0; r < twoH; ++r) raise_status(st, OKV_ST_UNMAPPED, index + r);
                continue;
            }
            uint32_t tag = layer * (1u << 20) + (uint32_t)c + 1u;
            if (s->tag[back][j] == tag) {
                s->used[back][j] = 0;
                cnt->kept += 1;
                continue;
            }
            if (s->tag[back][j] != 0) {
                cnt->evicted += 1;
                cnt->evicted_used += s->used[back][j] ? 1u : 0u;
            }
            s->tag[back][j] = tag;
            s->used[back][j] = 0;
            s->fill |= (uint8_t)(1u << j);
            cnt->fetched += 1;
            uint16_t *dst = l2 + (((uint64_t)back * cfg->max_seqs + b) * OKV_PF_SLOTS + j) * set_elems;
            for (uint32_t kv = 0; kv < 2u; ++kv)
                for (uint32_t h = 0; h < H; ++h) {
                    uint64_t before = stats ? stats->pages_decoded : 0;
                    fetch_page(cfg, pool, pte, block_table, b, layer, kv, h, (uint32_t)c,
                               dst + (uint64_t)(kv * H + h) * PAGE_ELEMS, index + kv * H + h, st, stats);
                    if (stats) cnt->pages += stats->pages_decoded - before;
                }
        }
        s->depth[back] = (uint8_t)k;
    }
    return 0;
}
