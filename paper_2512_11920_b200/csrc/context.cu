// Host side of the speckv C ABI: context, argument checks, launches.
#include <cstddef>
#include <cstring>
#include <new>

#include "speckv_dev.cuh"


using namespace speckv;

struct speckv_ctx {
    speckv_config cfg;
    int device, n_sm;
    unsigned long long n_slots;
    uint8_t *pool;
    unsigned long long *pte, *l2_tag;
    Ctl *ctl;
    ScanScratch *scan;
    uint32_t scan_tiles;   // capacity of scan->tile
    uint32_t epoch;        // gather calls so far (prefetch residency filter)
    uint32_t spin_limit;            // look-back polls per window (speckv_set_wait_limits)
    unsigned long long wait_ns;     // time limit of barrier waits
    uint32_t missing_tiles;         // fault injection for the next speckv_compress (speckv_inject_missing_tiles)
    // Gather launches still possibly in flight since the last ordinary (fully ordered) launch: their
    // destination ranges, and whether any of them skipped the wait for its predecessor.
    struct Span { uintptr_t lo, hi; };
    static constexpr int kMaxSpans = 256;
    Span span[kMaxSpans];
    int n_span;
    bool chain_live, chain_skipped, chain_enabled;
    cudaStream_t chain_stream;
    // speckv_pipeline_layers: the fetch stream and one pair of events per ring slot (made at the first call)
    static constexpr uint32_t kMaxRing = 8;
    cudaStream_t fetch_stream;
    cudaEvent_t ev_start, ev_fetched[kMaxRing], ev_consumed[kMaxRing];
    bool pipeline_ready;
};

// How the next gather may be launched (GatherArgs::chain), and the bookkeeping for the one after.
static uint32_t plan_gather_chain(speckv_ctx *c, cudaStream_t st, speckv_ctx::Span dst, speckv_ctx::Span l2, bool has_pf)
{
    uint32_t mode = 0;
    if (c->chain_enabled && c->chain_live && st == c->chain_stream && c->n_span + 2 <= speckv_ctx::kMaxSpans) {
        bool disjoint = true;
        for (int i = 0; i < c->n_span; ++i)
            if (dst.lo < c->span[i].hi && c->span[i].lo < dst.hi) disjoint = false;
        if (!has_pf && disjoint) mode = 2;          // nothing shared with any gather in flight
        else if (!c->chain_skipped) mode = 1;       // every gather in flight is ordered before the previous one
    }
    if (mode == 0) { c->n_span = 0; c->chain_skipped = false; }
    if (mode == 2) c->chain_skipped = true;
    if (dst.hi > dst.lo) c->span[c->n_span++] = dst;
    if (l2.hi > l2.lo) c->span[c->n_span++] = l2;
    c->chain_live = true;
    c->chain_stream = st;
    return mode;
}

static_assert(sizeof(speckv_vaddr) == 16 && sizeof(speckv_paddr) == 16 && sizeof(speckv_prefetch) == 12, "ABI layout");
static_assert(sizeof(speckv_pf_seq) == 80 && sizeof(speckv_pf_counters) == 80, "ABI layout");
static_assert(sizeof(speckv_stats) == 11 * 8 && sizeof(speckv_status) == 64, "ABI layout");

static size_t scan_bytes(uint32_t tiles) { return sizeof(ScanScratch) + (size_t)tiles * sizeof(unsigned long long); }

static int clear_ctl(speckv_ctx *c, bool cursor_too, cudaStream_t st)
{
    // counters to 0, "first index" words to 0xFFFFFFFF; two memsets, no host staging buffer
    size_t off = cursor_too ? 0 : offsetof(Ctl, status_count);
    if (cudaMemsetAsync((char *)c->ctl + off, 0, sizeof(Ctl) - off, st) != cudaSuccess) return SPECKV_E_CUDA;
    if (cudaMemsetAsync((char *)c->ctl + offsetof(Ctl, status_first), 0xFF, sizeof(unsigned int) * SPECKV_N_STATUS, st) != cudaSuccess)
        return SPECKV_E_CUDA;
    return 0;
}

extern "C" {

const char *speckv_version(void) { return "speckv 0.1 (sm_100a)"; }

int speckv_create(speckv_ctx **out, const speckv_config *cfg)
{
    if (!out || !cfg) return SPECKV_E_ARG;
    *out = nullptr;
    if (!cfg->n_layers || !cfg->n_kv_heads || !cfg->blocks_per_layer || !cfg->max_blocks_per_seq || !cfg->max_seqs ||
        cfg->n_kv_heads > 255 || cfg->n_layers > 4095 || cfg->blocks_per_layer >= (1u << 20) ||
        cfg->max_blocks_per_seq >= (1u << 20) || cfg->max_seqs > gather_max_seqs() || cfg->pool_bytes == 0 ||
        (unsigned long long)cfg->max_seqs * cfg->max_blocks_per_seq * 2ull * cfg->n_kv_heads > 0x7FFFFFFFull ||   // page indices are 32-bit
        cfg->pool_bytes % kGranule || cfg->pool_bytes / kGranule > 0xFFFFFFFFull)
        return SPECKV_E_ARG;
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return SPECKV_E_CUDA;
    if (prop.major != 10) return SPECKV_E_DEVICE;
    speckv_ctx *c = new (std::nothrow) speckv_ctx();
    if (!c) return SPECKV_E_CUDA;
    c->cfg = *cfg;
    c->device = dev;
    c->n_sm = prop.multiProcessorCount;
    c->n_slots = (unsigned long long)cfg->n_layers * cfg->blocks_per_layer * 2ull * cfg->n_kv_heads;
    c->epoch = 0;
    c->n_span = 0; c->chain_live = false; c->chain_skipped = false; c->chain_stream = nullptr; c->chain_enabled = true;
    c->pipeline_ready = false;
    c->spin_limit = kDefaultSpinLimit;
    c->wait_ns = kDefaultWaitNs;
    c->missing_tiles = 0;
    unsigned long long tiles = (c->n_slots + compress_min_tile_pages() - 1) / compress_min_tile_pages() + 1;
    c->scan_tiles = (uint32_t)(tiles > 0xFFFFFFFFull ? 0xFFFFFFFFull : tiles);
    bool ok = cudaMalloc(&c->pool, cfg->pool_bytes) == cudaSuccess &&
              cudaMalloc(&c->pte, c->n_slots * 8) == cudaSuccess &&
              cudaMalloc(&c->l2_tag, (size_t)cfg->max_seqs * SPECKV_L2_SLOTS * 8) == cudaSuccess &&
              cudaMalloc(&c->ctl, sizeof(Ctl)) == cudaSuccess && cudaMalloc(&c->scan, scan_bytes(c->scan_tiles)) == cudaSuccess;
    ok = ok && cudaMemset(c->pool, 0, cfg->pool_bytes) == cudaSuccess && speckv_reset(c, nullptr) == 0 &&
         cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        speckv_destroy(c);
        return SPECKV_E_CUDA;
    }
    *out = c;
    return 0;
}

int speckv_destroy(speckv_ctx *c)
{
    if (!c) return SPECKV_E_ARG;
    if (c->pipeline_ready) {
        cudaStreamDestroy(c->fetch_stream);
        cudaEventDestroy(c->ev_start);
        for (uint32_t i = 0; i < speckv_ctx::kMaxRing; ++i) { cudaEventDestroy(c->ev_fetched[i]); cudaEventDestroy(c->ev_consumed[i]); }
    }
    cudaFree(c->pool);
    cudaFree(c->pte);
    cudaFree(c->l2_tag);
    cudaFree(c->ctl);
    cudaFree(c->scan);
    delete c;
    return 0;
}

int speckv_reset(speckv_ctx *c, void *stream)
{
    if (!c) return SPECKV_E_ARG;
    c->chain_live = false;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(c->pte, 0, c->n_slots * 8, st) != cudaSuccess ||
        cudaMemsetAsync(c->l2_tag, 0, (size_t)c->cfg.max_seqs * SPECKV_L2_SLOTS * 8, st) != cudaSuccess)
        return SPECKV_E_CUDA;
    c->epoch = 0;
    return clear_ctl(c, true, st);
}

int speckv_set_wait_limits(speckv_ctx *c, uint32_t lookback_polls, uint64_t wait_ns)
{
    if (!c) return SPECKV_E_ARG;
    c->spin_limit = lookback_polls ? lookback_polls : kDefaultSpinLimit;
    c->wait_ns = wait_ns ? wait_ns : kDefaultWaitNs;
    return 0;
}

int speckv_set_gather_chaining(speckv_ctx *c, int enabled)
{
    if (!c) return SPECKV_E_ARG;
    c->chain_enabled = enabled != 0;
    c->chain_live = false;
    return 0;
}

int speckv_inject_missing_tiles(speckv_ctx *c, uint32_t n_tiles)
{
    if (!c) return SPECKV_E_ARG;
    c->missing_tiles = n_tiles;
    return 0;
}

int speckv_clear_status(speckv_ctx *c, void *stream)
{
    if (!c) return SPECKV_E_ARG;
    c->chain_live = false;
    return clear_ctl(c, false, (cudaStream_t)stream);
}

int speckv_compress(speckv_ctx *c, const void *src, uint32_t n_src_pages, const uint32_t *src_page,
                    const uint32_t *dst_slot, uint32_t n, int scheme, void *stream)
{
    if (!c || scheme < 0 || (scheme & ~SPECKV_GROUPED) > SPECKV_AUTO) return SPECKV_E_ARG;
    if (n == 0) return 0;
    c->chain_live = false;
    if (!src || !src_page || !dst_slot || ((uintptr_t)src & 15u) || (((uintptr_t)src_page | (uintptr_t)dst_slot) & 3u))
        return SPECKV_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t tp = compress_tile_pages(scheme);
    const uint32_t n_tiles = (uint32_t)(((unsigned long long)n + tp - 1) / tp);
    if (n_tiles > c->scan_tiles) return SPECKV_E_TOO_LARGE;   // more pages in one call than the context has slots
    if (cudaMemsetAsync(c->scan, 0, scan_bytes(n_tiles), st) != cudaSuccess) return SPECKV_E_CUDA;
    CompressArgs a;
    a.src = (const uint4 *)src; a.src_page = src_page; a.dst_slot = dst_slot;
    a.pool = c->pool; a.pte = c->pte; a.ctl = c->ctl; a.scan = c->scan;
    a.pool_gran = c->cfg.pool_bytes / kGranule; a.n_slots = c->n_slots;
    a.n_src_pages = n_src_pages; a.n = n; a.n_tiles = n_tiles; a.spin_limit = c->spin_limit; a.scheme = scheme;
    a.wait_ns = c->wait_ns;
    a.ticket0 = c->missing_tiles;   // one call only
    c->missing_tiles = 0;
    return launch_compress(a, c->n_sm, st) == cudaSuccess ? 0 : SPECKV_E_CUDA;
}

int speckv_translate(speckv_ctx *c, const int32_t *block_table, const speckv_vaddr *va, speckv_paddr *pa, uint32_t n,
                     void *stream)
{
    if (!c) return SPECKV_E_ARG;
    if (n == 0) return 0;
    if (!block_table || !va || !pa) return SPECKV_E_ARG;
    c->chain_live = false;
    TranslateArgs a;
    a.pte = c->pte; a.block_table = block_table; a.va = va; a.pa = pa; a.ctl = c->ctl;
    a.pool_bytes = c->cfg.pool_bytes; a.n = n; a.n_layers = c->cfg.n_layers; a.H = c->cfg.n_kv_heads;
    a.blocks_per_layer = c->cfg.blocks_per_layer; a.max_blocks_per_seq = c->cfg.max_blocks_per_seq;
    a.max_seqs = c->cfg.max_seqs;
    return launch_translate(a, (cudaStream_t)stream) == cudaSuccess ? 0 : SPECKV_E_CUDA;
}

int speckv_decompress_gather(speckv_ctx *c, uint32_t layer, const int32_t *block_table, const uint32_t *seq_lens,
                             const uint64_t *dst_tok_off, uint32_t B, const speckv_prefetch *pf, uint32_t n_pf,
                             void *dst_demand, uint64_t dst_cap_tokens, void *dst_l2, void *stream)
{
    if (!c || layer >= c->cfg.n_layers || B > c->cfg.max_seqs) return SPECKV_E_ARG;
    if (B == 0 && n_pf == 0) return 0;
    if (!block_table || (B && (!seq_lens || !dst_tok_off || !dst_demand)) || (n_pf && (!pf || !dst_l2))) return SPECKV_E_ARG;
    if (((uintptr_t)dst_demand & 15u) || ((uintptr_t)dst_l2 & 15u)) return SPECKV_E_ARG;
    if ((unsigned long long)n_pf * 2ull * c->cfg.n_kv_heads > 0x7FFFFFFFull) return SPECKV_E_ARG;
    c->epoch += 1;
    GatherArgs a;
    const uint64_t page_row = 2ull * c->cfg.n_kv_heads * SPECKV_HEAD_DIM * 2ull;   // bytes per token row of a sequence
    const speckv_ctx::Span dspan = {(uintptr_t)dst_demand, (uintptr_t)dst_demand + (B ? dst_cap_tokens * page_row : 0)};
    const speckv_ctx::Span lspan = {(uintptr_t)dst_l2, (uintptr_t)dst_l2 + (n_pf ? (uint64_t)c->cfg.max_seqs * SPECKV_L2_SLOTS * SPECKV_PAGE_TOKENS * page_row : 0)};
    a.chain = plan_gather_chain(c, (cudaStream_t)stream, dspan, lspan, n_pf != 0);
    a.pool = c->pool; a.pte = c->pte; a.l2_tag = c->l2_tag; a.ctl = c->ctl; a.block_table = block_table;
    a.seq_lens = seq_lens; a.dst_tok_off = (const unsigned long long *)dst_tok_off; a.pf = pf;
    a.dst_demand = (uint4 *)dst_demand; a.dst_l2 = (uint4 *)dst_l2; a.pool_bytes = c->cfg.pool_bytes;
    a.dst_cap_tokens = dst_cap_tokens; a.layer = layer; a.B = B; a.n_pf = n_pf; a.epoch = c->epoch;
    a.n_layers = c->cfg.n_layers; a.H = c->cfg.n_kv_heads; a.blocks_per_layer = c->cfg.blocks_per_layer;
    a.max_blocks_per_seq = c->cfg.max_blocks_per_seq; a.max_seqs = c->cfg.max_seqs;
    return launch_gather(a, c->n_sm, (cudaStream_t)stream) == cudaSuccess ? 0 : SPECKV_E_CUDA;
}

int speckv_compress_host(speckv_ctx *c, const void *src_host, uint32_t n_src_pages, void *staging,
                         const uint32_t *src_page, const uint32_t *dst_slot, uint32_t n, int scheme, void *stream)
{
    if (!c || !src_host || !staging || ((uintptr_t)staging & 15u)) return SPECKV_E_ARG;
    if (cudaMemcpyAsync(staging, src_host, (size_t)n_src_pages * kPageBytes, cudaMemcpyHostToDevice,
                        (cudaStream_t)stream) != cudaSuccess)
        return SPECKV_E_CUDA;
    return speckv_compress(c, staging, n_src_pages, src_page, dst_slot, n, scheme, stream);
}

int speckv_decompress_gather_host(speckv_ctx *c, uint32_t layer, const int32_t *block_table, const uint32_t *seq_lens,
                                  const uint64_t *dst_tok_off, uint32_t B, const speckv_prefetch *pf, uint32_t n_pf,
                                  void *dst_demand, uint64_t dst_cap_tokens, void *dst_l2, void *dst_host,
                                  uint64_t copy_bytes, void *stream)
{
    if (!c || !dst_host || !dst_demand) return SPECKV_E_ARG;
    if (copy_bytes > dst_cap_tokens * 2ull * c->cfg.n_kv_heads * SPECKV_HEAD_DIM * 2ull) return SPECKV_E_ARG;
    int rc = speckv_decompress_gather(c, layer, block_table, seq_lens, dst_tok_off, B, pf, n_pf, dst_demand,
                                      dst_cap_tokens, dst_l2, stream);
    if (rc) return rc;
    if (cudaMemcpyAsync(dst_host, dst_demand, copy_bytes, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return SPECKV_E_CUDA;
    return 0;
}

// ---- pool lifecycle

uint64_t speckv_compact_scratch_bytes(speckv_ctx *c)
{
    return c ? compact_scratch_bytes(c->n_slots, c->cfg.pool_bytes) : 0;
}

int speckv_compact(speckv_ctx *c, void *scratch, uint64_t scratch_bytes, void *stream)
{
    if (!c || !scratch || ((uintptr_t)scratch & 255u) || scratch_bytes < speckv_compact_scratch_bytes(c)) return SPECKV_E_ARG;
    c->chain_live = false;
    return launch_compact(c->pool, c->cfg.pool_bytes, c->pte, c->n_slots, c->ctl, (uint8_t *)scratch, c->n_sm,
                          (cudaStream_t)stream) == cudaSuccess ? 0 : SPECKV_E_CUDA;
}

int speckv_free_slots(speckv_ctx *c, const uint32_t *slots, uint32_t n, uint64_t *freed, void *stream)
{
    if (!c) return SPECKV_E_ARG;
    if (n == 0) return 0;
    if (!slots || ((uintptr_t)slots & 3u) || ((uintptr_t)freed & 7u)) return SPECKV_E_ARG;
    c->chain_live = false;
    return launch_free_slots(c->pte, c->n_slots, c->ctl, slots, n, (unsigned long long *)freed, (cudaStream_t)stream) == cudaSuccess
               ? 0 : SPECKV_E_CUDA;
}

// ---- decode-step attention over fetched pages

static size_t attend_prefix_bytes(uint32_t B) { return (((size_t)B + 1) * 4 + 255) & ~(size_t)255; }

// one partial result (8 heads x (128 + 2) binary32) per warp of the launch and per (sequence, KV head)
uint64_t speckv_attend_workspace_bytes(uint32_t B, uint32_t n_kv_heads)
{
    return attend_prefix_bytes(B) + ((uint64_t)attend_max_warps() + (uint64_t)B * n_kv_heads) * 8ull * 130ull * 4ull;
}

static int attend_common(speckv_ctx *c, AttendArgs &a, bool fused, const uint32_t *seq_lens, uint32_t B, const void *q,
                         uint32_t n_q_heads, void *out, void *workspace, uint64_t workspace_bytes, void *stream)
{
    const uint32_t H = c->cfg.n_kv_heads;
    if (B > 512u || n_q_heads == 0 || n_q_heads % H || n_q_heads / H > 8u) return SPECKV_E_ARG;
    if (B == 0) return 0;
    if (!seq_lens || !q || !out || !workspace || ((uintptr_t)q & 15u) || ((uintptr_t)out & 15u) || ((uintptr_t)workspace & 255u))
        return SPECKV_E_ARG;
    if (workspace_bytes < speckv_attend_workspace_bytes(B, H)) return SPECKV_E_ARG;
    if ((cudaStream_t)stream == c->chain_stream) c->chain_live = false;   // an ordinary launch: later gathers do not chain past it
    a.ctl = c->ctl; a.seq_lens = seq_lens; a.q = (const __half *)q; a.out = (__half *)out;
    a.prefix = (uint32_t *)workspace;
    a.partial = (float *)((uint8_t *)workspace + attend_prefix_bytes(B));
    a.B = B; a.H = H; a.G = n_q_heads / H;
    return launch_attend(a, fused, c->n_sm, (cudaStream_t)stream) == cudaSuccess ? 0 : SPECKV_E_CUDA;
}

int speckv_attend_dense(speckv_ctx *c, const void *kv, const uint32_t *seq_lens, const uint64_t *dst_tok_off, uint32_t B,
                        const void *q, uint32_t n_q_heads, void *out, void *workspace, uint64_t workspace_bytes, void *stream)
{
    if (!c) return SPECKV_E_ARG;
    if (B && (!kv || !dst_tok_off || ((uintptr_t)kv & 15u))) return SPECKV_E_ARG;
    AttendArgs a = {};
    a.kv = (const uint4 *)kv; a.tok_off = (const unsigned long long *)dst_tok_off;
    return attend_common(c, a, false, seq_lens, B, q, n_q_heads, out, workspace, workspace_bytes, stream);
}

int speckv_decompress_attend(speckv_ctx *c, uint32_t layer, const int32_t *block_table, const uint32_t *seq_lens, uint32_t B,
                             const void *q, uint32_t n_q_heads, void *out, void *workspace, uint64_t workspace_bytes,
                             void *stream)
{
    if (!c || layer >= c->cfg.n_layers || B > c->cfg.max_seqs) return SPECKV_E_ARG;
    if (B && !block_table) return SPECKV_E_ARG;
    AttendArgs a = {};
    a.pool = c->pool; a.pte = c->pte; a.block_table = block_table; a.pool_bytes = c->cfg.pool_bytes;
    a.layer = layer; a.blocks_per_layer = c->cfg.blocks_per_layer; a.max_blocks_per_seq = c->cfg.max_blocks_per_seq;
    return attend_common(c, a, true, seq_lens, B, q, n_q_heads, out, workspace, workspace_bytes, stream);
}

// ---- multi-layer pipelined prefetch (Sec. 3.4.4)

static int pipeline_setup(speckv_ctx *c)
{
    if (c->pipeline_ready) return 0;
    if (cudaStreamCreateWithFlags(&c->fetch_stream, cudaStreamNonBlocking) != cudaSuccess) return SPECKV_E_CUDA;
    bool ok = cudaEventCreateWithFlags(&c->ev_start, cudaEventDisableTiming) == cudaSuccess;
    for (uint32_t i = 0; i < speckv_ctx::kMaxRing; ++i)
        ok = ok && cudaEventCreateWithFlags(&c->ev_fetched[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->ev_consumed[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return SPECKV_E_CUDA;
    c->pipeline_ready = true;
    return 0;
}

int speckv_pipeline_layers(speckv_ctx *c, uint32_t layer0, uint32_t n_layers, const int32_t *block_table,
                           const uint32_t *seq_lens, const uint64_t *dst_tok_off, uint32_t B, void *ring,
                           uint32_t ring_slots, uint64_t slot_tokens, speckv_layer_fn consume, void *user, void *stream)
{
    if (!c || !consume || !ring || ((uintptr_t)ring & 15u) || ring_slots < 1 || ring_slots > speckv_ctx::kMaxRing ||
        (uint64_t)layer0 + n_layers > c->cfg.n_layers || B > c->cfg.max_seqs)
        return SPECKV_E_ARG;
    if (n_layers == 0) return 0;
    int rc = pipeline_setup(c);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream, fs = c->fetch_stream;
    const uint64_t slot_bytes = slot_tokens * 2ull * c->cfg.n_kv_heads * SPECKV_HEAD_DIM * 2ull;
    // the fetch stream starts after whatever the caller has enqueued so far (the writes of the pages, say)
    if (cudaEventRecord(c->ev_start, st) != cudaSuccess || cudaStreamWaitEvent(fs, c->ev_start, 0) != cudaSuccess) return SPECKV_E_CUDA;
    for (uint32_t l = 0; l < n_layers; ++l) {
        const uint32_t r = l % ring_slots;
        uint8_t *slot = (uint8_t *)ring + (uint64_t)r * slot_bytes;
        if (l >= ring_slots) {
            // the slot is free once the computation of the layer that used it has finished; a gather that
            // follows an event wait is launched as an ordinary, fully ordered kernel
            if (cudaStreamWaitEvent(fs, c->ev_consumed[r], 0) != cudaSuccess) return SPECKV_E_CUDA;
            c->chain_live = false;
        }
        rc = speckv_decompress_gather(c, layer0 + l, block_table, seq_lens, dst_tok_off, B, nullptr, 0, slot, slot_tokens, nullptr, fs);
        if (rc) return rc;
        if (cudaEventRecord(c->ev_fetched[r], fs) != cudaSuccess || cudaStreamWaitEvent(st, c->ev_fetched[r], 0) != cudaSuccess)
            return SPECKV_E_CUDA;
        rc = consume(user, layer0 + l, slot, stream);
        if (rc) return rc;
        if (cudaEventRecord(c->ev_consumed[r], st) != cudaSuccess) return SPECKV_E_CUDA;
    }
    c->chain_live = false;
    return 0;
}

struct PipelineAttend {
    speckv_ctx *c;
    const uint32_t *seq_lens;
    const uint64_t *tok_off;
    uint32_t B, n_q_heads, layer0;
    const uint8_t *q;
    uint8_t *out;
    void *workspace;
    uint64_t workspace_bytes;
};
static int pipeline_attend_layer(void *user, uint32_t layer, const void *kv, void *stream)
{
    const PipelineAttend *p = (const PipelineAttend *)user;
    const uint64_t per_layer = (uint64_t)p->B * p->n_q_heads * SPECKV_HEAD_DIM * 2ull;
    return speckv_attend_dense(p->c, kv, p->seq_lens, p->tok_off, p->B, p->q + (layer - p->layer0) * per_layer, p->n_q_heads,
                               p->out + (layer - p->layer0) * per_layer, p->workspace, p->workspace_bytes, stream);
}

int speckv_pipeline_attend(speckv_ctx *c, uint32_t layer0, uint32_t n_layers, const int32_t *block_table,
                           const uint32_t *seq_lens, const uint64_t *dst_tok_off, uint32_t B, void *ring, uint32_t ring_slots,
                           uint64_t slot_tokens, const void *q, uint32_t n_q_heads, void *out, void *workspace,
                           uint64_t workspace_bytes, void *stream)
{
    if (!c || !q || !out) return SPECKV_E_ARG;
    PipelineAttend p = {c, seq_lens, (const uint64_t *)dst_tok_off, B, n_q_heads, layer0, (const uint8_t *)q, (uint8_t *)out,
                        workspace, workspace_bytes};
    return speckv_pipeline_layers(c, layer0, n_layers, block_table, seq_lens, dst_tok_off, B, ring, ring_slots, slot_tokens,
                                  pipeline_attend_layer, &p, stream);
}

// ---- managed prefetch buffer

int speckv_prefetch_step(speckv_ctx *c, uint32_t layer, uint32_t back, const int32_t *block_table, const int32_t *access,
                         const int32_t *cand, uint32_t B, double beta, speckv_pf_seq *state, speckv_pf_counters *cnt,
                         void *l2, void *miss_dst, int32_t *where, void *stream)
{
    if (!c || layer >= c->cfg.n_layers || back > 1u || B > c->cfg.max_seqs || B > prefetch_max_seqs() || !(beta >= 0.0))
        return SPECKV_E_ARG;
    if (B == 0) return 0;
    if (!block_table || !access || !cand || !state || !cnt || !l2 || !miss_dst || !where || ((uintptr_t)l2 & 15u) ||
        ((uintptr_t)miss_dst & 15u) || ((uintptr_t)where & 15u) || ((uintptr_t)access & 15u) || ((uintptr_t)cand & 15u) ||
        ((uintptr_t)state & 15u) || ((uintptr_t)cnt & 15u) || ((uintptr_t)block_table & 15u))
        return SPECKV_E_ARG;
    c->chain_live = false;   // ordinary launches: later gathers do not chain past them
    PrefetchArgs a;
    a.pool = c->pool; a.pte = c->pte; a.ctl = c->ctl; a.block_table = block_table; a.access = access; a.cand = cand;
    a.state = state; a.cnt = cnt; a.l2 = (uint4 *)l2; a.miss_dst = (uint4 *)miss_dst; a.where = where; a.beta = beta;
    a.pool_bytes = c->cfg.pool_bytes; a.layer = layer; a.back = back; a.B = B; a.H = c->cfg.n_kv_heads;
    a.blocks_per_layer = c->cfg.blocks_per_layer; a.max_blocks_per_seq = c->cfg.max_blocks_per_seq; a.max_seqs = c->cfg.max_seqs;
    return launch_prefetch_step(a, c->n_sm, (cudaStream_t)stream) == cudaSuccess ? 0 : SPECKV_E_CUDA;
}

int speckv_get_status(speckv_ctx *c, speckv_status *out, void *stream)
{
    if (!c || !out) return SPECKV_E_ARG;
    c->chain_live = false;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return SPECKV_E_CUDA;
    Ctl h;
    if (cudaMemcpy(&h, c->ctl, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return SPECKV_E_CUDA;
    memcpy(out->count, h.status_count, sizeof(out->count));
    memcpy(out->first, h.status_first, sizeof(out->first));
    return 0;
}

int speckv_get_stats(speckv_ctx *c, speckv_stats *out, void *stream)
{
    if (!c || !out) return SPECKV_E_ARG;
    c->chain_live = false;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return SPECKV_E_CUDA;
    Ctl h;
    if (cudaMemcpy(&h, c->ctl, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return SPECKV_E_CUDA;
    memcpy(out, h.stats, sizeof(*out));
    return 0;
}

int speckv_get_cursor(speckv_ctx *c, uint64_t *cursor64, void *stream)
{
    if (!c || !cursor64) return SPECKV_E_ARG;
    c->chain_live = false;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return SPECKV_E_CUDA;
    unsigned long long v = 0;
    if (cudaMemcpy(&v, &c->ctl->cursor64, 8, cudaMemcpyDeviceToHost) != cudaSuccess) return SPECKV_E_CUDA;
    *cursor64 = v;
    return 0;
}

void *speckv_pool_ptr(speckv_ctx *c) { return c ? c->pool : nullptr; }
void *speckv_pte_ptr(speckv_ctx *c) { return c ? c->pte : nullptr; }
void *speckv_l2_tag_ptr(speckv_ctx *c) { return c ? c->l2_tag : nullptr; }

}  // extern "C"
