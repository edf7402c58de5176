// speckv_decompress_gather and speckv_translate on sm_100a.
//
// Decompression pipeline of CXL-SpecKV (run expansion -> running sum of deltas ->
// dequantisation, with the bypass for uncompressed records) fused with the paged gather that
// the address translation unit and the prefetch list feed.
//
// A warp takes its pages 32 at a time.  The translation chain (logical block -> block table ->
// page-table entry (+ residency tag) -> checks) is walked by the lanes side by side, one page per
// lane, so that every dependent load is in flight for 32 pages at once (the role of the paper's
// outstanding-request window) and the bookkeeping costs one instruction stream per 32 pages.
// Delivery is by the whole warp, page after page: bulk async copy of the record into one of two
// shared-memory buffers (mbarrier completion) while the previous record is decoded; header check,
// decode, eight coalesced 128-bit stores per lane.
// Lane layout of the decode is the compressor's: lane l, group k = the 8 elements at 256*k + 8*l.
#include "async_ptx.cuh"
#include "decode.cuh"
#include "speckv_dev.cuh"

namespace speckv {

constexpr int kGWarps = 8;
constexpr int kGThreads = kGWarps * 32;
constexpr uint32_t kMaxSeqs = 4096;
constexpr uint32_t kStage = kRecStage;                    // bytes per record buffer

// ---------------------------------------------------------------- address translation

__global__ void __launch_bounds__(256) translate_kernel(TranslateArgs a)
{
    uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.n) return;
    speckv_vaddr v = a.va[i];
    const uint32_t block = v.pos >> 4;
    Walk w{0ull, 0u, 0u, SPECKV_ST_UNMAPPED};
    if (v.seq < a.max_seqs && block < a.max_blocks_per_seq && v.layer < a.n_layers && v.kv <= 1u && v.head < a.H) {
        int32_t p = __ldg(a.block_table + (size_t)v.seq * a.max_blocks_per_seq + block);
        if (p >= 0 && (uint32_t)p < a.blocks_per_layer) {
            unsigned long long slot = (((unsigned long long)v.layer * a.blocks_per_layer + (uint32_t)p) * 2u + v.kv) * a.H + v.head;
            w = decode_pte(__ldg(a.pte + slot), a.pool_bytes);
        }
    }
    speckv_paddr p;
    p.byte_off = w.rc ? 0ull : w.byte_off;
    p.rec_len = w.rc ? 0u : w.rec_len;
    p.mode = w.rc ? 0 : (uint8_t)w.mode;
    p.status = (uint8_t)w.rc;
    p.rsvd = 0;
    a.pa[i] = p;
    if (w.rc) raise_status(a.ctl, w.rc, i);
}

// ---------------------------------------------------------------- the pipelined gather

__global__ void __launch_bounds__(kGThreads, 4) gather_kernel(GatherArgs a)
{
    extern __shared__ __align__(16) uint8_t smem[];
    uint8_t *s_rec = smem;                                                        // [kGWarps][2][kStage]
    uint4 *s_lut = reinterpret_cast<uint4 *>(smem + kGWarps * 2 * kStage);   // [256]
    unsigned long long *s_bar = reinterpret_cast<unsigned long long *>(s_lut + 256);   // [kGWarps][2]
    unsigned long long *s_tok = s_bar + kGWarps * 2;                              // [B] first token row of each sequence
    uint32_t *s_pref = reinterpret_cast<uint32_t *>(s_tok + a.B);                 // [B + 1] exclusive prefix of blocks

    // Consecutive gather launches are chained programmatically: the next launch may become resident
    // while this one drains.  A chained launch runs everything that only reads (set-up, translation,
    // record fetches) at once; it waits for its predecessor before it writes a page or touches a
    // residency tag, unless the host has established that the two launches are independent
    // (no prefetch lists, destinations that do not overlap).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const uint32_t tid = threadIdx.x, lane = tid & 31u;
    const uint32_t warp = __shfl_sync(kFull, tid >> 5, 0);                        // warp-uniform for the compiler too
    s_lut[tid & 255u] = expand_entry(tid & 255u);
    if (tid < kGWarps * 2) mbar_init(smem_u32(s_bar + tid), 1);
    // blocks per sequence; a length that the block table cannot describe contributes none (reported below)
    for (uint32_t b = tid; b < a.B; b += kGThreads) {
        const uint32_t nb = (uint32_t)(((unsigned long long)a.seq_lens[b] + 15ull) >> 4);
        s_pref[b + 1] = nb > a.max_blocks_per_seq ? 0u : nb;
        s_tok[b] = a.dst_tok_off[b];
    }
    if (tid == 0) s_pref[0] = 0;
    mbar_init_fence();
    __syncthreads();
    for (uint32_t d = 1; d < a.B; d <<= 1) {                                      // inclusive scan in place
        uint32_t add[(kMaxSeqs + kGThreads - 1) / kGThreads];
        int j = 0;
        for (uint32_t b = tid; b < a.B; b += kGThreads, ++j) add[j] = (b >= d) ? s_pref[b + 1 - d] : 0u;
        __syncthreads();
        j = 0;
        for (uint32_t b = tid; b < a.B; b += kGThreads, ++j) s_pref[b + 1] += add[j];
        __syncthreads();
    }

    if (blockIdx.x == 0)      // once per launch: sequences left out, at the index their first page would have had
        for (uint32_t b = tid; b < a.B; b += kGThreads)
            if ((((unsigned long long)a.seq_lens[b] + 15ull) >> 4) > a.max_blocks_per_seq) raise_status(a.ctl, SPECKV_ST_UNMAPPED, s_pref[b] * 2u * a.H);
    // Unit decomposition: a unit is a logical block (demand blocks first, then prefetch entries);
    // this warp serves page r = (kv, head) of the units g0, g0 + gstep, ...  The host sizes the grid so
    // that the number of warps is a multiple of 2*H.
    const uint32_t twoH = 2u * a.H;
    const uint32_t n_blocks = s_pref[a.B], n_units = n_blocks + a.n_pf;
    const uint32_t n_warps = gridDim.x * kGWarps, gw = blockIdx.x * kGWarps + warp;
    const uint32_t r = gw % twoH, gstep = n_warps / twoH, g0 = gw / twoH;
    const uint32_t n_mine = g0 < n_units ? (n_units - g0 + gstep - 1u) / gstep : 0u;
    uint32_t n_issued = 0, n_consumed = 0;
    uint8_t *my_rec = s_rec + warp * 2 * kStage;
    const uint32_t my_bar = smem_u32(s_bar + warp * 2);
    const unsigned long long layer_slot0 = (unsigned long long)a.layer * a.blocks_per_layer * twoH + r;
    unsigned long long st_decoded = 0, st_issued = 0, st_skipped = 0;

    // Prefetch entries read and write the residency tags, which the previous launch may still be
    // updating: with a prefetch list, wait for it before translating anything.
    if (a.chain != 2u && a.n_pf) asm volatile("griddepcontrol.wait;" ::: "memory");
    bool waited = a.chain == 2u || a.n_pf != 0u;

    // The warp's pages are taken 32 at a time.  Translation is done by the lanes side by side, one page
    // per lane (sequence look-up, block table, page-table entry, checks: each dependent load is in
    // flight for 32 pages at once); then the pages are delivered one after the other by the whole
    // warp, the next record's bulk copy running while the current one is decoded.
    for (uint32_t first = 0; first < n_mine; first += 32u) {
        // ---- translation: lane l owns page first + l of this warp
        uint4 *dst = nullptr;
        unsigned long long pte = 0ull;
        uint32_t index = 0;
        int state = 0;               // 0 = nothing to deliver, 3 = packed record, 4 = raw record
        if (first + lane < n_mine) {
            const uint32_t unit = g0 + (first + lane) * gstep;
            index = unit * twoH + r;
            int32_t bt_val = -1;
            bool go = false;
            if (unit < n_blocks) {
                uint32_t lo = 0, hi = a.B;                                   // sequence: last b with s_pref[b] <= unit
                while (hi - lo > 1u) { const uint32_t mid = (lo + hi) >> 1; if (s_pref[mid] <= unit) lo = mid; else hi = mid; }
                const uint32_t seq = lo, seq_first = s_pref[seq], block = unit - seq_first;
                const unsigned long long tpad = (unsigned long long)(s_pref[seq + 1] - seq_first) * 16ull, tok = s_tok[seq];
                if (tok + tpad > a.dst_cap_tokens) raise_status(a.ctl, SPECKV_ST_BAD_DST, index);
                else if (block >= a.max_blocks_per_seq) raise_status(a.ctl, SPECKV_ST_UNMAPPED, index);
                else {
                    dst = a.dst_demand + (tok * twoH + (unsigned long long)r * tpad) * 16ull + (size_t)block * (kPageBytes / 16);
                    bt_val = __ldg(a.block_table + (size_t)seq * a.max_blocks_per_seq + block);
                    go = true;
                }
            } else {
                // prefetch entry: translate and pass the residency filter
                const speckv_prefetch p = a.pf[unit - n_blocks];
                int32_t pb = -1;
                if (p.seq < a.max_seqs && p.l2_slot < SPECKV_L2_SLOTS && p.block < a.max_blocks_per_seq)
                    pb = __ldg(a.block_table + (size_t)p.seq * a.max_blocks_per_seq + p.block);
                if (pb < 0 || (uint32_t)pb >= a.blocks_per_layer) raise_status(a.ctl, SPECKV_ST_UNMAPPED, index);
                else {
                    const uint32_t tag = a.layer * (1u << 20) + p.block + 1u;
                    unsigned long long *tp = a.l2_tag + (size_t)p.seq * SPECKV_L2_SLOTS + p.l2_slot;
                    const unsigned long long old = *reinterpret_cast<volatile unsigned long long *>(tp);
                    if ((uint32_t)old == tag && (uint32_t)(old >> 32) != a.epoch) {      // tagged by an earlier call: resident
                        if (r == 0) st_skipped += 1;
                    } else {
                        if (r == 0) {
                            *reinterpret_cast<volatile unsigned long long *>(tp) = ((unsigned long long)a.epoch << 32) | tag;
                            st_issued += 1;
                        }
                        dst = a.dst_l2 + (((size_t)p.seq * SPECKV_L2_SLOTS + p.l2_slot) * twoH + r) * (kPageBytes / 16);
                        bt_val = pb;
                        go = true;
                    }
                }
            }
            if (go) {
                if (bt_val < 0 || (uint32_t)bt_val >= a.blocks_per_layer) raise_status(a.ctl, SPECKV_ST_UNMAPPED, index);
                else {
                    pte = __ldg(a.pte + layer_slot0 + (unsigned long long)(uint32_t)bt_val * twoH);
                    const Walk w = decode_pte(pte, a.pool_bytes);
                    if (w.rc) raise_status(a.ctl, w.rc, index);
                    else if (w.mode == SPECKV_RAW) state = 4;
                    else if ((w.mode & ~(uint32_t)SPECKV_GROUPED) - 1u > 2u || w.rec_len > kMaxPackedRec) raise_status(a.ctl, SPECKV_ST_BAD_RECORD, index);
                    else state = 3;
                }
            }
        }
        // ---- delivery, in page order
        uint32_t live = __ballot_sync(kFull, state != 0), packed = __ballot_sync(kFull, state == 3);
        uint32_t ahead = packed;                             // packed records whose copy has not been issued yet
        while (live) {
            const uint32_t l = __ffs(live) - 1u;
            live &= live - 1u;
            const bool is_packed = (packed >> l) & 1u;
            // keep two bulk copies in flight: this page's record (if not requested yet) and the next one's
            while (is_packed && ahead && n_issued < n_consumed + 2u) {
                const uint32_t nl = __ffs(ahead) - 1u;
                ahead &= ahead - 1u;
                const unsigned long long ne = __shfl_sync(kFull, pte, nl);
                if (lane == 0) {
                    const uint32_t bytes = (((uint32_t)(ne >> 32) & 0xFFFFu) + 15u) & ~15u, buf = n_issued & 1u, bar = my_bar + 8u * buf;
                    mbar_expect_tx(bar, bytes);
                    bulk_g2s(smem_u32(my_rec + buf * kStage), a.pool + (ne & 0xFFFFFFFFull) * kGranule, bytes, bar);
                }
                ++n_issued;
            }
            // destinations may be shared with the previous launch: no page is written before it has finished
            if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
            const unsigned long long e = __shfl_sync(kFull, pte, l);
            uint4 *d = reinterpret_cast<uint4 *>(__shfl_sync(kFull, (unsigned long long)dst, l));
            const uint32_t rec_len = (uint32_t)(e >> 32) & 0xFFFFu, pte_mode = (uint32_t)(e >> 48) & 0xFFu;
            bool ok;
            if (!is_packed) {                                                         // bypass: straight copy of the page
                const uint4 *src = reinterpret_cast<const uint4 *>(a.pool + (e & 0xFFFFFFFFull) * kGranule);
                const uint4 hdr = __ldg(src);
                ok = (hdr.y >> 24) == kVersion && ((hdr.y >> 16) & 0xFFu) == SPECKV_RAW && (hdr.y & 0xFFFFu) == kPageBytes &&
                     rec_len == kHdrBytes + kPageBytes;
                if (ok) {
                    uint4 t[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) t[k] = __ldg(src + 1 + k * 32 + lane);
#pragma unroll
                    for (int k = 0; k < 8; ++k) d[k * 32 + lane] = t[k];
                }
            } else {
                const uint32_t buf = n_consumed & 1u, parity = (n_consumed >> 1) & 1u;
                ++n_consumed;
                const uint8_t *rec = my_rec + buf * kStage;
                if (!mbar_wait(my_bar + 8u * buf, parity)) {                          // never expected: report, skip the page
                    if (lane == l) raise_status(a.ctl, SPECKV_ST_TIMEOUT, index);
                    continue;
                }
                const uint4 hdr = *reinterpret_cast<const uint4 *>(rec);
                const uint32_t payload_len = hdr.y & 0xFFFFu, mode = (hdr.y >> 16) & 0xFFu;
                ok = (hdr.y >> 24) == kVersion && mode == pte_mode && kHdrBytes + payload_len == rec_len;
                if (ok) ok = decode_page(rec, mode, payload_len, hdr.z & 0xFFFFu, __uint_as_float(hdr.x), s_lut, lane,
                                         [&](int k, const uint4 &v) { d[k * 32 + lane] = v; });
                __syncwarp();                                                         // buffer may be refilled after this
            }
            if (!ok) { if (lane == l) raise_status(a.ctl, SPECKV_ST_BAD_RECORD, index); continue; }
            st_decoded += 1;
        }
    }
    // A chained launch that was allowed to skip the wait (independent of its predecessor) still may not
    // end before it: work ordered after this grid must find the predecessor's pages written too.  Waiting
    // here, after the last store, costs nothing but keeps completion in stream order.
    if (!waited || a.chain == 2u) asm volatile("griddepcontrol.wait;" ::: "memory");
    // st_decoded is warp-uniform; st_issued and st_skipped are per lane (one prefetch entry each)
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        st_issued += __shfl_xor_sync(kFull, st_issued, d);
        st_skipped += __shfl_xor_sync(kFull, st_skipped, d);
    }
    if (lane == 0) {
        if (st_decoded) atomicAdd(&a.ctl->stats[kStDecoded], st_decoded);
        if (st_issued) atomicAdd(&a.ctl->stats[kStPfIssued], st_issued);
        if (st_skipped) atomicAdd(&a.ctl->stats[kStPfSkipped], st_skipped);
    }
}

static size_t gather_smem_bytes(uint32_t B)
{
    return (size_t)kGWarps * 2 * kStage + 256 * 16 + kGWarps * 2 * 8 + (size_t)B * 8 + ((size_t)B + 1) * 4;
}

cudaError_t launch_gather(const GatherArgs &a, int n_sm, cudaStream_t stream)
{
    const size_t smem = gather_smem_bytes(a.B);
    if (smem > 48u * 1024u) {   // only long batches need the opt-in limit
        cudaError_t e = cudaFuncSetAttribute(gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gather_smem_bytes(kMaxSeqs));
        if (e != cudaSuccess) return e;
    }
    // the kernel needs a warp count that is a multiple of 2*H (every warp keeps one (kv, head))
    const uint32_t twoH = 2u * a.H;
    uint32_t m = twoH, x = kGWarps;
    while (x) { uint32_t t = m % x; m = x; x = t; }          // m = gcd(twoH, kGWarps)
    const uint32_t mult = twoH / m;
    uint32_t grid = (uint32_t)n_sm * 4u;                     // 32 warps per SM at 64 registers: measured faster than 24 at 80
    grid = grid >= mult ? grid - grid % mult : mult;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kGThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.chain ? 1 : 0;                          // an ordinary launch waits for all earlier work
    return cudaLaunchKernelEx(&cfg, gather_kernel, a);
}

cudaError_t launch_translate(const TranslateArgs &a, cudaStream_t stream)
{
    translate_kernel<<<(a.n + 255u) / 256u, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

uint32_t gather_max_seqs() { return kMaxSeqs; }

}  // namespace speckv
