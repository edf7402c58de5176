// speckv_prefetch_step: the managed prefetch buffer of CXL-SpecKV on sm_100a — tier L2 with its two
// banks (Sec. 3.3.1), misprediction handling (Sec. 3.4.3: lazy invalidation, fallback fetch, depth
// adapted per request) and the depth rule of Sec. 3.6.3 (upper confidence bound over depths 1..4).
//
// Two launches per call:
//   pf_plan_kernel   four threads per sequence (one per depth score): looks this step's reads up in the readable bank, scores
//                    the fill that is about to be overwritten, picks the depth, retags the slots of the
//                    bank being filled.  Everything that touches tags and statistics happens here, in a
//                    fixed order per sequence, so the outcome does not depend on scheduling.
//   pf_fetch_kernel  the transfers the plan decided on — reads that missed and slots to refill — as a
//                    paged gather with decompression: every CTA compacts the live (sequence, read|slot)
//                    units into shared memory, then each warp takes its pages 32 at a time like the
//                    demand gather: translation (block table -> page-table entry -> checks) by the lanes
//                    side by side, delivery page after page with two record copies in flight.  It is
//                    launched programmatically dependent on the plan, so its set-up overlaps the plan
//                    and it waits for the plan's results before it reads them.
#include "async_ptx.cuh"
#include "decode.cuh"
#include "speckv_dev.cuh"

namespace speckv {

constexpr uint32_t kPfMaxSeqs = 512;
constexpr int kPfWarps = 8;
constexpr int kPfThreads = kPfWarps * 32;
constexpr uint32_t kPfUnits = 2u * SPECKV_L2_SLOTS;             // per sequence: 4 reads + 4 slots

// ---------------------------------------------------------------- depth rule

// mu_k + beta * sqrt(2 ln T / N_k), binary64, one rounding per operation (no contraction);
// ln T is kept to 20 fractional bits so that the choice does not hang on the logarithm's last bits
__device__ __forceinline__ double depth_score(int reward, uint32_t plays, uint32_t steps, double beta)
{
    const double n = (double)plays;
    const double mean = __ddiv_rn((double)reward, __dmul_rn(8.0, n));
    const double ln_t = __ddiv_rn(rint(__dmul_rn(log((double)steps), 1048576.0)), 1048576.0);
    const double bonus = __dmul_rn(beta, __dsqrt_rn(__ddiv_rn(__dmul_rn(2.0, ln_t), n)));
    return __dadd_rn(mean, bonus);
}

__global__ void __launch_bounds__(32) pf_plan_kernel(PrefetchArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the fetch kernel may start its set-up
    // Four threads per sequence.  All four walk the sequence's (short) bookkeeping alike, so that each holds
    // the updated statistics; the four depth scores — a binary64 logarithm, square root and two divisions
    // each, the long pole of this kernel — are then evaluated side by side, one per thread.  Only the first
    // thread of a quad reports, counts and stores.
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t b = t >> 2, arm = t & 3u;
    const bool lead = arm == 0;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t live = __ballot_sync(kFull, b < a.B);   // whole quads: the lanes that take part in the shuffles below
    unsigned long long n_acc = 0, n_hit = 0, n_late = 0, n_miss = 0, n_fetch = 0, n_kept = 0, n_evict = 0, n_evict_used = 0;
    if (b < a.B) {
        speckv_pf_seq s = a.state[b];
        const uint32_t back = a.back, front = back ^ 1u, twoH = 2u * a.H;
        const int4 acc4 = reinterpret_cast<const int4 *>(a.access)[b];
        const int4 cand4 = reinterpret_cast<const int4 *>(a.cand)[b];
        const int32_t acc[4] = {acc4.x, acc4.y, acc4.z, acc4.w}, cand[4] = {cand4.x, cand4.y, cand4.z, cand4.w};
        // 1. reads: only the bank filled by the previous call may be read
        int32_t wh[4];
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) {
            wh[i] = -2;
            if (acc[i] < 0) continue;
            if ((uint32_t)acc[i] >= a.max_blocks_per_seq) {
                if (lead)
                    for (uint32_t r = 0; r < twoH; ++r) raise_status(a.ctl, SPECKV_ST_UNMAPPED, (b * 4u + i) * twoH + r);
                continue;
            }
            const uint32_t tag = a.layer * (1u << 20) + (uint32_t)acc[i] + 1u;
            n_acc += 1;
            int hit = -1;
            bool late = false;
#pragma unroll
            for (int j = 3; j >= 0; --j) {
                if (s.tag[front][j] == tag) hit = j;                  // the lowest matching slot wins
                if (s.tag[back][j] == tag) late = true;
            }
            if (hit >= 0) {
                s.used[front][hit] = 1;
                n_hit += 1;
                wh[i] = (int32_t)(front * 4u) + hit;
            } else {
                n_miss += 1;
                if (late) n_late += 1;
                wh[i] = -1;
            }
        }
        if (lead) reinterpret_cast<int4 *>(a.where)[b] = make_int4(wh[0], wh[1], wh[2], wh[3]);
        // 2. score the fill that is about to be overwritten
        const uint32_t d = s.depth[back];
        if (d > 0) {
            int valid = 0, useful = 0;
            for (uint32_t j = 0; j < d && j < 4u; ++j)
                if (s.tag[back][j] != 0) { valid += 1; useful += s.used[back][j] ? 1 : 0; }
            s.reward[d - 1] += 3 * useful - valid;
            s.plays[d - 1] += 1;
            s.steps += 1;
        }
        // 3. depth of this fill
        uint32_t k = 0;
        for (uint32_t j = 0; j < 4 && !k; ++j)
            if (s.plays[j] == 0) k = j + 1;
        // (every thread of the quad takes this branch or none does: they hold the same statistics)
        const double mine = k ? 0.0 : depth_score(s.reward[arm], s.plays[arm], s.steps, a.beta);
        double sc[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) sc[j] = __shfl_sync(live, mine, j, 4);
        if (!k) {
            k = 1;
            double best = sc[0];
            for (uint32_t j = 1; j < 4; ++j)
                if (sc[j] > best) { best = sc[j]; k = j + 1; }                 // ties: the smaller depth
        }
        // 4. retag the slots of the bank being filled; the transfers follow in pf_fetch_kernel
        uint32_t fill = 0;
        for (uint32_t j = 0; j < k; ++j) {
            const int32_t cb = cand[j];
            if (cb < 0 || (uint32_t)cb >= a.max_blocks_per_seq) continue;
            const int32_t p = __ldg(a.block_table + (size_t)b * a.max_blocks_per_seq + (uint32_t)cb);
            if (p < 0 || (uint32_t)p >= a.blocks_per_layer) {
                if (lead)
                    for (uint32_t r = 0; r < twoH; ++r) raise_status(a.ctl, SPECKV_ST_UNMAPPED, ((a.B + b) * 4u + j) * twoH + r);
                continue;
            }
            const uint32_t tag = a.layer * (1u << 20) + (uint32_t)cb + 1u;
            if (s.tag[back][j] == tag) { s.used[back][j] = 0; n_kept += 1; continue; }
            if (s.tag[back][j] != 0) { n_evict += 1; n_evict_used += s.used[back][j] ? 1u : 0u; }
            s.tag[back][j] = tag;
            s.used[back][j] = 0;
            fill |= 1u << j;
            n_fetch += 1;
        }
        s.fill = (uint8_t)fill;
        s.depth[back] = (uint8_t)k;
        if (lead) a.state[b] = s;
    }
    if (!lead) n_acc = n_hit = n_late = n_miss = n_fetch = n_kept = n_evict = n_evict_used = 0;
    unsigned long long v[8] = {n_acc, n_hit, n_late, n_miss, n_fetch, n_kept, n_evict, n_evict_used};
    unsigned long long *out = reinterpret_cast<unsigned long long *>(a.cnt);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        unsigned long long x = v[c];
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) x += __shfl_xor_sync(kFull, x, d);
        if (lane == 0 && x) atomicAdd(out + c, x);
    }
}

// ---------------------------------------------------------------- the transfers

__global__ void __launch_bounds__(kPfThreads, 3) pf_fetch_kernel(PrefetchArgs a)
{
    extern __shared__ __align__(16) uint8_t smem[];
    uint8_t *s_rec = smem;                                                        // [kPfWarps][2][kRecStage]
    uint4 *s_lut = reinterpret_cast<uint4 *>(smem + kPfWarps * 2 * kRecStage);   // [256]
    unsigned long long *s_bar = reinterpret_cast<unsigned long long *>(s_lut + 256);   // [kPfWarps][2]
    uint32_t *s_cnt = reinterpret_cast<uint32_t *>(s_bar + kPfWarps * 2);         // [B + 1] live units before sequence b
    uint32_t *s_unit = s_cnt + a.B + 1;                                           // [<= 8 B] block << 12 | sequence << 3 | unit

    const uint32_t tid = threadIdx.x, lane = tid & 31u;
    const uint32_t warp = __shfl_sync(kFull, tid >> 5, 0);
    const uint32_t back = a.back, twoH = 2u * a.H;
    s_lut[tid & 255u] = expand_entry(tid & 255u);
    if (tid < kPfWarps * 2) mbar_init(smem_u32(s_bar + tid), 1);
    asm volatile("griddepcontrol.wait;" ::: "memory");                            // the plan's `where`, tags and fill masks
    // live units of each sequence: reads that missed (where = -1), slots transferred (fill bit)
    for (uint32_t b = tid; b < a.B; b += kPfThreads) {
        const int4 w = reinterpret_cast<const int4 *>(a.where)[b];
        const uint32_t n = (w.x == -1) + (w.y == -1) + (w.z == -1) + (w.w == -1) + __popc(a.state[b].fill & 15u);
        s_cnt[b + 1] = n;
    }
    if (tid == 0) s_cnt[0] = 0;
    mbar_init_fence();
    __syncthreads();
    for (uint32_t d = 1; d < a.B; d <<= 1) {                                      // inclusive scan in place
        uint32_t add[(kPfMaxSeqs + kPfThreads - 1) / kPfThreads];
        int j = 0;
        for (uint32_t b = tid; b < a.B; b += kPfThreads, ++j) add[j] = (b >= d) ? s_cnt[b + 1 - d] : 0u;
        __syncthreads();
        j = 0;
        for (uint32_t b = tid; b < a.B; b += kPfThreads, ++j) s_cnt[b + 1] += add[j];
        __syncthreads();
    }
    for (uint32_t b = tid; b < a.B; b += kPfThreads) {
        const int4 w = reinterpret_cast<const int4 *>(a.where)[b];
        const int4 ac = reinterpret_cast<const int4 *>(a.access)[b];
        const int32_t wh[4] = {w.x, w.y, w.z, w.w}, blk[4] = {ac.x, ac.y, ac.z, ac.w};
        const uint32_t fill = a.state[b].fill & 15u;
        uint32_t o = s_cnt[b];
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i)
            if (wh[i] == -1) s_unit[o++] = ((uint32_t)blk[i] << 12) | (b << 3) | i;
#pragma unroll
        for (uint32_t j = 0; j < 4; ++j)
            if (fill & (1u << j)) s_unit[o++] = (((a.state[b].tag[back][j] & 0xFFFFFu) - 1u) << 12) | (b << 3) | (4u + j);
    }
    __syncthreads();

    // this warp serves page r = (kv, head) of the live units g0, g0 + gstep, ...; the host sizes the grid
    // so that the number of warps is a multiple of 2*H
    const uint32_t n_units = s_cnt[a.B];
    const uint32_t n_warps = gridDim.x * kPfWarps, gw = blockIdx.x * kPfWarps + warp;
    const uint32_t r = gw % twoH, gstep = n_warps / twoH, g0 = gw / twoH;
    const uint32_t n_mine = g0 < n_units ? (n_units - g0 + gstep - 1u) / gstep : 0u;
    uint32_t n_issued = 0, n_consumed = 0;
    uint8_t *my_rec = s_rec + warp * 2 * kRecStage;
    const uint32_t my_bar = smem_u32(s_bar + warp * 2);
    const unsigned long long layer_slot0 = (unsigned long long)a.layer * a.blocks_per_layer * twoH + r;
    unsigned long long st_pages = 0;

    for (uint32_t first = 0; first < n_mine; first += 32u) {
        // ---- translation: lane l owns page first + l of this warp
        uint4 *dst = nullptr;
        unsigned long long pte = 0ull;
        uint32_t index = 0;
        int state = 0;               // 0 = nothing to deliver, 3 = packed record, 4 = raw record
        if (first + lane < n_mine) {
            const uint32_t u = s_unit[g0 + (first + lane) * gstep];
            const uint32_t block = u >> 12, b = (u >> 3) & 511u, i = u & 7u;
            if (i < 4u) {
                index = (b * 4u + i) * twoH + r;
                dst = a.miss_dst + ((size_t)(b * 4u + i) * twoH + r) * (kPageBytes / 16);
            } else {
                index = ((a.B + b) * 4u + (i - 4u)) * twoH + r;
                dst = a.l2 + ((((size_t)back * a.max_seqs + b) * 4u + (i - 4u)) * twoH + r) * (kPageBytes / 16);
            }
            const int32_t bt_val = __ldg(a.block_table + (size_t)b * a.max_blocks_per_seq + block);
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
        // ---- delivery, in page order
        uint32_t live = __ballot_sync(kFull, state != 0);
        const uint32_t packed = __ballot_sync(kFull, state == 3);
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
                    bulk_g2s(smem_u32(my_rec + buf * kRecStage), a.pool + (ne & 0xFFFFFFFFull) * kGranule, bytes, bar);
                }
                ++n_issued;
            }
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
                const uint8_t *rec = my_rec + buf * kRecStage;
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
            st_pages += 1;
        }
    }
    if (lane == 0 && st_pages) {
        atomicAdd(reinterpret_cast<unsigned long long *>(&a.cnt->pages), st_pages);
        atomicAdd(&a.ctl->stats[kStDecoded], st_pages);
    }
}

static size_t pf_fetch_smem(uint32_t B)
{
    return (size_t)kPfWarps * 2 * kRecStage + 256 * 16 + kPfWarps * 2 * 8 + ((size_t)B + 1) * 4 + (size_t)B * kPfUnits * 4;
}

cudaError_t launch_prefetch_step(const PrefetchArgs &a, int n_sm, cudaStream_t stream)
{
    pf_plan_kernel<<<(a.B + 7u) / 8u, 32, 0, stream>>>(a);   // one warp = eight sequences
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t smem = pf_fetch_smem(a.B);
    if (smem > 48u * 1024u) {
        e = cudaFuncSetAttribute(pf_fetch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pf_fetch_smem(kPfMaxSeqs));
        if (e != cudaSuccess) return e;
    }
    // a warp count that is a multiple of 2*H (every warp keeps one (kv, head)), and no more CTAs than
    // the largest possible number of transfers can occupy
    const uint32_t twoH = 2u * a.H;
    uint32_t m = twoH, x = kPfWarps;
    while (x) { uint32_t t = m % x; m = x; x = t; }          // m = gcd(twoH, kPfWarps)
    const uint32_t mult = twoH / m;
    const unsigned long long max_pages = (unsigned long long)a.B * kPfUnits * twoH;
    unsigned long long want = (max_pages + kPfWarps - 1) / kPfWarps;
    uint32_t grid = (uint32_t)n_sm * 3u;
    if (want < grid) grid = (uint32_t)want;
    grid = grid >= mult ? grid - grid % mult : mult;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kPfThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in both kernels
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, pf_fetch_kernel, a);
}

uint32_t prefetch_max_seqs() { return kPfMaxSeqs; }

}  // namespace speckv
