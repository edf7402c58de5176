// speckv_compress: Algorithm "KV-Cache Compression" of CXL-SpecKV on sm_100a.
//
// A CTA is kEnc encoder warps, a loader warp and a scanner warp, and works on tiles of kEnc pages
// (tile numbers are tickets from an atomic counter, so a tile's predecessors are always in progress).
//   loader warp  : draws the ticket, reads the tile's list entries, starts bulk-async loads of its
//                  pages into shared memory (mbarrier completion); paced only by the encoders
//                  releasing page buffers.
//   encoder warp : one 16x128 fp16 page per tile.  Lane l holds, for k = 0..7, the 8 consecutive
//                  elements at flat index 256*k + 8*l (token row 2*k + l/16, channels 8*(l%16)...).
//                  scale -> quantise (page buffer released) -> delta -> run heads -> value
//                  compaction, record staged in shared memory.
//   scanner warp : once a tile is encoded, its place in the log = exclusive prefix sum of record
//                  sizes in list order, from a single-pass chained scan over tiles (decoupled
//                  look-back over 64 tiles per poll, bounded polling); then bulk-async stores of
//                  the staged records, page-table entries, counters.
// One page buffer per encoder (released as soon as the page is in registers) and three record
// stages: encoders wait for the scan only when they are three tiles ahead of it.  One CTA of 20
// encoders per SM fills the SM's shared memory (80 KiB of page buffers + 139 KiB of record stages);
// measured against 2 CTAs x 8 encoders x 4 stages it is 5 % faster (five encoder warps per
// scheduler instead of four, two control warps per SM instead of four), and the number of
// stages matters more than anything else (two stages: -11 %).
#include <mutex>

#include "async_ptx.cuh"
#include "speckv_dev.cuh"

namespace speckv {

constexpr int kEnc = 20;                                  // encoder warps = pages per tile
constexpr int kCThreads = (kEnc + 2) * 32;
constexpr uint32_t kRing = 8;                             // tiles described in the loader -> scanner ring
constexpr uint32_t kLutBytes = 256 * 16;

constexpr uint32_t kRecStages = 3;                         // tiles the encoders may run ahead of the scan
constexpr uint32_t kRecSlot = 2368;                        // bytes per staged record (largest packed record, padded)

// dynamic shared memory layout
constexpr uint32_t kOffIn = 0;                                            // [kEnc][4096]  one page buffer per encoder
constexpr uint32_t kOffRec = kOffIn + kEnc * kPageBytes;                  // [kRecStages][kEnc][kRecSlot] records
constexpr uint32_t kOffLut = kOffRec + kRecStages * kEnc * kRecSlot;      // [256] uint4 compaction table
constexpr uint32_t kOffMeta = kOffLut + kLutBytes;                        // [kRecStages][kEnc] uint4 {rec_len, mode, n_runs, gran}
constexpr uint32_t kOffConst = kOffMeta + kRecStages * kEnc * 16;         // 64 B: raw-record header + 48 zero bytes
constexpr uint32_t kOffInfo = kOffConst + 64;                             // [kEnc] valid flags, done flag, tile id, [kRecStages] size accumulators
constexpr uint32_t kInfoWords = kEnc + 2 + kRecStages;
constexpr uint32_t kOffRing = kOffInfo + kInfoWords * 4;                  // [kRing] {tile, pad, i[kEnc], slot[kEnc]} u32
constexpr uint32_t kRingWords = 2 * kEnc + 2;
constexpr uint32_t kOffBar = (kOffRing + kRing * kRingWords * 4 + 7) & ~7u;   // mbarriers
constexpr uint32_t kBarInFull = 0;                                        // [kEnc]        loader  -> encoder
constexpr uint32_t kBarInEmpty = kEnc;                                    // [1]           encoder -> loader
constexpr uint32_t kBarEncDone = kEnc + 1;                                // [kRecStages]  encoder -> scanner
constexpr uint32_t kBarRecFree = kEnc + 1 + kRecStages;                   // [kRecStages]  scanner -> encoder
constexpr uint32_t kNumBars = kEnc + 1 + 2 * kRecStages;
constexpr uint32_t kOffAbort = kOffBar + kNumBars * 8;
constexpr uint32_t kCompressSmem = kOffAbort + 16;
static_assert(kCompressSmem + 1024 <= 233472, "one CTA per SM");

// Compaction table entry for a run-head mask m.  The j-th head byte comes from symbol position >= j, so the
// output bytes 4-7 only ever come from the second word: x = PRMT selector over (q0, q1) for output bytes 0-3,
// y = PRMT selector over (q1, zero) for output bytes 4-7 with the unused positions pointing at the zero word,
// z = byte mask keeping the first min(popcount(m), 4) bytes of the low word (w unused).
__device__ __forceinline__ uint4 lut_entry(uint32_t m)
{
    const uint32_t c = __popc(m);
    const uint32_t keep_lo = c >= 4 ? 0xFFFFFFFFu : ((1u << (8 * c)) - 1u);
    const uint32_t sel = compact_sel(m);
    uint32_t y = 0;
    for (uint32_t j = 4; j < 8; ++j) {
        const uint32_t pos = (sel >> (4 * j)) & 15u;                  // symbol position of head j (4..7) if j < c
        y |= (j < c ? pos - 4u : 4u) << (4 * (j - 4));                // 4 = first byte of the zero word
    }
    return make_uint4(sel & 0xFFFFu, y, keep_lo, 0u);
}

// two fused multiply-adds a*b + c on packed binary32 pairs (one rounding each)
__device__ __forceinline__ void fma_x2(float a0, float a1, unsigned long long B, unsigned long long C, float &r0, float &r1)
{
    unsigned long long A, T;
    asm("mov.b64 %0, {%1, %2};" : "=l"(A) : "f"(a0), "f"(a1));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(T) : "l"(A), "l"(B), "l"(C));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(r0), "=f"(r1) : "l"(T));
}

// packs the low bytes of four words
__device__ __forceinline__ uint32_t pack4(uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3)
{
    return __byte_perm(__byte_perm(r0, r1, 0x0040), __byte_perm(r2, r3, 0x0040), 0x5410);
}

// Quantise 8 halves: r[e] = bit pattern of fma(x_e, inv, 1.5 * 2^23) = 0x4B400000 + q_e, where
// q_e = round-half-even of the exact product x_e * inv (two's complement in the low bits).
__device__ __forceinline__ void quant8(const uint4 &v, unsigned long long inv2, unsigned long long magic2, uint32_t (&r)[8])
{
    const uint32_t h[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&h[i]));
        float r0, r1;
        fma_x2(a.x, a.y, inv2, magic2, r0, r1);
        r[2 * i] = __float_as_uint(r0);
        r[2 * i + 1] = __float_as_uint(r1);
    }
}

// per binary16 half: the larger magnitude of a and b (the sign bit of the result is not meaningful);
// a NaN in either gives the NaN pattern 0x7FFF
__device__ __forceinline__ uint32_t absmax2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.NaN.xorsign.abs.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// OR into a 32-bit word of shared memory (no return value)
__device__ __forceinline__ void smem_or(uint32_t addr, uint32_t v)
{
    asm volatile("red.shared.or.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// ---------------------------------------------------------------- encoder warp: one page

// Reads the page from `in` (shared memory), builds the record in `rec` (shared memory, filled by
// this warp only) and returns {rec_len, mode, n_runs, granules}.  `scheme` is the scheme without
// the SPECKV_GROUPED flag; with `grouped`, the lanes l and l + 16, which hold the same 8 channels of
// all 16 token rows, share a scale of their own and the 16 maxima precede the payload.  Calls release_in() once the
// page has been copied to registers (not for a bypassed page, whose buffer is the payload),
// and wait_rec() before its first write to `rec` (the buffer may still be read by bulk stores).
template <class Release, class WaitRec>
__device__ __forceinline__ uint4 encode_page(const uint4 *in, int scheme, bool grouped, uint8_t *rec, const uint4 *lut,
                                             uint32_t lane, Release release_in, WaitRec wait_rec)
{
    // ---- scale: max |x| over the page (half-precision maximum of magnitudes: exact, subnormals
    // kept, NaN propagated).  Across lanes |x| is compared as an unsigned 16-bit integer, which
    // orders like |x| with the Inf and NaN patterns on top
    uint32_t ma = 0, mb = 0;
    uint4 x[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint4 v = x[k] = in[k * 32 + lane];
        ma = absmax2(absmax2(ma, v.x), v.z);
        mb = absmax2(absmax2(mb, v.y), v.w);
    }
    uint32_t mi = absmax2(ma, mb) & 0x7FFF7FFFu;
    mi = max(mi & 0xFFFFu, mi >> 16);
    const uint32_t amax_bits = __reduce_max_sync(kFull, mi);
    const __half mh = __ushort_as_half((unsigned short)amax_bits);
    if (scheme == SPECKV_RAW || amax_bits >= 0x7C00u)       // bypass: the page buffer itself is the payload
        return make_uint4(kHdrBytes + kPageBytes, SPECKV_RAW, 0u, (kHdrBytes + kPageBytes + kGranule - 1u) / kGranule);
    release_in();                                           // the page now lives in registers
    const float amax = __half2float(mh);
    float s = 0.0f, inv = 0.0f;
    if (amax_bits != 0) {
        s = __fdiv_rn(amax, 127.0f);
        inv = __fdiv_rn(127.0f, amax);
    }
    uint32_t gmax = 0;                                      // grouped: largest |x| of this lane's 8 channels
    if (grouped) {
        gmax = max(mi, __shfl_xor_sync(kFull, mi, 16));
        inv = gmax ? __fdiv_rn(127.0f, __half2float(__ushort_as_half((unsigned short)gmax))) : 0.0f;
        rec += kGroupBytes;                                 // the payload moves back by the table of maxima
    }
    const uint32_t grp = grouped ? kGroupBytes : 0u;
    unsigned long long inv2, magic2;
    asm("mov.b64 %0, {%1, %1};" : "=l"(inv2) : "f"(inv));
    asm("mov.b64 %0, {%1, %1};" : "=l"(magic2) : "f"(kMagic));

    // ---- quantise (+ delta along the channel axis, restarting at channel 0 of every token row):
    // q[k][0] = elements 0-3, q[k][1] = elements 4-7 of this lane's group k.  The delta is taken
    // on the magic-float bit patterns, whose difference is the difference of the quantised values.
    uint32_t q[8][2];
    uint2 *pay = reinterpret_cast<uint2 *>(rec + kHdrBytes);
    uint32_t payload_len = kPageElems, n_runs = 0, mode = (uint32_t)scheme;
    if (scheme == SPECKV_INT8) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t r[8];
            quant8(x[k], inv2, magic2, r);
            q[k][0] = pack4(r[0], r[1], r[2], r[3]);
            q[k][1] = pack4(r[4], r[5], r[6], r[7]);
        }
        wait_rec();
        if (lane < 3u - grp / 16u) reinterpret_cast<uint4 *>(rec + kHdrBytes + kPageElems)[lane] = make_uint4(0u, 0u, 0u, 0u);   // padding
#pragma unroll
        for (int k = 0; k < 8; ++k) pay[k * 32 + lane] = make_uint2(q[k][0], q[k][1]);
    } else {
        const bool row_start = (lane & 15u) == 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t r[8];
            quant8(x[k], inv2, magic2, r);
            const uint32_t up = __shfl_up_sync(kFull, r[7], 1);
            const uint32_t prev = row_start ? __float_as_uint(kMagic) : up;
            q[k][0] = pack4(r[0] - prev, r[1] - r[0], r[2] - r[1], r[3] - r[2]);
            q[k][1] = pack4(r[4] - r[3], r[5] - r[4], r[6] - r[5], r[7] - r[6]);
        }
        // ---- run heads: symbol differs from its predecessor in the flat stream
        bool rle = scheme != SPECKV_INT8_DELTA;
        uint32_t mk[8];
        if (rle) {
            uint32_t carry = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                uint32_t rot = __shfl_sync(kFull, q[k][1], (lane + 31u) & 31u);
                uint32_t pw = lane ? rot : carry;   // lane 0: the previous group row's last word (of lane 31)
                carry = rot;
                uint32_t p0 = __byte_perm(pw, q[k][0], 0x6543);   // predecessor symbols of elements 0-3
                uint32_t p1 = __funnelshift_l(q[k][0], q[k][1], 8);
                // bit 7 of every differing byte, weighted 1,2,4,..,128 per element, all times 128
                mk[k] = __dp4a(nz4(q[k][1] ^ p1), 0x80402010u, __dp4a(nz4(q[k][0] ^ p0), 0x08040201u, 0u)) >> 7;
            }
            if (lane == 0) mk[0] |= 1u;             // symbol 0 always starts a run
            if (scheme == SPECKV_AUTO) {
                // adaptive selection: keep the run-length stage only if bitmap + run values are
                // smaller than the 2,048-byte delta stream (equal size: the simpler mode)
                uint32_t heads = 0;
#pragma unroll
                for (int k = 0; k < 8; ++k) heads += __popc(mk[k]);
                rle = __reduce_add_sync(kFull, heads) < kPageElems - kBitmapBytes;
            }
        }
        if (!rle) {
            mode = SPECKV_INT8_DELTA;
            wait_rec();
            if (lane < 3u - grp / 16u) reinterpret_cast<uint4 *>(rec + kHdrBytes + kPageElems)[lane] = make_uint4(0u, 0u, 0u, 0u);   // padding
#pragma unroll
            for (int k = 0; k < 8; ++k) pay[k * 32 + lane] = make_uint2(q[k][0], q[k][1]);
        } else {
            mode = SPECKV_INT8_DELTA_RLE;
            // (first, so that these stores are under way while the scan below waits for its shuffles)
            wait_rec();
            // zero the value area and the padding (values are OR-ed in), store the bitmap
            {
                uint4 *z = reinterpret_cast<uint4 *>(rec + kValuesOff);
                constexpr uint32_t n16max = (kRecSlot - kValuesOff) / 16;
                const uint32_t n16 = n16max - grp / 16u;     // up to the end of this warp's staging slot
#pragma unroll
                for (uint32_t jj = 0; jj < (n16max + 31u) / 32u; ++jj)
                    if (jj * 32u + lane < n16) z[jj * 32u + lane] = make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) rec[kHdrBytes + k * 32 + lane] = (uint8_t)mk[k];
            // ---- offset of each group's run values: exclusive prefix sum of the popcounts in (k, lane)
            // order.  Within a group row the exclusive sums stay below 8 * 31 = 248, so four rows share a
            // word as byte fields and nothing carries between them; the row totals (up to 256) are warp
            // reductions, and the rows' bases accumulate from them.
            uint32_t c[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) c[k] = __popc(mk[k]);
            uint32_t ea = scan_excl_bytes(c[0] + (c[1] << 8) + (c[2] << 16) + (c[3] << 24));
            uint32_t eb = scan_excl_bytes(c[4] + (c[5] << 8) + (c[6] << 16) + (c[7] << 24));
            uint32_t excl[8], tot[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                excl[k] = __byte_perm(k < 4 ? ea : eb, 0u, 0x4440 + (k & 3));
                tot[k] = __reduce_add_sync(kFull, c[k]);
            }
            __syncwarp();
            // ---- compaction: head bytes moved to the front of the group (PRMT), shifted to the byte
            // offset inside their words, OR-ed into the staged value stream
            const uint32_t vals = smem_u32(rec + kValuesOff);
            uint32_t base = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t o = base + excl[k];
                const uint4 e = lut[mk[k]];
                const uint32_t lo = __byte_perm(q[k][0], q[k][1], e.x) & e.z;        // PRMT reads 16 selector bits
                const uint32_t hi = __byte_perm(q[k][1], 0u, e.y);
                const uint32_t sh = o << 3;          // funnel shifts use the low 5 bits: 8 * (o & 3)
                const uint32_t w0 = __funnelshift_l(0u, lo, sh), w1 = __funnelshift_l(lo, hi, sh), w2 = __funnelshift_l(hi, 0u, sh);
                const uint32_t p = vals + (o & ~3u);
                smem_or(p, w0); smem_or(p + 4, w1);
                smem_or(p + 8, w2);
                base += tot[k];
            }
            n_runs = base;
            payload_len = kBitmapBytes + base;
        }
    }
    if (grouped) {
        rec -= kGroupBytes;
        payload_len += kGroupBytes;
        mode |= SPECKV_GROUPED;
        if (lane < 16) reinterpret_cast<uint16_t *>(rec + kHdrBytes)[lane] = (uint16_t)gmax;
    }
    const uint32_t rec_len = kHdrBytes + payload_len;
    if (lane == 0)
        *reinterpret_cast<uint4 *>(rec) = make_uint4(__float_as_uint(s), payload_len | (mode << 16) | (kVersion << 24),
                                                     n_runs | (amax_bits << 16), 0u);
    return make_uint4(rec_len, mode, n_runs, (rec_len + kGranule - 1u) / kGranule);
}

// ---------------------------------------------------------------- control warp: chained scan

constexpr int kLook = 2;   // groups of 32 tiles inspected per look-back step (64 tiles)

// Exclusive prefix (in granules, from the start of the pool) of tile `tile`, whose own total
// `agg` its encoders have already published.  Publishes the tile's inclusive prefix.  Returns
// false if a wait gave up or a predecessor failed (the failure is passed on to later tiles).
//
// Group m, lane l looks at tile look - (32*m + l), i.e. at distance 32*m + l: one coalesced
// 256-byte read per group, all groups at once (one round trip).  Only words nearer than the
// nearest prefix seen so far matter; while some of those are unpublished, only they are read
// again, with a pause in between, so that many waiting CTAs neither hammer the cache lines that
// the publishers are writing nor eat the encoders' issue slots.
__device__ __forceinline__ bool tile_base(const CompressArgs &a, uint32_t tile, unsigned long long agg, uint32_t lane,
                                          unsigned long long &base)
{
    volatile unsigned long long *ts = a.scan->tile;
    if (tile == 0) {
        base = *reinterpret_cast<volatile unsigned long long *>(&a.ctl->cursor64);
        if (lane == 0) ts[0] = kFlagPrefix | (base + agg);
        return true;
    }
    base = 0;
    bool fail = false;
    long long look = (long long)tile - 1;
    for (;;) {
        unsigned long long v[kLook];
#pragma unroll
        for (int m = 0; m < kLook; ++m) v[m] = 0ull;
        uint32_t stop = 32u * kLook;                 // distance of the nearest prefix / failed tile seen so far
        uint32_t spins = 0;
        for (;;) {
            uint32_t my_stop = 32u * kLook;
#pragma unroll
            for (int m = 0; m < kLook; ++m) {
                const uint32_t dist = 32u * m + lane;
                if ((v[m] & kFlagMask) == 0ull && dist < stop) {
                    const long long idx = look - (long long)dist;
                    v[m] = idx >= 0 ? (unsigned long long)ts[idx] : (2ull << 62);   // before tile 0: an empty prefix
                }
                const unsigned long long f = v[m] & kFlagMask;
                if (f >= kFlagPrefix) my_stop = min(my_stop, dist);                  // prefix or failure
            }
            stop = min(stop, __reduce_min_sync(kFull, my_stop));
            // words beyond the (possibly nearer) stop no longer matter
            bool still = false;
#pragma unroll
            for (int m = 0; m < kLook; ++m) still = still || ((v[m] & kFlagMask) == 0ull && 32u * m + lane < stop);
            if (!__any_sync(kFull, still)) break;
            if (++spins >= a.spin_limit) { fail = true; break; }
            __nanosleep(200);
        }
        if (fail) break;
        unsigned long long sum = 0;
        uint32_t stop_flag = 0;
#pragma unroll
        for (int m = 0; m < kLook; ++m) {
            const uint32_t dist = 32u * m + lane;
            if (dist <= stop) sum += v[m] & ~kFlagMask;
            if (dist == stop) stop_flag = (uint32_t)(v[m] >> 62);
        }
        if (stop < 32u * kLook && __reduce_max_sync(kFull, stop_flag) == 3u) { fail = true; break; }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) sum += __shfl_xor_sync(kFull, sum, d);
        base += sum;
        if (stop < 32u * kLook) break;
        look -= 32 * kLook;
    }
    if (lane == 0) ts[tile] = fail ? kFlagFail : (kFlagPrefix | (base + agg));
    return !fail;
}

__global__ void __launch_bounds__(kCThreads, 1) compress_kernel(CompressArgs a)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t tid = threadIdx.x, lane = tid & 31u;
    const uint32_t warp = __shfl_sync(kFull, tid >> 5, 0);
    uint4 *s_lut = reinterpret_cast<uint4 *>(smem + kOffLut);
    uint4 *s_meta = reinterpret_cast<uint4 *>(smem + kOffMeta);
    volatile uint32_t *s_info = reinterpret_cast<volatile uint32_t *>(smem + kOffInfo);   // [kInfoWords]
    volatile uint32_t *s_ring = reinterpret_cast<volatile uint32_t *>(smem + kOffRing);   // [kRing][kRingWords]
    volatile int *s_abort = reinterpret_cast<volatile int *>(smem + kOffAbort);
    const uint32_t bars = smem_u32(smem + kOffBar);
    auto bar_in_full = [&](uint32_t w) { return bars + 8u * (kBarInFull + w); };
    const uint32_t bar_in_empty = bars + 8u * kBarInEmpty;
    auto bar_enc_done = [&](uint32_t rs) { return bars + 8u * (kBarEncDone + rs); };
    auto bar_rec_free = [&](uint32_t rs) { return bars + 8u * (kBarRecFree + rs); };
    auto give_up = [&](uint32_t where) {
        if (lane == 0 && !*s_abort) { *s_abort = 1; raise_status(a.ctl, SPECKV_ST_TIMEOUT, where); }
    };

    if (tid < 256) s_lut[tid] = lut_entry(tid);
    if (tid < 4) reinterpret_cast<uint4 *>(smem + kOffConst)[tid] =
        tid == 0 ? make_uint4(0u, kPageBytes | (kVersion << 24), 0u, 0u) : make_uint4(0u, 0u, 0u, 0u);
    if (tid == 0) {
        for (uint32_t w = 0; w < kEnc; ++w) mbar_init(bar_in_full(w), 1);
        mbar_init(bar_in_empty, kEnc);
        for (uint32_t rs = 0; rs < kRecStages; ++rs) {
            mbar_init(bar_enc_done(rs), kEnc);
            mbar_init(bar_rec_free(rs), 1);
            s_info[kEnc + 2 + rs] = 0;
        }
        *s_abort = 0;
        mbar_init_fence();
    }
    fence_async_smem();                     // constants are read by bulk stores
    __syncthreads();

    if (warp < kEnc) {
        // ================================================= encoder warp
        const uint4 *in = reinterpret_cast<const uint4 *>(smem + kOffIn) + warp * (kPageBytes / 16);
        for (uint32_t j = 0;; ++j) {
            const uint32_t rs = j % kRecStages, rpar = (j / kRecStages) & 1u;
            if (!mbar_wait_warp(bar_in_full(warp), j & 1u, s_abort, a.wait_ns)) { give_up(0xFFFFFFF0u); return; }
            // read now: the loader reuses these words as soon as the page buffers are released
            const bool done = s_info[kEnc] != 0u, live = s_info[warp] != 0u;
            const uint32_t tile = s_info[kEnc + 1];
            uint4 meta = make_uint4(0u, 0u, 0u, 0u);
            bool dead = false, released = false, owned = false;
            auto release_in = [&]() {
                released = true;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_in_empty);
            };
            auto wait_rec = [&]() {
                owned = true;
                if (!mbar_wait_warp(bar_rec_free(rs), rpar ^ 1u, s_abort, a.wait_ns)) dead = true;
            };
            if (!done && live)
                meta = encode_page(in, a.scheme & ~SPECKV_GROUPED, (a.scheme & SPECKV_GROUPED) != 0,
                                   smem + kOffRec + (rs * kEnc + warp) * kRecSlot, s_lut, lane, release_in, wait_rec);
            // A bypassed page, an absent page and the closing iteration build no record, but they do write the
            // stage's description and size accumulator below: the stage must be theirs first, or a scanner that
            // is a full ring of stages behind would read this tile's words in place of its own.
            if (!owned) wait_rec();
            if (dead) { give_up(0xFFFFFFF1u); return; }
            if (!released && meta.x == 0u) release_in();            // nothing was loaded for this warp
            fence_async_smem();                                     // record bytes -> visible to the bulk stores
            __syncwarp();
            if (lane == 0) {
                s_meta[rs * kEnc + warp] = meta;
                // the last encoder of a tile publishes the tile's size right away: other tiles' scans
                // then depend on encoding progress only (tile 0 is published by the scanner, as a prefix)
                uint32_t *acc = const_cast<uint32_t *>(s_info) + kEnc + 2 + rs;
                const uint32_t old = atomicAdd(acc, meta.w | (1u << 16));
                if ((old >> 16) == kEnc - 1u) {
                    *acc = 0u;
                    if (!done && tile != 0u)
                        *reinterpret_cast<volatile unsigned long long *>(&a.scan->tile[tile]) = kFlagAgg | ((old & 0xFFFFu) + meta.w);
                }
                mbar_arrive(bar_enc_done(rs));
            }
            if (done) return;
        }
    }

    if (warp == kEnc) {
        // ================================================= loader warp
        // One tile ahead: while the encoders still hold their page buffers, the ticket and the list
        // entries of the tile after are fetched and its pages are requested into L2, so that the copies
        // into shared memory, which can only start when the buffers are free, find them there.
        uint32_t n_tile = 0, n_i = 0, n_sp = 0, n_slot = 0xFFFFFFFFu;
        bool n_done = false, n_valid = false;
        auto draw = [&]() {
            uint32_t t = lane == 0 ? atomicAdd(&a.scan->ticket, 1u) : 0u;
            n_tile = __shfl_sync(kFull, t, 0) + a.ticket0;
            n_done = n_tile >= a.n_tiles;
            n_i = n_tile * kEnc + lane;
            n_sp = 0; n_slot = 0xFFFFFFFFu; n_valid = false;
            if (lane < kEnc && !n_done && n_i < a.n) {
                n_sp = a.src_page[n_i];
                n_slot = a.dst_slot[n_i];
                n_valid = n_sp < a.n_src_pages && n_slot < a.n_slots;
                if (!n_valid) { raise_status(a.ctl, SPECKV_ST_BAD_INDEX, n_i); n_slot = 0xFFFFFFFFu; }
                else prefetch_l2(a.src + (size_t)n_sp * (kPageBytes / 16), kPageBytes);
            }
        };
        draw();
        for (uint32_t j = 0;; ++j) {
            const uint32_t tile = n_tile, i = n_i, sp = n_sp, slot = n_slot;
            const bool done = n_done, valid = n_valid;
            if (!done) draw();
            if (!mbar_wait_warp(bar_in_empty, (j & 1u) ^ 1u, s_abort, a.wait_ns)) {                                 // page buffers are free
                give_up(0xFFFFFFF2u);
                // giving up: the previous tile's loads may still be in flight towards this CTA's shared
                // memory; stay (bounded) until they have landed, so that the memory outlives them
                if (j > 0 && lane < kEnc) mbar_wait(bar_in_full(lane), (j - 1u) & 1u, nullptr, a.wait_ns);
                return;
            }
            if (lane < kEnc) {
                volatile uint32_t *r = s_ring + (j % kRing) * kRingWords;
                if (lane == 0) r[0] = tile;
                r[2 + lane] = i;
                r[2 + kEnc + lane] = slot;                          // 0xFFFFFFFF = no page
                s_info[lane] = valid ? 1u : 0u;
                if (lane == 0) { s_info[kEnc] = done ? 1u : 0u; s_info[kEnc + 1] = tile; }
                __syncwarp((1u << kEnc) - 1u);
                const uint32_t bar = bar_in_full(lane);
                if (valid) {
                    mbar_expect_tx(bar, kPageBytes);
                    bulk_g2s(smem_u32(smem + kOffIn + lane * kPageBytes), a.src + (size_t)sp * (kPageBytes / 16), kPageBytes, bar);
                } else {
                    mbar_arrive(bar);                                // nothing to load: complete the phase
                }
            }
            __syncwarp();
            if (done) return;
        }
    }

    // ===================================================== scanner warp
    unsigned long long st_gran = 0, st_payload = 0, st_runs = 0, st_nonfinite = 0, st_m0 = 0, st_m1 = 0, st_m2 = 0, st_m3 = 0;
    bool chain_ok = true;
    for (uint32_t j = 0;; ++j) {
        const uint32_t rs = j % kRecStages, rpar = (j / kRecStages) & 1u;
        if (!mbar_wait_warp(bar_enc_done(rs), rpar, s_abort, a.wait_ns)) { give_up(0xFFFFFFF3u); break; }
        volatile uint32_t *r = s_ring + (j % kRing) * kRingWords;
        const uint32_t tile = r[0];
        if (tile >= a.n_tiles) break;                                // the loader ran out of tiles
        uint4 meta = make_uint4(0u, 0u, 0u, 0u);
        uint32_t page_i = 0, slot = 0xFFFFFFFFu;
        if (lane < kEnc) { meta = s_meta[rs * kEnc + lane]; page_i = r[2 + lane]; slot = r[2 + kEnc + lane]; }
        const uint32_t gran = meta.w;
        uint32_t incl = gran;
#pragma unroll
        for (int d = 1; d < kEnc; d <<= 1) {
            uint32_t t = __shfl_up_sync(kFull, incl, d);
            if (lane >= (uint32_t)d) incl += t;
        }
        const unsigned long long agg = __shfl_sync(kFull, incl, kEnc - 1);
        unsigned long long base = 0;
        if (chain_ok) {
            chain_ok = tile_base(a, tile, agg, lane, base);
            if (!chain_ok && lane == 0) raise_status(a.ctl, SPECKV_ST_TIMEOUT, tile * kEnc);
        } else if (lane == 0) {
            a.scan->tile[tile] = kFlagFail;                          // keep later tiles from waiting
        }
        const bool raw = lane < kEnc && slot != 0xFFFFFFFFu && meta.y == SPECKV_RAW;
        if (chain_ok) {
            if (lane == 0 && tile == a.n_tiles - 1) a.ctl->cursor64 = base + agg;
            if (lane < kEnc && slot != 0xFFFFFFFFu) {
                const unsigned long long off64 = base + incl - gran;
                if (off64 + gran > a.pool_gran) {
                    raise_status(a.ctl, SPECKV_ST_POOL_FULL, page_i);
                } else {
                    uint8_t *dst = a.pool + off64 * kGranule;
                    if (raw) {                                       // header | page | zero padding
                        bulk_s2g(dst, smem_u32(smem + kOffConst), 16);
                        bulk_s2g(dst + 16, smem_u32(smem + kOffIn + lane * kPageBytes), kPageBytes);
                        bulk_s2g(dst + 16 + kPageBytes, smem_u32(smem + kOffConst + 16), 48);
                        st_m0 += 1;
                        if ((a.scheme & ~SPECKV_GROUPED) != SPECKV_RAW) st_nonfinite += 1;
                    } else {
                        bulk_s2g(dst, smem_u32(smem + kOffRec + (rs * kEnc + lane) * kRecSlot), gran * kGranule);
                        const uint32_t m = meta.y & 3u;             // grouped records count under their base mode
                        if (m == 1u) st_m1 += 1; else if (m == 2u) st_m2 += 1; else st_m3 += 1;
                    }
                    a.pte[slot] = off64 | ((unsigned long long)meta.x << 32) | ((unsigned long long)meta.y << 48) | kPteValid;
                    st_gran += gran; st_payload += meta.x - kHdrBytes; st_runs += meta.z;
                }
            }
        }
        bulk_commit();
        bulk_wait_read();                                            // stage buffers may be overwritten from here on
        if (raw) mbar_arrive(bar_in_empty);                          // a bypassed page's buffer was the payload
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_rec_free(rs));
    }
    bulk_wait_all();
    // counters: one atomic per counter and CTA
    unsigned long long *cnt[8] = {&st_m0, &st_m1, &st_m2, &st_m3, &st_gran, &st_payload, &st_runs, &st_nonfinite};
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        unsigned long long v = *cnt[c];
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
        if (lane == 0 && v) atomicAdd(&a.ctl->stats[c], v);
    }
}

// ---------------------------------------------------------------- scheme SPECKV_RAW: the bypass as a copy
//
// A call with scheme SPECKV_RAW stores every page as it is (the uncompressed share of the traffic, which
// the paper's engine lets bypass the pipeline).  Every record has the same size, so a tile's size is
// known as soon as its list entries have been read, long before its pages arrive: the chained scan runs
// ahead of the data and a page leaves for the pool the moment it has landed.  No encoder, no record
// staging: each of kRawWarps warps owns kRawTile page buffers and takes whole tiles of kRawTile pages
// (ticket order, as above).  Lane l < kRawTile of a warp handles page l of the tile with bulk copies of
// its own: global -> its buffer (mbarrier), then header | page | zero padding -> pool.
constexpr int kRawWarps = 3;
constexpr uint32_t kRawTile = 16;                                         // pages per tile and per warp
constexpr uint32_t kRawGran = (kHdrBytes + kPageBytes + kGranule - 1u) / kGranule;   // 65 granules per record
constexpr uint32_t kRawOffConst = kRawWarps * kRawTile * kPageBytes;      // 64 B: raw-record header + 48 zero bytes
constexpr uint32_t kRawOffBar = kRawOffConst + 64;                        // [kRawWarps][kRawTile] mbarriers
constexpr uint32_t kRawSmem = kRawOffBar + kRawWarps * kRawTile * 8;
static_assert(kRawSmem + 1024 <= 233472, "one CTA per SM");

__global__ void __launch_bounds__(kRawWarps * 32, 1) raw_copy_kernel(CompressArgs a)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const uint32_t tid = threadIdx.x, lane = tid & 31u;
    const uint32_t warp = __shfl_sync(kFull, tid >> 5, 0);
    if (tid < 4) reinterpret_cast<uint4 *>(smem + kRawOffConst)[tid] =
        tid == 0 ? make_uint4(0u, kPageBytes | (kVersion << 24), 0u, 0u) : make_uint4(0u, 0u, 0u, 0u);
    if (tid < kRawWarps * kRawTile) mbar_init(smem_u32(smem + kRawOffBar) + 8u * tid, 1);
    mbar_init_fence();
    fence_async_smem();                     // the constants are read by bulk stores
    __syncthreads();

    const uint32_t my_buf = smem_u32(smem + (warp * kRawTile + lane) * kPageBytes);     // lanes < kRawTile only
    const uint32_t my_bar = smem_u32(smem + kRawOffBar) + 8u * (warp * kRawTile + lane);
    const uint32_t hdr = smem_u32(smem + kRawOffConst);
    unsigned long long st_pages = 0;
    uint32_t phase = 0;                     // loads this lane has waited for: its barrier's parity
    bool chain_ok = true, in_flight = false;
    for (;;) {
        uint32_t t = lane == 0 ? atomicAdd(&a.scan->ticket, 1u) : 0u;
        const uint32_t tile = __shfl_sync(kFull, t, 0) + a.ticket0;
        if (tile >= a.n_tiles) break;
        const uint32_t i = tile * kRawTile + lane;
        uint32_t sp = 0, slot = 0;
        bool valid = false;
        if (lane < kRawTile && i < a.n) {
            sp = a.src_page[i];
            slot = a.dst_slot[i];
            valid = sp < a.n_src_pages && slot < a.n_slots;
            if (!valid) raise_status(a.ctl, SPECKV_ST_BAD_INDEX, i);
        }
        const uint32_t vmask = __ballot_sync(kFull, valid);
        const unsigned long long agg = (unsigned long long)__popc(vmask) * kRawGran;
        // the tile's size is known: publish it before anything else, later tiles' scans depend on it
        if (lane == 0 && tile != 0u) *reinterpret_cast<volatile unsigned long long *>(&a.scan->tile[tile]) = kFlagAgg | agg;
        // this lane's buffer is free once its previous record has been read out of shared memory
        bulk_wait_read();
        if (!chain_ok) valid = false;                                // nothing of this tile can be placed any more
        if (valid) {
            mbar_expect_tx(my_bar, kPageBytes);
            bulk_g2s(my_buf, a.src + (size_t)sp * (kPageBytes / 16), kPageBytes, my_bar);
        }
        in_flight = valid;
        unsigned long long base = 0;
        if (chain_ok) {
            chain_ok = tile_base(a, tile, agg, lane, base);
            if (!chain_ok && lane == 0) raise_status(a.ctl, SPECKV_ST_TIMEOUT, tile * kRawTile);
        } else if (lane == 0) {
            a.scan->tile[tile] = kFlagFail;                          // keep later tiles from waiting
        }
        if (chain_ok && lane == 0 && tile == a.n_tiles - 1) a.ctl->cursor64 = base + agg;
        if (valid) {
            // the page must have landed before the buffer is read or reused, whatever became of the scan
            const bool landed = mbar_wait(my_bar, phase & 1u, nullptr, a.wait_ns);
            in_flight = !landed;
            if (landed) phase += 1;
            if (!landed) raise_status(a.ctl, SPECKV_ST_TIMEOUT, i);
            else if (chain_ok) {
                const unsigned long long off64 = base + (unsigned long long)__popc(vmask & ((1u << lane) - 1u)) * kRawGran;
                if (off64 + kRawGran > a.pool_gran) {
                    raise_status(a.ctl, SPECKV_ST_POOL_FULL, i);
                } else {
                    uint8_t *dst = a.pool + off64 * kGranule;
                    bulk_s2g(dst, hdr, 16);
                    bulk_s2g(dst + 16, my_buf, kPageBytes);
                    bulk_s2g(dst + 16 + kPageBytes, hdr + 16, 48);
                    bulk_commit();
                    a.pte[slot] = off64 | ((unsigned long long)(kHdrBytes + kPageBytes) << 32) | kPteValid;   // mode 0
                    st_pages += 1;
                }
            }
        }
        if (__any_sync(kFull, in_flight)) break;                     // a copy towards this CTA never completed: stop taking tiles
    }
    // Leaving: nothing may still be on its way into this CTA's shared memory, and the stores must have
    // read it.  (A load that did not complete within its limit gets one more bounded wait.)
    if (in_flight) mbar_wait(my_bar, phase & 1u, nullptr, a.wait_ns);
    bulk_wait_all();
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) st_pages += __shfl_xor_sync(kFull, st_pages, d);
    if (lane == 0 && st_pages) {
        atomicAdd(&a.ctl->stats[kStMode0], st_pages);
        atomicAdd(&a.ctl->stats[kStGranules], st_pages * kRawGran);
        atomicAdd(&a.ctl->stats[kStPayload], st_pages * kPageBytes);
    }
}

cudaError_t launch_compress(const CompressArgs &a, int n_sm, cudaStream_t stream)
{
    uint32_t grid = a.n_tiles < (uint32_t)n_sm ? a.n_tiles : (uint32_t)n_sm;   // one persistent CTA per SM
    if ((a.scheme & ~SPECKV_GROUPED) == SPECKV_RAW) {
        cudaError_t e = cudaFuncSetAttribute(raw_copy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRawSmem);
        if (e != cudaSuccess) return e;
        raw_copy_kernel<<<grid, kRawWarps * 32, kRawSmem, stream>>>(a);
        return cudaGetLastError();
    }
    cudaError_t e = cudaFuncSetAttribute(compress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCompressSmem);
    if (e != cudaSuccess) return e;
    compress_kernel<<<grid, kCThreads, kCompressSmem, stream>>>(a);
    return cudaGetLastError();
}

// pages per tile (= per ticket) for a scheme, and the smallest of them (sizes the scan scratch)
uint32_t compress_tile_pages(int scheme) { return (scheme & ~SPECKV_GROUPED) == SPECKV_RAW ? kRawTile : (uint32_t)kEnc; }
uint32_t compress_min_tile_pages() { return kRawTile < (uint32_t)kEnc ? kRawTile : (uint32_t)kEnc; }

// ---------------------------------------------------------------- entry point without allocation

constexpr uint32_t kStaticMaxTiles = (SPECKV_STATIC_MAX_PAGES + kRawTile - 1) / kRawTile;   // the smaller tile decides

// Scan scratch of speckv_compress_static: ticket counter + one status word per tile.  Lives in
// every GPU context that loads the library (256 KiB) until the process exits.
static __device__ __align__(256) unsigned long long g_static_scan[2 + kStaticMaxTiles];

struct StaticSetup { ScanScratch *scan; int n_sm; bool ready; };
static StaticSetup g_static_setup[64];   // per device ordinal
static std::mutex g_static_mutex;

}  // namespace speckv

extern "C" int speckv_compress_static(const void *src, uint32_t n_src_pages, const uint32_t *src_page,
                                      const uint32_t *dst_slot, uint32_t n, int scheme, void *pool, uint64_t pool_bytes,
                                      uint64_t *pte, uint64_t n_slots, speckv_ctl_block *ctl, void *stream)
{
    using namespace speckv;
    static_assert(sizeof(speckv_ctl_block) == sizeof(Ctl), "control block layout");
    if (scheme < 0 || (scheme & ~SPECKV_GROUPED) > SPECKV_AUTO) return SPECKV_E_ARG;
    if (n > SPECKV_STATIC_MAX_PAGES) return SPECKV_E_TOO_LARGE;
    if (n == 0) return 0;
    if (!src || !src_page || !dst_slot || !pool || !pte || !ctl || ((uintptr_t)src & 15u) || ((uintptr_t)pool & 63u) ||
        (((uintptr_t)ctl | (uintptr_t)pte) & 7u) || (((uintptr_t)src_page | (uintptr_t)dst_slot) & 3u) ||
        pool_bytes == 0 || pool_bytes % kGranule || pool_bytes / kGranule > 0xFFFFFFFFull || n_slots == 0)
        return SPECKV_E_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SPECKV_E_CUDA;
    if (dev < 0 || dev >= 64) return SPECKV_E_ARG;
    StaticSetup su;
    {
        // Once per device, with that device current: in host code the array's name is only a handle,
        // the address the kernel needs comes from the runtime.  Under a lock, so that two host threads
        // making their first call at the same time both see a complete entry.
        std::lock_guard<std::mutex> guard(g_static_mutex);
        StaticSetup &slot = g_static_setup[dev];
        if (!slot.ready) {
            int major = 0, n_sm = 0;
            void *p = nullptr;
            if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
                cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
                return SPECKV_E_CUDA;
            if (major != 10) return SPECKV_E_DEVICE;
            if (cudaGetSymbolAddress(&p, g_static_scan) != cudaSuccess || !p) { cudaGetLastError(); return SPECKV_E_CUDA; }
            slot.scan = reinterpret_cast<ScanScratch *>(p);
            slot.n_sm = n_sm;
            slot.ready = true;
        }
        su = slot;
    }
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t tp = compress_tile_pages(scheme);
    const uint32_t n_tiles = (n + tp - 1) / tp;
    // the array keeps the previous call's tickets and status words: clear what this call will use
    if (cudaMemsetAsync(su.scan, 0, sizeof(ScanScratch) + (size_t)n_tiles * sizeof(unsigned long long), st) != cudaSuccess)
        return SPECKV_E_CUDA;
    CompressArgs a;
    a.src = (const uint4 *)src; a.src_page = src_page; a.dst_slot = dst_slot;
    a.pool = (uint8_t *)pool; a.pte = (unsigned long long *)pte; a.ctl = reinterpret_cast<Ctl *>(ctl); a.scan = su.scan;
    a.pool_gran = pool_bytes / kGranule; a.n_slots = n_slots;
    a.n_src_pages = n_src_pages; a.n = n; a.n_tiles = n_tiles; a.spin_limit = kDefaultSpinLimit; a.wait_ns = kDefaultWaitNs; a.ticket0 = 0; a.scheme = scheme;
    return launch_compress(a, su.n_sm, st) == cudaSuccess ? 0 : SPECKV_E_CUDA;
}
