// speckv_compact: pool lifecycle.  The record log only grows and a slot that is written again leaves
// its old record behind; this rewrites the pool so that it holds exactly the records that page-table
// entries point at, in slot order, from granule 0 on.  Four small kernels on one stream:
//   sizes     : one thread per slot -> granules of its record (0 if none); entries whose record is not
//               inside the pool are reported and cleared; per-block (512 slots) totals; the granules
//               that live records occupy are marked in a bitmap (one bit per granule of the pool)
//   scan      : one CTA, exclusive prefix of the block totals, new cursor
//   move      : one CTA per block: prefix inside the block, then one warp per record.  If no marked
//               granule lies in the record's new place, nothing that is still to be read can be
//               overwritten there: the warp reads the whole record into registers and writes it
//               straight to its final place.  Otherwise the record goes to the same place in the
//               scratch area and is flagged.  Either way the entry is rewritten.
//   copy back : one warp per flagged record: scratch -> pool
// A record moved directly costs one read and one write, a flagged one two of each.
#include "speckv_dev.cuh"

namespace speckv {

constexpr uint32_t kCBlock = 512;       // slots per CTA: 64 records per warp (1,024: a small pool leaves SMs idle; 256: 3 % slower on a full one)
constexpr uint32_t kCThreadsC = 256;
constexpr uint32_t kMaxRecPieces = ((kHdrBytes + kPageBytes + kGranule - 1u) / kGranule * 4u + 31u) / 32u;   // 16-byte pieces per lane: 9

struct CompactArgs {
    uint8_t *pool, *scratch;
    unsigned long long *pte;
    Ctl *ctl;
    uint32_t *gran;                       // [n_slots] granules per slot; bit 31: the record waits in the scratch area
    uint32_t *dest;                       // [n_slots] new place (granule) of a flagged record
    unsigned long long *block_base;       // [n_blocks + 1] totals, then exclusive prefixes
    uint32_t *live;                       // [ceil(pool_gran / 32)] bit g: granule g belongs to a live record's old place
    unsigned long long n_slots, pool_gran;
    uint32_t n_blocks;
};

__device__ __forceinline__ uint32_t block_sum_256(uint32_t v, uint32_t *s_warp)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    uint32_t t = 0;
    for (uint32_t i = 0; i < kCThreadsC / 32; ++i) t += s_warp[i];
    __syncthreads();
    return t;
}

__global__ void __launch_bounds__(kCThreadsC) compact_sizes_kernel(CompactArgs a)
{
    __shared__ uint32_t s_warp[kCThreadsC / 32];
    uint32_t mine = 0;
    for (uint32_t i = 0; i < kCBlock / kCThreadsC; ++i) {
        const unsigned long long slot = (unsigned long long)blockIdx.x * kCBlock + i * kCThreadsC + threadIdx.x;
        if (slot >= a.n_slots) continue;
        const unsigned long long e = a.pte[slot];
        uint32_t g = 0;
        if (e & kPteValid) {
            const uint32_t rec_len = (uint32_t)(e >> 32) & 0xFFFFu;
            g = (rec_len + kGranule - 1u) / kGranule;
            if (rec_len < kHdrBytes || (e & 0xFFFFFFFFull) + g > a.pool_gran) {
                raise_status(a.ctl, SPECKV_ST_BAD_RECORD, (uint32_t)slot);
                a.pte[slot] = 0ull;
                g = 0;
            } else {
                const unsigned long long lo = e & 0xFFFFFFFFull, hi = lo + g;          // granules [lo, hi)
                for (unsigned long long w = lo >> 5; w <= (hi - 1) >> 5; ++w) {
                    const unsigned long long b0 = w << 5;
                    const uint32_t from = lo > b0 ? (uint32_t)(lo - b0) : 0u, to = hi < b0 + 32 ? (uint32_t)(hi - b0) : 32u;
                    atomicOr(&a.live[w], (to == 32u ? 0xFFFFFFFFu : ((1u << to) - 1u)) & ~((1u << from) - 1u));
                }
            }
        }
        a.gran[slot] = g;
        mine += g;
    }
    const uint32_t total = block_sum_256(mine, s_warp);
    if (threadIdx.x == 0) a.block_base[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024) compact_scan_kernel(CompactArgs a)
{
    __shared__ unsigned long long s_part[32];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    unsigned long long carry = 0;
    for (uint32_t b0 = 0; b0 < a.n_blocks; b0 += 1024) {
        const uint32_t b = b0 + threadIdx.x;
        const unsigned long long v = b < a.n_blocks ? a.block_base[b] : 0ull;
        unsigned long long incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long t = __shfl_up_sync(kFull, incl, d);
            if (lane >= (uint32_t)d) incl += t;
        }
        if (lane == 31) s_part[warp] = incl;
        __syncthreads();
        unsigned long long before = carry, all = 0;
        for (uint32_t i = 0; i < 32; ++i) { if (i < warp) before += s_part[i]; all += s_part[i]; }
        if (b < a.n_blocks) a.block_base[b] = before + incl - v;
        carry += all;
        __syncthreads();
    }
    if (threadIdx.x == 0) { a.block_base[a.n_blocks] = carry; a.ctl->cursor64 = carry; }
}

__global__ void __launch_bounds__(kCThreadsC) compact_move_kernel(CompactArgs a)
{
    __shared__ uint32_t s_off[kCBlock];       // exclusive prefix of the block's sizes
    __shared__ uint32_t s_warp[kCThreadsC / 32];
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const unsigned long long slot0 = (unsigned long long)blockIdx.x * kCBlock;
    // thread t owns the kPer consecutive slots kPer * t ..
    constexpr uint32_t kPer = kCBlock / kCThreadsC;
    uint32_t g[kPer], sum = 0;
#pragma unroll
    for (uint32_t i = 0; i < kPer; ++i) {
        const unsigned long long slot = slot0 + kPer * tid + i;
        g[i] = slot < a.n_slots ? a.gran[slot] : 0u;
        sum += g[i];
    }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(kFull, incl, d);
        if (lane >= (uint32_t)d) incl += t;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t before = 0;
    for (uint32_t i = 0; i < warp; ++i) before += s_warp[i];
    uint32_t run = before + incl - sum;
#pragma unroll
    for (uint32_t i = 0; i < kPer; ++i) { s_off[kPer * tid + i] = run; run += g[i]; }
    __syncthreads();
    const unsigned long long base = a.block_base[blockIdx.x];
    for (uint32_t s = warp; s < kCBlock; s += kCThreadsC / 32) {
        const unsigned long long slot = slot0 + s;
        if (slot >= a.n_slots) break;
        const uint32_t n_gran = a.gran[slot];
        if (n_gran == 0) continue;
        const unsigned long long e = a.pte[slot];
        const uint4 *src = reinterpret_cast<const uint4 *>(a.pool + (e & 0xFFFFFFFFull) * kGranule);
        const unsigned long long at = base + s_off[s];
        if (at + n_gran > a.pool_gran) {                  // only if entries share records: more live bytes than pool
            if (lane == 0) { raise_status(a.ctl, SPECKV_ST_POOL_FULL, (uint32_t)slot); a.pte[slot] = 0ull; }
            continue;
        }
        // is any granule of the new place still somebody's old place (this record's own included: another
        // entry may share it)?
        bool busy = false;
        {
            const unsigned long long lo = at, hi = at + n_gran, w = (lo >> 5) + lane;
            if (w <= (hi - 1) >> 5) {
                const unsigned long long b0 = w << 5;
                const uint32_t from = lo > b0 ? (uint32_t)(lo - b0) : 0u, to = hi < b0 + 32 ? (uint32_t)(hi - b0) : 32u;
                busy = (a.live[w] & (to == 32u ? 0xFFFFFFFFu : ((1u << to) - 1u)) & ~((1u << from) - 1u)) != 0u;
            }
        }
        if (__any_sync(kFull, busy)) {
            uint4 *dst = reinterpret_cast<uint4 *>(a.scratch + at * kGranule);
            for (uint32_t i = lane; i < n_gran * 4u; i += 32) dst[i] = src[i];    // plain loads: this kernel also writes the pool
            if (lane == 0) { a.gran[slot] = n_gran | 0x80000000u; a.dest[slot] = (uint32_t)at; }
        } else {
            uint4 buf[kMaxRecPieces];                      // the whole record (at most 4,160 bytes) in the warp's registers
#pragma unroll
            for (uint32_t j = 0; j < kMaxRecPieces; ++j)
                if (j * 32u + lane < n_gran * 4u) buf[j] = src[j * 32u + lane];
            uint4 *dst = reinterpret_cast<uint4 *>(a.pool + at * kGranule);
#pragma unroll
            for (uint32_t j = 0; j < kMaxRecPieces; ++j)
                if (j * 32u + lane < n_gran * 4u) dst[j * 32u + lane] = buf[j];
        }
        if (lane == 0) a.pte[slot] = (e & ~0xFFFFFFFFull) | at;
    }
}

__global__ void __launch_bounds__(256) compact_copy_back_kernel(CompactArgs a)
{
    const uint32_t lane = threadIdx.x & 31u;
    const unsigned long long n_warps = (unsigned long long)gridDim.x * (blockDim.x >> 5);
    for (unsigned long long s0 = ((unsigned long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 32ull; s0 < a.n_slots;
         s0 += n_warps * 32ull) {
        // 32 slots at a time: one coalesced read of their flags, then the flagged ones in turn
        const unsigned long long mine = s0 + lane;
        const uint32_t g = mine < a.n_slots ? a.gran[mine] : 0u;
        uint32_t todo = __ballot_sync(kFull, (g & 0x80000000u) != 0u);
        while (todo) {
            const uint32_t l = __ffs(todo) - 1u;
            todo &= todo - 1u;
            const uint32_t n_gran = __shfl_sync(kFull, g, l) & 0x7FFFFFFFu;
            const uint32_t at = a.dest[s0 + l];
            const uint4 *src = reinterpret_cast<const uint4 *>(a.scratch + (unsigned long long)at * kGranule);
            uint4 *dst = reinterpret_cast<uint4 *>(a.pool + (unsigned long long)at * kGranule);
            for (uint32_t i = lane; i < n_gran * 4u; i += 32) dst[i] = src[i];
        }
    }
}

// speckv_free_slots: one thread per list entry swaps the page-table entry for zero; what it found there
// decides what is counted, so a slot named twice counts once whatever the scheduling.
__global__ void __launch_bounds__(256) free_slots_kernel(unsigned long long *pte, unsigned long long n_slots, Ctl *ctl,
                                                        const uint32_t *slots, uint32_t n, unsigned long long *freed)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t entries = 0, gran = 0;
    if (i < n) {
        const uint32_t slot = slots[i];
        if (slot >= n_slots) raise_status(ctl, SPECKV_ST_BAD_INDEX, i);
        else {
            const unsigned long long e = atomicExch(&pte[slot], 0ull);
            if (e & kPteValid) { entries = 1; gran = (((uint32_t)(e >> 32) & 0xFFFFu) + kGranule - 1u) / kGranule; }
        }
    }
    entries = __reduce_add_sync(kFull, entries);
    gran = __reduce_add_sync(kFull, gran);
    if ((threadIdx.x & 31u) == 0 && entries && freed) {
        atomicAdd(&freed[0], (unsigned long long)entries);
        atomicAdd(&freed[1], (unsigned long long)gran);
    }
}

cudaError_t launch_free_slots(unsigned long long *pte, unsigned long long n_slots, Ctl *ctl, const uint32_t *slots, uint32_t n,
                              unsigned long long *freed, cudaStream_t stream)
{
    free_slots_kernel<<<(n + 255u) / 256u, 256, 0, stream>>>(pte, n_slots, ctl, slots, n, freed);
    return cudaGetLastError();
}

static unsigned long long align256(unsigned long long v) { return (v + 255ull) & ~255ull; }

// scratch layout: [pool_bytes] records | [n_slots] granules | [n_slots] new places | block prefixes | live bitmap
size_t compact_scratch_bytes(unsigned long long n_slots, unsigned long long pool_bytes)
{
    const unsigned long long n_blocks = (n_slots + kCBlock - 1) / kCBlock;
    return (size_t)(pool_bytes + 2 * align256(n_slots * 4) + align256((n_blocks + 1) * 8) + align256((pool_bytes / kGranule + 31) / 32 * 4));
}

cudaError_t launch_compact(uint8_t *pool, unsigned long long pool_bytes, unsigned long long *pte, unsigned long long n_slots,
                           Ctl *ctl, uint8_t *scratch, int n_sm, cudaStream_t stream)
{
    CompactArgs a;
    a.pool = pool; a.scratch = scratch; a.pte = pte; a.ctl = ctl;
    const unsigned long long n_blocks = (n_slots + kCBlock - 1) / kCBlock;
    uint8_t *p = scratch + pool_bytes;
    a.gran = reinterpret_cast<uint32_t *>(p); p += align256(n_slots * 4);
    a.dest = reinterpret_cast<uint32_t *>(p); p += align256(n_slots * 4);
    a.block_base = reinterpret_cast<unsigned long long *>(p); p += align256((n_blocks + 1) * 8);
    a.live = reinterpret_cast<uint32_t *>(p);
    a.n_slots = n_slots; a.pool_gran = pool_bytes / kGranule;
    a.n_blocks = (uint32_t)n_blocks;
    cudaError_t e = cudaMemsetAsync(a.live, 0, (size_t)((a.pool_gran + 31) / 32 * 4), stream);
    if (e != cudaSuccess) return e;
    compact_sizes_kernel<<<a.n_blocks, kCThreadsC, 0, stream>>>(a);
    compact_scan_kernel<<<1, 1024, 0, stream>>>(a);
    compact_move_kernel<<<a.n_blocks, kCThreadsC, 0, stream>>>(a);
    compact_copy_back_kernel<<<n_sm * 8, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace speckv
