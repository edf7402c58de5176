// Device-side definitions shared by the speckv kernels (sm_100a).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "speckv.h"

namespace speckv {

constexpr uint32_t kPageElems = 2048;
constexpr uint32_t kPageBytes = 4096;
constexpr uint32_t kHdrBytes = 16;
constexpr uint32_t kGranule = 64;
constexpr uint32_t kBitmapBytes = 256;
constexpr uint32_t kValuesOff = kHdrBytes + kBitmapBytes;        // 272
constexpr uint32_t kGroupBytes = 32;                                  // grouped scales: 16 binary16 maxima before the payload
constexpr uint32_t kMaxPackedRec = kHdrBytes + kGroupBytes + kBitmapBytes + kPageElems;  // 2352 (mode 3 | grouped, every symbol a run)
constexpr uint32_t kRecStage = 2432;                             // staging bytes per warp (38 granules)
constexpr uint32_t kVersion = 1;
constexpr uint32_t kFull = 0xFFFFFFFFu;
constexpr float kMagic = 12582912.0f;                            // 1.5 * 2^23: fma(x, inv, kMagic) rounds to integer

constexpr uint64_t kPteValid = 1ull << 56;

// Control block in device memory, one per context.
struct Ctl {
    unsigned long long cursor64;              // next free granule of the pool
    unsigned int status_count[SPECKV_N_STATUS];
    unsigned int status_first[SPECKV_N_STATUS];
    unsigned long long stats[11];             // same order as speckv_stats
};
enum { kStMode0 = 0, kStGranules = 4, kStPayload = 5, kStRuns = 6, kStNonfinite = 7, kStDecoded = 8,
       kStPfIssued = 9, kStPfSkipped = 10 };

// Scratch of the compressor's chained scan: one ticket counter + one status word per tile.
struct ScanScratch {
    unsigned int ticket;
    unsigned int pad;
    unsigned long long tile[1];               // [n_tiles]: flag << 62 | value
};
constexpr unsigned long long kFlagAgg = 1ull << 62, kFlagPrefix = 2ull << 62, kFlagFail = 3ull << 62;
constexpr unsigned long long kFlagMask = 3ull << 62;

__device__ __forceinline__ void raise_status(Ctl *ctl, int code, uint32_t index)
{
    atomicAdd(&ctl->status_count[code], 1u);
    atomicMin(&ctl->status_first[code], index);
}

// ---- SIMD-in-a-word helpers (also compiled for the host so that they can be unit-tested) ----

// per-byte a - b (mod 256)
__host__ __device__ __forceinline__ uint32_t bsub4(uint32_t a, uint32_t b)
{
    uint32_t t = (a | 0x80808080u) - (b & 0x7F7F7F7Fu);
    return t ^ ((a ^ ~b) & 0x80808080u);
}
// per-byte a + b (mod 256)
__host__ __device__ __forceinline__ uint32_t badd4(uint32_t a, uint32_t b)
{
    uint32_t t = (a & 0x7F7F7F7Fu) + (b & 0x7F7F7F7Fu);
    return t ^ ((a ^ b) & 0x80808080u);
}
// bit 7 of each byte set iff that byte of d is non-zero
__host__ __device__ __forceinline__ uint32_t nz4(uint32_t d)
{
    return (((d & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | d) & 0x80808080u;
}
// gather bit 7 of the 4 bytes of n0 into bits 0-3 and of n1 into bits 4-7
__host__ __device__ __forceinline__ uint32_t msb8(uint32_t n0, uint32_t n1)
{
    uint32_t t = (n0 >> 7) | (n1 >> 3);
    return ((t * 0x00204081u) >> 21) & 0xFFu;
}

// Selector tables.  compact_sel(m): nibble j = position of the j-th set bit of m (for PRMT over
// the 8 symbol bytes); expand_sel(h): nibble e = number of set bits of the 4-bit mask h at or
// below position e (index into "carry byte + following values").
__host__ __device__ inline uint32_t compact_sel(uint32_t m)
{
    uint32_t sel = 0, j = 0;
    for (uint32_t e = 0; e < 8; ++e)
        if ((m >> e) & 1u) { sel |= e << (4 * j); ++j; }
    return sel;
}
__host__ __device__ inline uint32_t expand_sel(uint32_t h)
{
    uint32_t sel = 0, c = 0;
    for (uint32_t e = 0; e < 4; ++e) { c += (h >> e) & 1u; sel |= c << (4 * e); }
    return sel;
}

// Exclusive prefix sum over the lanes of four byte fields at once.  The caller guarantees that no
// field's sum over any 31 lanes reaches 256.  The shuffle's own "source lane exists" predicate guards
// the additions.
__device__ __forceinline__ uint32_t scan_excl_bytes(uint32_t v)
{
    uint32_t e;
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\t"
                 "shfl.sync.up.b32 %0|p, %1, 1, 0, 0xffffffff;\n\t@!p mov.b32 %0, 0;\n\t"
                 "shfl.sync.up.b32 t|p, %0, 1, 0, 0xffffffff;\n\t@p add.u32 %0, %0, t;\n\t"
                 "shfl.sync.up.b32 t|p, %0, 2, 0, 0xffffffff;\n\t@p add.u32 %0, %0, t;\n\t"
                 "shfl.sync.up.b32 t|p, %0, 4, 0, 0xffffffff;\n\t@p add.u32 %0, %0, t;\n\t"
                 "shfl.sync.up.b32 t|p, %0, 8, 0, 0xffffffff;\n\t@p add.u32 %0, %0, t;\n\t"
                 "shfl.sync.up.b32 t|p, %0, 16, 0, 0xffffffff;\n\t@p add.u32 %0, %0, t;\n\t}"
                 : "=&r"(e) : "r"(v));
    return e;
}

// ---- kernel arguments and launchers ----

struct CompressArgs {
    const uint4 *src;
    const uint32_t *src_page, *dst_slot;
    uint8_t *pool;
    unsigned long long *pte;
    Ctl *ctl;
    ScanScratch *scan;
    unsigned long long pool_gran, n_slots;
    uint32_t n_src_pages, n, n_tiles;
    uint32_t spin_limit;            // polls of one look-back window before the scan gives up
    unsigned long long wait_ns;     // time limit of every wait on a shared-memory barrier
    uint32_t ticket0;               // first tile number drawn (0 except under fault injection: lower tiles never appear)
    int scheme;
};
constexpr uint32_t kDefaultSpinLimit = 4u << 20;               // >= 200 ns per poll: gives up after a few seconds
constexpr unsigned long long kDefaultWaitNs = 2000000000ull;
struct GatherArgs {
    const uint8_t *pool;
    const unsigned long long *pte;
    unsigned long long *l2_tag;
    Ctl *ctl;
    const int32_t *block_table;
    const uint32_t *seq_lens;
    const unsigned long long *dst_tok_off;
    const speckv_prefetch *pf;
    uint4 *dst_demand, *dst_l2;
    unsigned long long pool_bytes, dst_cap_tokens;
    uint32_t layer, B, n_pf, epoch;
    uint32_t chain;   // 0 = ordinary launch; 1 = chained to the previous gather, waits for it before writing; 2 = chained, independent of it
    uint32_t n_layers, H, blocks_per_layer, max_blocks_per_seq, max_seqs;
};
struct TranslateArgs {
    const unsigned long long *pte;
    const int32_t *block_table;
    const speckv_vaddr *va;
    speckv_paddr *pa;
    Ctl *ctl;
    unsigned long long pool_bytes;
    uint32_t n, n_layers, H, blocks_per_layer, max_blocks_per_seq, max_seqs;
};
struct AttendArgs {
    // fused source: records through the page table
    const uint8_t *pool;
    const unsigned long long *pte;
    const int32_t *block_table;
    unsigned long long pool_bytes;
    uint32_t layer, blocks_per_layer, max_blocks_per_seq;
    // dense source: the demand workspace of speckv_decompress_gather
    const uint4 *kv;
    const unsigned long long *tok_off;
    // common
    Ctl *ctl;
    const uint32_t *seq_lens;
    const __half *q;
    __half *out;
    float *partial;       // workspace: per partial result o[8][128], m[8], l[8]
    uint32_t *prefix;     // workspace: 16-token blocks of the sequences before b, [B + 1]
    uint32_t B, H, G;
};
struct PrefetchArgs {
    const uint8_t *pool;
    const unsigned long long *pte;
    Ctl *ctl;
    const int32_t *block_table, *access, *cand;
    speckv_pf_seq *state;
    speckv_pf_counters *cnt;
    uint4 *l2, *miss_dst;
    int32_t *where;
    double beta;
    unsigned long long pool_bytes;
    uint32_t layer, back, B, H, blocks_per_layer, max_blocks_per_seq, max_seqs;
};
cudaError_t launch_prefetch_step(const PrefetchArgs &a, int n_sm, cudaStream_t stream);
uint32_t prefetch_max_seqs();
cudaError_t launch_compress(const CompressArgs &a, int n_sm, cudaStream_t stream);
cudaError_t launch_attend(const AttendArgs &a, bool fused, int n_sm, cudaStream_t stream);
uint32_t attend_max_warps();
size_t compact_scratch_bytes(unsigned long long n_slots, unsigned long long pool_bytes);
cudaError_t launch_compact(uint8_t *pool, unsigned long long pool_bytes, unsigned long long *pte, unsigned long long n_slots,
                           Ctl *ctl, uint8_t *scratch, int n_sm, cudaStream_t stream);
cudaError_t launch_free_slots(unsigned long long *pte, unsigned long long n_slots, Ctl *ctl, const uint32_t *slots, uint32_t n,
                              unsigned long long *freed, cudaStream_t stream);
cudaError_t launch_gather(const GatherArgs &a, int n_sm, cudaStream_t stream);
cudaError_t launch_translate(const TranslateArgs &a, cudaStream_t stream);
uint32_t compress_tile_pages(int scheme);
uint32_t compress_min_tile_pages();
uint32_t gather_max_seqs();


}  // namespace speckv
