// The per-layer computation that consumes fetched KV pages (the T_layer stage of CXL-SpecKV's
// multi-layer prefetch pipeline, Sec. 3.4.4): decode-step attention, one query token per sequence.
//
//   attend_dense_kernel : reads K/V from the workspace that speckv_decompress_gather wrote.
//   attend_fused_kernel : fetches the records itself (block table -> PTE -> bulk copy -> decode into
//                         shared memory), so the decompressed K/V never touch HBM.
//   attend_combine_kernel : merges the partial results of each (sequence, KV head).
//
// Work is split evenly: the blocks of all (sequence, KV head) pairs form one long list, every warp of
// the grid takes an equal contiguous share of it and emits one partial result per (sequence, KV head)
// it touches; partial number = warp + pair number, which is unique because both only grow along the
// list.  A warp serves the KV head's G <= 8 query heads at once.  Per 16-token block, with the tile in shared memory
// ([16 tokens][128 channels] binary16, rows 272 bytes apart so that ldmatrix is conflict-free):
//   S^T[token][head] = K Q^T        8 x mma.m16n8k16 (tokens are the M dimension: no padding)
//   online softmax in binary32 (base 2), per head column; P rounded to binary16
//   O^T[channel][head] += V^T P^T   8 x mma.m16n8k16, V^T via ldmatrix.trans, P^T via movmatrix
// The contraction is 16 rows per page and the kernels are bound by memory and by the decoder, which
// is why this uses warp-level MMA and not the 128-row tcgen05 path.
#include <cuda_fp16.h>

#include "async_ptx.cuh"
#include "decode.cuh"
#include "speckv_dev.cuh"

namespace speckv {

constexpr uint32_t kTilePitch = 272;                    // bytes between token rows of a tile
constexpr uint32_t kTileBytes = 16 * kTilePitch;        // 4,352
constexpr uint32_t kHeadsPad = 8;                       // query heads per KV head, padded to the MMA's n
constexpr uint32_t kPartialFloats = kHeadsPad * 130;    // per partial result: o[8][128], then m[8], l[8]
constexpr float kNegInf = -__builtin_huge_valf();

// ---------------------------------------------------------------- warp-level MMA wrappers

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// c += a (16x16, row-major) * b (16x8, column-major), binary16 inputs, binary32 accumulation
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transposes an 8x8 binary16 matrix held in fragment layout
__device__ __forceinline__ uint32_t movm_trans(uint32_t x)
{
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---------------------------------------------------------------- attention state of one (sequence, KV head) piece

// Lane l holds, of S^T and O^T, the head columns 2*(l%4) and 2*(l%4)+1.
struct AttnState {
    uint32_t qf[8][2];   // Q^T as the MMA's B operand: [channel step][2]
    float o[8][4];       // O^T accumulators: [16-channel tile][fragment]
    float m[2], l[2];    // running maximum (base-2 scores) and this lane's share of the denominator
};

__device__ __forceinline__ void attn_begin(AttnState &st, const __half *q_heads, uint32_t G, uint32_t lane)
{
    const uint32_t head = lane >> 2;
    const uint32_t *qw = reinterpret_cast<const uint32_t *>(q_heads + head * 128u) + (lane & 3u);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        st.qf[ks][0] = head < G ? __ldg(qw + ks * 8) : 0u;          // channels 16*ks + 2*(l%4), +1
        st.qf[ks][1] = head < G ? __ldg(qw + ks * 8 + 4) : 0u;      // channels 16*ks + 8 + 2*(l%4), +1
    }
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) st.o[mt][0] = st.o[mt][1] = st.o[mt][2] = st.o[mt][3] = 0.0f;
    st.m[0] = st.m[1] = kNegInf;
    st.l[0] = st.l[1] = 0.0f;
}

// One 16-token block: tiles at shared-memory addresses k_tile, v_tile; tok0 = sequence position of
// the block's first token; tokens at or beyond len are masked.
__device__ __forceinline__ void attn_block(AttnState &st, uint32_t k_tile, uint32_t v_tile, uint32_t tok0, uint32_t len, uint32_t lane)
{
    const float scale = 0.12752551286084112f;            // log2(e) / sqrt(128)
    const uint32_t jm = lane >> 3, r = lane & 7u;
    float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    const uint32_t ka = k_tile + ((jm & 1u) * 8u + r) * kTilePitch + (jm >> 1) * 16u;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        uint32_t a[4];
        ldsm_x4(ka + ks * 32, a);
        mma_16816(c, a, st.qf[ks][0], st.qf[ks][1]);
    }
    const uint32_t t0 = tok0 + (lane >> 2), t1 = t0 + 8u;
    const float s0 = t0 < len ? c[0] * scale : kNegInf, s1 = t0 < len ? c[1] * scale : kNegInf;
    const float s2 = t1 < len ? c[2] * scale : kNegInf, s3 = t1 < len ? c[3] * scale : kNegInf;
    float mxa = fmaxf(s0, s2), mxb = fmaxf(s1, s3);
#pragma unroll
    for (int d = 4; d < 32; d <<= 1) {
        mxa = fmaxf(mxa, __shfl_xor_sync(kFull, mxa, d));
        mxb = fmaxf(mxb, __shfl_xor_sync(kFull, mxb, d));
    }
    const float ma = fmaxf(st.m[0], mxa), mb = fmaxf(st.m[1], mxb);
    const float ra = ma == kNegInf ? 0.0f : ma, rb = mb == kNegInf ? 0.0f : mb;   // nothing valid yet: keep exponents finite
    const float ala = ex2(st.m[0] - ra), alb = ex2(st.m[1] - rb);
    const float p0 = ex2(s0 - ra), p1 = ex2(s1 - rb), p2 = ex2(s2 - ra), p3 = ex2(s3 - rb);
    st.m[0] = ma; st.m[1] = mb;
    st.l[0] = st.l[0] * ala + p0 + p2;
    st.l[1] = st.l[1] * alb + p1 + p3;
    const uint32_t b0 = movm_trans(pack_h2(p0, p1)), b1 = movm_trans(pack_h2(p2, p3));
    const uint32_t va = v_tile + ((jm >> 1) * 8u + r) * kTilePitch + (jm & 1u) * 16u;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
        st.o[mt][0] *= ala; st.o[mt][1] *= alb; st.o[mt][2] *= ala; st.o[mt][3] *= alb;
        uint32_t a[4];
        ldsm_x4_trans(va + mt * 32, a);
        mma_16816(st.o[mt], a, b0, b1);
    }
}

// Writes the piece's partial result: o[8 heads][128 channels], then m[8], l[8].
__device__ __forceinline__ void attn_end(AttnState &st, float *partial, uint32_t lane)
{
#pragma unroll
    for (int d = 4; d < 32; d <<= 1) {
        st.l[0] += __shfl_xor_sync(kFull, st.l[0], d);
        st.l[1] += __shfl_xor_sync(kFull, st.l[1], d);
    }
    const uint32_t h0 = (lane & 3u) * 2u, ch = lane >> 2;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
        partial[h0 * 128u + 16u * mt + ch] = st.o[mt][0];
        partial[(h0 + 1u) * 128u + 16u * mt + ch] = st.o[mt][1];
        partial[h0 * 128u + 16u * mt + 8u + ch] = st.o[mt][2];
        partial[(h0 + 1u) * 128u + 16u * mt + 8u + ch] = st.o[mt][3];
    }
    if (lane < 4) {
        float *ml = partial + kHeadsPad * 128u;
        ml[h0] = st.m[0]; ml[h0 + 1u] = st.m[1];
        ml[kHeadsPad + h0] = st.l[0]; ml[kHeadsPad + h0 + 1u] = st.l[1];
    }
}

// ---------------------------------------------------------------- work split

// s_blk[b] = number of 16-token blocks of the sequences before b (shared memory, [B + 1]); also
// written to the workspace for the merge pass.
// `limit`: most blocks a sequence may have (the block table's width for the fused source); a longer one is
// reported once as unmapped, at the index its first page would have had, and contributes no blocks.
__device__ __forceinline__ void build_prefix(const AttendArgs &a, uint32_t *s_blk, uint32_t tid, uint32_t n_threads, uint32_t limit)
{
    for (uint32_t b = tid; b < a.B; b += n_threads) {
        const unsigned long long nb = ((unsigned long long)a.seq_lens[b] + 15ull) >> 4;
        s_blk[b + 1] = nb > limit ? 0u : (uint32_t)nb;
    }
    if (tid == 0) s_blk[0] = 0;
    __syncthreads();
    if (tid < 32) {                                       // one warp: serial over 32-wide pieces
        uint32_t run = 0;
        for (uint32_t b0 = 0; b0 < a.B; b0 += 32) {
            const uint32_t b = b0 + tid;
            uint32_t v = b < a.B ? s_blk[b + 1] : 0u;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t t = __shfl_up_sync(kFull, v, d);
                if (tid >= (uint32_t)d) v += t;
            }
            if (b < a.B) s_blk[b + 1] = run + v;
            run += __shfl_sync(kFull, v, 31);
        }
    }
    __syncthreads();
    if (blockIdx.x == 0) {
        for (uint32_t b = tid; b <= a.B; b += n_threads) a.prefix[b] = s_blk[b];
        for (uint32_t b = tid; b < a.B; b += n_threads)
            if ((((unsigned long long)a.seq_lens[b] + 15ull) >> 4) > limit) raise_status(a.ctl, SPECKV_ST_UNMAPPED, s_blk[b] * 2u * a.H);
    }
}

// This warp's share [g0, g1) of the list of T = H * (all blocks) block positions, ordered by
// (sequence, KV head, block): equal shares of ceil(T / warps).
struct Share { unsigned long long g, g1; uint32_t b, h, n; };

__device__ __forceinline__ Share first_piece(const uint32_t *s_blk, uint32_t B, uint32_t H, uint32_t w, uint32_t n_warps)
{
    Share sh;
    const unsigned long long T = (unsigned long long)s_blk[B] * H;
    const unsigned long long per = (T + n_warps - 1) / n_warps;
    sh.g = min(T, (unsigned long long)w * per);
    sh.g1 = min(T, sh.g + per);
    sh.b = sh.h = sh.n = 0;
    if (sh.g < sh.g1) {
        uint32_t lo = 0, hi = B;                           // invariant: s_blk[lo] * H <= g < s_blk[hi] * H
        while (hi - lo > 1u) {
            const uint32_t mid = (lo + hi) >> 1;
            if ((unsigned long long)s_blk[mid] * H <= sh.g) lo = mid; else hi = mid;
        }
        const uint32_t nblk = s_blk[lo + 1] - s_blk[lo];
        const uint32_t r = (uint32_t)(sh.g - (unsigned long long)s_blk[lo] * H);
        sh.b = lo; sh.h = r / nblk; sh.n = r % nblk;
    }
    return sh;
}

// after nb blocks of (b, h) have been taken: move to the next non-empty (sequence, KV head)
__device__ __forceinline__ void advance(Share &sh, const uint32_t *s_blk, uint32_t B, uint32_t H, uint32_t nb)
{
    sh.g += nb;
    sh.n += nb;
    if (sh.n == s_blk[sh.b + 1] - s_blk[sh.b]) {
        sh.n = 0;
        if (++sh.h == H) {
            sh.h = 0;
            do ++sh.b; while (sh.b < B && s_blk[sh.b + 1] == s_blk[sh.b]);
        }
    }
}

// ---------------------------------------------------------------- dense source

constexpr int kDWarps = 4;
constexpr uint32_t kDStages = 2;   // K+V tile pairs per warp: the block in use and the next one on its way

__global__ void __launch_bounds__(kDWarps * 32, 3) attend_dense_kernel(AttendArgs a)
{
    extern __shared__ __align__(16) uint8_t smem[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");          // the merge kernel may be scheduled behind this grid
    unsigned long long *s_bar = reinterpret_cast<unsigned long long *>(smem + kDWarps * kDStages * 2 * kTileBytes);   // [kDWarps][kDStages]
    uint32_t *s_blk = reinterpret_cast<uint32_t *>(s_bar + kDWarps * kDStages);
    const uint32_t tid = threadIdx.x, lane = tid & 31u;
    const uint32_t warp = __shfl_sync(kFull, tid >> 5, 0);
    if (tid < kDWarps * kDStages) mbar_init(smem_u32(s_bar + tid), 1);
    mbar_init_fence();
    build_prefix(a, s_blk, tid, kDWarps * 32, 0xFFFFFFFFu);   // the workspace holds what the lengths say: no table to exceed
    const uint32_t tiles = smem_u32(smem + warp * kDStages * 2 * kTileBytes);   // [stage][K|V]
    const uint32_t my_bar = smem_u32(s_bar + warp * kDStages);
    uint32_t phases = 0;                                                        // bit s: parity of stage s's barrier
    const uint32_t w = blockIdx.x * kDWarps + warp;

    for (Share sh = first_piece(s_blk, a.B, a.H, w, gridDim.x * kDWarps); sh.g < sh.g1;) {
        const uint32_t b = sh.b, h = sh.h, n0 = sh.n;
        const uint32_t len = a.seq_lens[b], nblk = s_blk[b + 1] - s_blk[b];
        const uint32_t nb = (uint32_t)min((unsigned long long)(nblk - n0), sh.g1 - sh.g);
        const unsigned long long tpad = (unsigned long long)nblk * 16u;
        // workspace of the demand path: [K|V][head][token][channel] per sequence
        const uint4 *kbase = a.kv + (a.tok_off[b] * 2u * a.H * 128u + ((unsigned long long)h * tpad + 16u * n0) * 128u) / 8u;
        const uint4 *vbase = kbase + ((unsigned long long)a.H * tpad * 128u) / 8u;
        // block n0 + i -> stage i % kDStages: one bulk copy per token row (256 B) and lane — lanes 0-15 the K rows,
        // 16-31 the V rows — onto the stage's barrier; the copy engine does the moving, the warp only waits
        auto load = [&](uint32_t i) {
            const uint32_t stg = i % kDStages, dst = tiles + stg * 2u * kTileBytes, bar = my_bar + 8u * stg;
            if (lane == 0) mbar_expect_tx(bar, 2u * 16u * 256u);
            __syncwarp();
            const uint4 *src = (lane < 16 ? kbase : vbase) + (size_t)i * 256u + (lane & 15u) * 16u;
            bulk_g2s(dst + (lane >> 4) * kTileBytes + (lane & 15u) * kTilePitch, src, 256u, bar);
        };
        AttnState st;
        attn_begin(st, a.q + ((size_t)b * a.H + h) * a.G * 128u, a.G, lane);
#pragma unroll
        for (uint32_t i = 0; i + 1 < kDStages; ++i)
            if (i < nb) load(i);
        for (uint32_t i = 0; i < nb; ++i) {
            if (i + kDStages - 1 < nb) load(i + kDStages - 1);                // into the stage freed by block i - 1
            const uint32_t stg = i % kDStages;
            if (!mbar_wait_warp(my_bar + 8u * stg, (phases >> stg) & 1u)) {        // never expected: report once, drop the rest of the piece
                if (lane == 0) raise_status(a.ctl, SPECKV_ST_TIMEOUT, s_blk[b] * 2u * a.H);
                break;
            }
            phases ^= 1u << stg;
            const uint32_t t = tiles + stg * 2u * kTileBytes;
            attn_block(st, t, t + kTileBytes, 16u * (n0 + i), len, lane);
            __syncwarp();                                                     // the stage is refilled by the next iteration's load
        }
        attn_end(st, a.partial + (size_t)(w + b * a.H + h) * kPartialFloats, lane);
        advance(sh, s_blk, a.B, a.H, nb);
    }
}

// ---------------------------------------------------------------- fused source: records -> tiles

constexpr int kFWarps = 8;
constexpr uint32_t kFStage = kRecStage;                   // bytes per record buffer
constexpr uint32_t kFWarpBytes = 2 * kFStage + 2 * kTileBytes;

__global__ void __launch_bounds__(kFWarps * 32, 2) attend_fused_kernel(AttendArgs a)
{
    extern __shared__ __align__(16) uint8_t smem[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");          // the merge kernel may be scheduled behind this grid
    uint4 *s_lut = reinterpret_cast<uint4 *>(smem + kFWarps * kFWarpBytes);          // [256]
    unsigned long long *s_bar = reinterpret_cast<unsigned long long *>(s_lut + 256);      // [kFWarps][2]
    uint32_t *s_blk = reinterpret_cast<uint32_t *>(s_bar + kFWarps * 2);
    const uint32_t tid = threadIdx.x, lane = tid & 31u;
    const uint32_t warp = __shfl_sync(kFull, tid >> 5, 0);
    s_lut[tid & 255u] = expand_entry(tid & 255u);
    if (tid < kFWarps * 2) mbar_init(smem_u32(s_bar + tid), 1);
    mbar_init_fence();
    build_prefix(a, s_blk, tid, kFWarps * 32, a.max_blocks_per_seq);
    uint8_t *my = smem + warp * kFWarpBytes;
    uint8_t *my_rec = my;                                                     // [2][kFStage]
    uint8_t *my_tile = my + 2 * kFStage;                                      // [K|V][kTileBytes]
    const uint32_t my_bar = smem_u32(s_bar + warp * 2);
    const uint32_t twoH = 2u * a.H;
    const unsigned long long layer_slot0 = (unsigned long long)a.layer * a.blocks_per_layer * twoH;
    uint32_t n_issued = 0, n_consumed = 0;                                    // record copies, over the whole kernel
    uint32_t st_decoded = 0;

    const uint32_t w = blockIdx.x * kFWarps + warp;
    for (Share sh = first_piece(s_blk, a.B, a.H, w, gridDim.x * kFWarps); sh.g < sh.g1;) {
      const uint32_t b = sh.b, h = sh.h;
      const uint32_t len = a.seq_lens[b], nblk = s_blk[b + 1] - s_blk[b];
      const uint32_t n_piece = (uint32_t)min((unsigned long long)(nblk - sh.n), sh.g1 - sh.g);
      const uint32_t index0 = s_blk[b] * twoH;                                // page numbering of the demand fetch
      AttnState st;
      attn_begin(st, a.q + ((size_t)b * a.H + h) * a.G * 128u, a.G, lane);
      // the piece in runs of up to 16 blocks: one lane translates one page
      for (uint32_t done = 0; done < n_piece; done += 16u) {
        const uint32_t n0 = sh.n + done, nb = min(16u, n_piece - done);

        // ---- translation of the run's 2*nb pages, one lane each: page j = block n0 + j/2, K (0) or V (1)
        unsigned long long pte = 0;
        int rc = -1;                                                          // -1: no page on this lane
        uint32_t pidx = 0;
        if (lane < 2u * nb) {
            const uint32_t n = n0 + (lane >> 1), kv = lane & 1u;
            pidx = index0 + (n * 2u + kv) * a.H + h;
            rc = SPECKV_ST_UNMAPPED;
            if (n < a.max_blocks_per_seq) {
                const int32_t p = __ldg(a.block_table + (size_t)b * a.max_blocks_per_seq + n);
                if (p >= 0 && (uint32_t)p < a.blocks_per_layer) {
                    pte = __ldg(a.pte + layer_slot0 + ((unsigned long long)(uint32_t)p * 2u + kv) * a.H + h);
                    const Walk wk = decode_pte(pte, a.pool_bytes);
                    rc = wk.rc;
                    if (!rc && wk.mode != SPECKV_RAW && ((wk.mode & ~(uint32_t)SPECKV_GROUPED) - 1u > 2u || wk.rec_len > kMaxPackedRec))
                        rc = SPECKV_ST_BAD_RECORD;
                }
            }
            if (rc) raise_status(a.ctl, rc, pidx);
        }
        auto issue = [&](uint32_t j) {                                        // start the copy of page j's record, if it has one
            const unsigned long long e = __shfl_sync(kFull, pte, j);
            const int r = __shfl_sync(kFull, rc, j);
            const uint32_t mode = (uint32_t)(e >> 48) & 0xFFu;
            if (r != 0 || mode == SPECKV_RAW) return;
            if (lane == 0) {
                const uint32_t rec_len = (uint32_t)(e >> 32) & 0xFFFFu;
                const uint32_t bytes = (rec_len + 15u) & ~15u, buf = n_issued & 1u, bar = my_bar + 8u * buf;
                mbar_expect_tx(bar, bytes);
                bulk_g2s(smem_u32(my_rec + buf * kFStage), a.pool + (e & 0xFFFFFFFFull) * kGranule, bytes, bar);
            }
            ++n_issued;
        };

        issue(0);
        bool k_ok = false;
        for (uint32_t j = 0; j < 2u * nb; ++j) {
            if (j + 1 < 2u * nb) issue(j + 1);
            const unsigned long long e = __shfl_sync(kFull, pte, j);
            const int r = __shfl_sync(kFull, rc, j);
            const uint32_t index = __shfl_sync(kFull, pidx, j);
            const uint32_t rec_len = (uint32_t)(e >> 32) & 0xFFFFu, pte_mode = (uint32_t)(e >> 48) & 0xFFu;
            uint8_t *tile = my_tile + (j & 1u) * kTileBytes;
            auto put = [&](int k, const uint4 &v) {
                *reinterpret_cast<uint4 *>(tile + (2u * k + (lane >> 4)) * kTilePitch + (lane & 15u) * 16u) = v;
            };
            bool ok = false;
            if (r == 0) {
                if (pte_mode == SPECKV_RAW) {                                 // bypass: the payload is the page
                    const uint4 *src = reinterpret_cast<const uint4 *>(a.pool + (e & 0xFFFFFFFFull) * kGranule);
                    const uint4 hdr = __ldg(src);
                    ok = (hdr.y >> 24) == kVersion && ((hdr.y >> 16) & 0xFFu) == SPECKV_RAW && (hdr.y & 0xFFFFu) == kPageBytes &&
                         rec_len == kHdrBytes + kPageBytes;
                    if (ok) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) put(k, __ldg(src + 1 + k * 32 + lane));
                    }
                } else {
                    const uint32_t buf = n_consumed & 1u, parity = (n_consumed >> 1) & 1u;
                    ++n_consumed;
                    const uint8_t *rec = my_rec + buf * kFStage;
                    if (!mbar_wait(my_bar + 8u * buf, parity)) {              // never expected: report and stop this warp
                        if (lane == 0) raise_status(a.ctl, SPECKV_ST_TIMEOUT, index);
                        // the next record's copy may be in flight: stay (bounded) until it has landed
                        if (n_issued > n_consumed) mbar_wait(my_bar + 8u * (n_consumed & 1u), (n_consumed >> 1) & 1u);
                        return;
                    }
                    const uint4 hdr = *reinterpret_cast<const uint4 *>(rec);
                    const uint32_t payload_len = hdr.y & 0xFFFFu, mode = (hdr.y >> 16) & 0xFFu;
                    ok = (hdr.y >> 24) == kVersion && mode == pte_mode && kHdrBytes + payload_len == rec_len;
                    if (ok) ok = decode_page(rec, mode, payload_len, hdr.z & 0xFFFFu, __uint_as_float(hdr.x), s_lut, lane, put);
                }
                if (!ok && lane == 0) raise_status(a.ctl, SPECKV_ST_BAD_RECORD, index);
                if (ok) st_decoded += 1;
            }
            __syncwarp();                                                     // tile written; record buffer free
            if ((j & 1u) == 0) {
                k_ok = ok;
            } else {
                if (k_ok && ok) attn_block(st, smem_u32(my_tile), smem_u32(my_tile + kTileBytes), 16u * (n0 + (j >> 1)), len, lane);
                __syncwarp();                                                 // tiles are rewritten by the next block
            }
        }
      }
      attn_end(st, a.partial + (size_t)(w + b * a.H + h) * kPartialFloats, lane);
      advance(sh, s_blk, a.B, a.H, n_piece);
    }
    if (lane == 0 && st_decoded) atomicAdd(&a.ctl->stats[kStDecoded], st_decoded);
}

// ---------------------------------------------------------------- merge of the partial results

// One warp per (sequence, query head): out = sum_i w_i o_i / sum_i w_i l_i over the partial results
// i of its (sequence, KV head) pair, w_i = 2^(m_i - max m).  The pair's blocks start at list position
// S = prefix[b]*H + h*nblk, so its partials come from the warps S/per .. (S + nblk - 1)/per.
__global__ void __launch_bounds__(128) attend_combine_kernel(AttendArgs a, uint32_t n_warps)
{
    // launched while the attention kernel is still running (programmatic dependent launch): its blocks are
    // resident and past their set-up when the last partial result lands
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t wid = blockIdx.x * 4u + (threadIdx.x >> 5), Hq = a.H * a.G;
    if (wid >= a.B * Hq) return;
    const uint32_t b = wid / Hq, hq = wid % Hq, h = hq / a.G, g = hq % a.G;
    const uint32_t nblk = a.prefix[b + 1] - a.prefix[b];
    float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    float den = 0.0f;
    if (nblk) {
        const unsigned long long T = (unsigned long long)a.prefix[a.B] * a.H, per = (T + n_warps - 1) / n_warps;
        const unsigned long long S = (unsigned long long)a.prefix[b] * a.H + (unsigned long long)h * nblk;
        const uint32_t w0 = (uint32_t)(S / per), w1 = (uint32_t)((S + nblk - 1) / per), pair = b * a.H + h;
        const float *base = a.partial + (size_t)pair * kPartialFloats;
        float mx = kNegInf;
        for (uint32_t w = w0 + lane; w <= w1; w += 32) mx = fmaxf(mx, base[(size_t)w * kPartialFloats + kHeadsPad * 128u + g]);
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, d));
        if (mx != kNegInf) {
#pragma unroll 4
            for (uint32_t w = w0; w <= w1; ++w) {
                const float *p = base + (size_t)w * kPartialFloats;
                const float wgt = ex2(p[kHeadsPad * 128u + g] - mx);
                den += wgt * p[kHeadsPad * 128u + kHeadsPad + g];
                const float4 o = *reinterpret_cast<const float4 *>(p + g * 128u + lane * 4u);
                acc.x += wgt * o.x; acc.y += wgt * o.y; acc.z += wgt * o.z; acc.w += wgt * o.w;
            }
        }
    }
    const float inv = den > 0.0f ? 1.0f / den : 0.0f;
    uint2 r;
    r.x = pack_h2(acc.x * inv, acc.y * inv);
    r.y = pack_h2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2 *>(a.out + ((size_t)b * Hq + hq) * 128u + lane * 4u) = r;
}

// ---------------------------------------------------------------- launchers

static size_t prefix_smem(uint32_t B) { return ((size_t)B + 1) * 4; }

uint32_t attend_max_warps() { return 8192; }                                  // bound on warps per launch (sizes the workspace)

cudaError_t launch_attend(const AttendArgs &a, bool fused, int n_sm, cudaStream_t stream)
{
    cudaError_t e;
    uint32_t n_warps;
    if (fused) {
        const size_t smem = (size_t)kFWarps * kFWarpBytes + 256 * 16 + kFWarps * 2 * 8 + prefix_smem(a.B);
        e = cudaFuncSetAttribute(attend_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        uint32_t grid = min((uint32_t)n_sm * 2u, attend_max_warps() / kFWarps);
        n_warps = grid * kFWarps;
        attend_fused_kernel<<<grid, kFWarps * 32, smem, stream>>>(a);
    } else {
        const size_t smem = (size_t)kDWarps * kDStages * 2 * kTileBytes + kDWarps * kDStages * 8 + prefix_smem(a.B);
        e = cudaFuncSetAttribute(attend_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        uint32_t grid = min((uint32_t)n_sm * 3u, attend_max_warps() / kDWarps);
        n_warps = grid * kDWarps;
        attend_dense_kernel<<<grid, kDWarps * 32, smem, stream>>>(a);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const uint32_t n_out = a.B * a.H * a.G;
    if (n_out) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((n_out + 3u) / 4u);
        cfg.blockDim = dim3(128);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // see griddepcontrol.wait in the kernel
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, attend_combine_kernel, a, n_warps);
    }
    return cudaGetLastError();
}

}  // namespace speckv
