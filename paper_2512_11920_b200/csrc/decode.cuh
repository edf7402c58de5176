// Decoder shared by the kernels that read records: page-table entry fields, and the decompression
// pipeline of CXL-SpecKV (run expansion -> running sum of deltas -> dequantisation) for one staged
// record, one warp per page.
#pragma once
#include <cuda_fp16.h>

#include "speckv_dev.cuh"

namespace speckv {

// ---------------------------------------------------------------- page-table entry

struct Walk { unsigned long long byte_off; uint32_t rec_len, mode; int rc; };

__device__ __forceinline__ Walk decode_pte(unsigned long long e, unsigned long long pool_bytes)
{
    Walk w{0ull, 0u, 0u, 0};
    if (!(e & kPteValid)) { w.rc = SPECKV_ST_BAD_PTE; return w; }
    w.byte_off = (e & 0xFFFFFFFFull) * kGranule;
    w.rec_len = (uint32_t)(e >> 32) & 0xFFFFu;
    w.mode = (uint32_t)(e >> 48) & 0xFFu;
    if (w.rec_len < kHdrBytes || w.byte_off + w.rec_len > pool_bytes) w.rc = SPECKV_ST_BAD_RECORD;
    return w;
}

// Table entry of the run expansion for a head mask m of 8 symbols: x, y = PRMT selectors of symbols 0-3 and 4-7
// (index into "byte in progress + following run values"), z = 8 * number of heads among symbols 0-3 (how far the
// second word's window is shifted).
__device__ __forceinline__ uint4 expand_entry(uint32_t m)
{
    return make_uint4(expand_sel(m & 15u), expand_sel((m >> 4) & 15u), 8u * __popc(m & 15u), 0u);
}

// ---------------------------------------------------------------- small PTX wrappers

// packed binary32 pairs: (a - b) * c with one rounding per operation and element
__device__ __forceinline__ void sub_mul_x2(float a0, float a1, float negb, float c, float &r0, float &r1)
{
    unsigned long long A, B, C, T;
    asm("mov.b64 %0, {%1, %2};" : "=l"(A) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %1};" : "=l"(B) : "f"(negb));
    asm("mov.b64 %0, {%1, %1};" : "=l"(C) : "f"(c));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(T) : "l"(A), "l"(B));
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(T) : "l"(T), "l"(C));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(r0), "=f"(r1) : "l"(T));
}
__device__ __forceinline__ uint32_t pack_h2(float a, float b)
{
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}
// low byte of t = q + 128  ->  binary32 value 2^23 + (q + 128)
__device__ __forceinline__ float biased(uint32_t t) { return __uint_as_float(__byte_perm(t, 0x4B000000u, 0x7540)); }

// ---------------------------------------------------------------- decode of one staged record

// Decodes the staged record (mode 1..3, with or without SPECKV_GROUPED) and hands the page out as
// eight calls store(k, v): v = the 8 binary16 values at flat index 256*k + 8*lane (token row
// 2*k + lane/16, channels 8*(lane%16)..).  Returns false if the record is inconsistent (nothing
// is stored then).  `lut` = 256 entries made by expand_entry().
template <class Store>
__device__ __forceinline__ bool decode_page(const uint8_t *rec, uint32_t mode, uint32_t payload_len, uint32_t n_runs,
                                            float s, const uint4 *lut, uint32_t lane, Store store)
{
    if (mode & SPECKV_GROUPED) {
        // one scale per group of 8 channels = per pair of lanes (l, l + 16), from the stored maximum
        if (payload_len < kGroupBytes) return false;
        const uint32_t gmax = reinterpret_cast<const uint16_t *>(rec + kHdrBytes)[lane & 15u];
        if (__any_sync(kFull, gmax >= 0x7C00u)) return false;
        s = __fdiv_rn(__half2float(__ushort_as_half((unsigned short)gmax)), 127.0f);
        rec += kGroupBytes;
        payload_len -= kGroupBytes;
        mode &= ~(uint32_t)SPECKV_GROUPED;
    }
    uint32_t sy[8][2];   // symbols (modes 2, 3) or quantised bytes (mode 1) of this lane's groups
    const uint2 *pay = reinterpret_cast<const uint2 *>(rec + kHdrBytes);
    if (mode == SPECKV_INT8_DELTA_RLE) {
        if (n_runs < 1u || n_runs > kPageElems || payload_len != kBitmapBytes + n_runs) return false;
        uint32_t mk[8], c[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) { mk[k] = rec[kHdrBytes + k * 32 + lane]; c[k] = __popc(mk[k]); }
        // rank of each group's first run = exclusive prefix sum of popcounts in (k, lane) order: within a row the
        // exclusive sums stay below 8 * 31, so four rows share a word as byte fields; row totals by warp reduction
        const uint32_t ea = scan_excl_bytes(c[0] + (c[1] << 8) + (c[2] << 16) + (c[3] << 24));
        const uint32_t eb = scan_excl_bytes(c[4] + (c[5] << 8) + (c[6] << 16) + (c[7] << 24));
        uint32_t excl[8], tot[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            excl[k] = __byte_perm(k < 4 ? ea : eb, 0u, 0x4440 + (k & 3));
            tot[k] = __reduce_add_sync(kFull, c[k]);
        }
        uint32_t total = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) total += tot[k];
        uint32_t first_ok = __shfl_sync(kFull, mk[0] & 1u, 0);
        if (total != n_runs || !first_ok) return false;
        uint32_t base = kValuesOff - 1u;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            // bytes [R-1, R+8) of the value stream: the run in progress, then this group's new runs
            uint32_t A = base + excl[k];
            const uint32_t *w = reinterpret_cast<const uint32_t *>(rec + (A & ~3u));
            uint32_t sh = A << 3;                             // funnel shifts use the low 5 bits: 8 * (A & 3)
            uint32_t w0 = w[0], w1 = w[1], w2 = w[2];
            uint32_t v0 = __funnelshift_r(w0, w1, sh), v1 = __funnelshift_r(w1, w2, sh), v2 = __funnelshift_r(w2, 0u, sh);
            const uint4 e = lut[mk[k]];                       // selectors of the two words, 8 * (heads in the first word)
            sy[k][0] = __byte_perm(v0, v1, e.x);
            uint32_t u0 = __funnelshift_rc(v0, v1, e.z), u1 = __funnelshift_rc(v1, v2, e.z);
            sy[k][1] = __byte_perm(u0, u1, e.y);
            base += tot[k];
        }
    } else {
        if (payload_len != kPageElems) return false;
#pragma unroll
        for (int k = 0; k < 8; ++k) { uint2 t = pay[k * 32 + lane]; sy[k][0] = t.x; sy[k][1] = t.y; }
    }

    uint32_t cb[8];      // per group: value to add to its running sums so that the low byte is q + 128
    if (mode == SPECKV_INT8) {
#pragma unroll
        for (int k = 0; k < 8; ++k) cb[k] = 0;
    } else {
        // Running sum of the deltas along each token row (16 lanes).  Only the sums' low bytes matter (mod 256),
        // but a group total is at most 8 * 255 and a row has 16 lanes, so whole sums fit 16-bit fields: two groups
        // per word, plain additions, no carries between fields.  Segmented inclusive scan over the 16 lanes of a
        // row, then exclusive = inclusive - own, plus 128 (the low byte of every running sum is then q + 128).
        uint32_t p[4];
#pragma unroll
        for (int k = 0; k < 8; k += 2) {
            const uint32_t t0 = __dp4a(sy[k][1], 0x01010101u, __dp4a(sy[k][0], 0x01010101u, 0u));
            const uint32_t t1 = __dp4a(sy[k + 1][1], 0x01010101u, __dp4a(sy[k + 1][0], 0x01010101u, 0u));
            p[k / 2] = t0 + (t1 << 16);
        }
        uint32_t inc[4] = {p[0], p[1], p[2], p[3]};
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) {
            const bool take = (lane & 15u) >= (uint32_t)d;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t up = __shfl_up_sync(kFull, inc[j], d, 16);
                if (take) inc[j] += up;
            }
        }
        // cb[k]: anything whose low byte is (exclusive sum + 128) mod 256 — the bits above are never looked at
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t e = inc[j] - p[j] + 0x00800080u;
            cb[2 * j] = e;
            cb[2 * j + 1] = e >> 16;
        }
    }
    const float negb = -8388736.0f;   // -(2^23 + 128)
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        uint32_t t[8];
        if (mode == SPECKV_INT8) {
            uint32_t b0 = sy[k][0] ^ 0x80808080u, b1 = sy[k][1] ^ 0x80808080u;
            t[0] = b0; t[1] = b0 >> 8; t[2] = b0 >> 16; t[3] = b0 >> 24;
            t[4] = b1; t[5] = b1 >> 8; t[6] = b1 >> 16; t[7] = b1 >> 24;
        } else {
            t[0] = __dp4a(sy[k][0], 0x00000001u, cb[k]);
            t[1] = __dp4a(sy[k][0], 0x00000101u, cb[k]);
            t[2] = __dp4a(sy[k][0], 0x00010101u, cb[k]);
            t[3] = __dp4a(sy[k][0], 0x01010101u, cb[k]);
            t[4] = __dp4a(sy[k][1], 0x00000001u, t[3]);
            t[5] = __dp4a(sy[k][1], 0x00000101u, t[3]);
            t[6] = __dp4a(sy[k][1], 0x00010101u, t[3]);
            t[7] = __dp4a(sy[k][1], 0x01010101u, t[3]);
        }
        float f[8];
#pragma unroll
        for (int e = 0; e < 8; e += 2) sub_mul_x2(biased(t[e]), biased(t[e + 1]), negb, s, f[e], f[e + 1]);
        store(k, make_uint4(pack_h2(f[0], f[1]), pack_h2(f[2], f[3]), pack_h2(f[4], f[5]), pack_h2(f[6], f[7])));
    }
    return true;
}

}  // namespace speckv
