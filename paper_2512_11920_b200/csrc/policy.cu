// Compression selection per layer (Sec. 3.6.3 of CXL-SpecKV):
//     C*(l,t) = argmax_{C}  w_r R_c(C,l) + w_q Q(C,l) - w_c L_comp(C)   subject to  Q(C,l) >= Q_min.
// speckv_probe_pages measures a sample of a layer's pages under every candidate scheme on the GPU (what the
// records would take, what the quantiser loses); speckv_select_scheme evaluates the objective on the host.
//
// Probe kernel: one warp per page, the compressor's lane layout (lane l, group k = the 8 elements at flat
// index 256*k + 8*l).  The two quantisers (one scale per page, one per group of 8 channels) are run one after
// the other; for each, the run heads of the delta stream are counted (sizes of the run-length modes) and
// the squared reconstruction error is summed in binary64 (every term is exact, only the order of the
// additions differs from a sequential sum).
#include <cmath>

#include "speckv_dev.cuh"

namespace speckv {

constexpr int kProbeWarps = 8;

struct ProbeArgs {
    const uint4 *src;
    const uint32_t *src_page;
    speckv_probe *out;
    uint32_t n_src_pages, n;
};

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
    return v;
}

// Quantises this lane's 64 elements with the reciprocal scale `inv`, returns the number of run heads of the
// page's delta-symbol stream that fall into this lane's elements (symbol 0 of the page included), and adds
// the squared error of the reconstruction fp16(q * s) to err.
__device__ __forceinline__ uint32_t quantise_count_heads(const uint4 (&x)[8], float inv, float s, uint32_t lane, double &err)
{
    const bool row_start = (lane & 15u) == 0;
    uint32_t heads = 0, carry = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint32_t h[4] = {x[k].x, x[k].y, x[k].z, x[k].w};
        uint32_t r[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&h[i]));
            const float v[2] = {a.x, a.y};
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const uint32_t bits = __float_as_uint(__fmaf_rn(v[j], inv, kMagic));   // 0x4B400000 + q
                r[2 * i + j] = bits;
                const float q = (float)((int)bits - (int)__float_as_uint(kMagic));
                const float back = __half2float(__float2half_rn(__fmul_rn(q, s)));
                const double e = (double)(v[j] - back);                              // exact in binary32
                err += e * e;
            }
        }
        // delta along the channels (restarting at channel 0 of a token row), low byte = symbol
        const uint32_t up = __shfl_up_sync(kFull, r[7], 1);
        const uint32_t prev = row_start ? __float_as_uint(kMagic) : up;
        uint32_t sym[8];
        sym[0] = (r[0] - prev) & 0xFFu;
#pragma unroll
        for (int e = 1; e < 8; ++e) sym[e] = (r[e] - r[e - 1]) & 0xFFu;
        // predecessor of this lane's first symbol in the flat stream: the previous lane's last symbol, for
        // lane 0 the last symbol of lane 31's previous group
        const uint32_t rot = __shfl_sync(kFull, sym[7], (lane + 31u) & 31u);
        const uint32_t before = lane ? rot : carry;
        carry = rot;
        uint32_t c = (sym[0] != before) || (k == 0 && lane == 0);
#pragma unroll
        for (int e = 1; e < 8; ++e) c += sym[e] != sym[e - 1];
        heads += c;
    }
    return heads;
}

__global__ void __launch_bounds__(kProbeWarps * 32) probe_kernel(ProbeArgs a)
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, n_warps = (gridDim.x * blockDim.x) >> 5;
    unsigned long long pages = 0, nonfinite = 0, bad = 0, gran[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    double err[2] = {0.0, 0.0}, sum = 0.0;
    for (uint32_t i = gw; i < a.n; i += n_warps) {
        const uint32_t sp = a.src_page[i];
        if (sp >= a.n_src_pages) { bad += 1; continue; }
        const uint4 *in = a.src + (size_t)sp * (kPageBytes / 16);
        uint4 x[8];
        uint32_t mi = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            x[k] = __ldg(in + k * 32 + lane);
            const uint32_t w[4] = {x[k].x, x[k].y, x[k].z, x[k].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) mi = max(mi, max(w[j] & 0x7FFFu, (w[j] >> 16) & 0x7FFFu));
        }
        const uint32_t amax_bits = __reduce_max_sync(kFull, mi);
        if (amax_bits >= 0x7C00u) { nonfinite += 1; continue; }          // stored raw whatever the scheme
        pages += 1;
        const uint32_t gmax = max(mi, __shfl_xor_sync(kFull, mi, 16));    // lanes l and l + 16 hold the same 8 channels
        double page_sum = 0.0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t w[4] = {x[k].x, x[k].y, x[k].z, x[k].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 v = __half22float2(*reinterpret_cast<const __half2 *>(&w[j]));
                page_sum += (double)v.x * (double)v.x + (double)v.y * (double)v.y;
            }
        }
        sum += page_sum;
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const uint32_t mb = g ? gmax : amax_bits;
            const float m = __half2float(__ushort_as_half((unsigned short)mb));
            const float s = mb ? __fdiv_rn(m, 127.0f) : 0.0f, inv = mb ? __fdiv_rn(127.0f, m) : 0.0f;
            const uint32_t n_runs = __reduce_add_sync(kFull, quantise_count_heads(x, inv, s, lane, err[g]));
            const uint32_t extra = g ? kGroupBytes : 0u;
            const uint32_t plain = (kHdrBytes + extra + kPageElems + kGranule - 1u) / kGranule;
            const uint32_t rle = (kHdrBytes + extra + kBitmapBytes + n_runs + kGranule - 1u) / kGranule;
            const uint32_t autom = kBitmapBytes + n_runs < kPageElems ? rle : plain;
            gran[4 * g + 0] += plain; gran[4 * g + 1] += plain; gran[4 * g + 2] += rle; gran[4 * g + 3] += autom;
        }
    }
    // every counter above except the sums of squares is warp-uniform
    const double e0 = warp_sum(err[0]), e1 = warp_sum(err[1]), ss = warp_sum(sum);
    if (lane == 0) {
        unsigned long long *o = reinterpret_cast<unsigned long long *>(a.out);
        if (pages) atomicAdd(&o[0], pages);
        if (nonfinite) atomicAdd(&o[1], nonfinite);
        if (bad) atomicAdd(&o[2], bad);
        if (pages) {
#pragma unroll
            for (int c = 0; c < 8; ++c) atomicAdd(&o[3 + c], gran[c]);
            atomicAdd(&a.out->sq_err[0], e0);
            atomicAdd(&a.out->sq_err[1], e1);
            atomicAdd(&a.out->sq_sum, ss);
        }
    }
}

static double probe_quality(const speckv_probe *p, int grouped)
{
    const double err = p->sq_err[grouped ? 1 : 0];
    if (!(err > 0.0) || !(p->sq_sum > 0.0)) return 200.0;
    const double q = 10.0 * std::log10(p->sq_sum / err);
    return q > 200.0 ? 200.0 : q;
}

}  // namespace speckv

extern "C" {

int speckv_probe_pages(const void *src, uint32_t n_src_pages, const uint32_t *src_page, uint32_t n, speckv_probe *out,
                       void *stream)
{
    using namespace speckv;
    static_assert(sizeof(speckv_probe) == 112 && sizeof(speckv_policy) == 96, "ABI layout");
    if (n == 0) return 0;
    if (!src || !src_page || !out || ((uintptr_t)src & 15u) || ((uintptr_t)src_page & 3u) || ((uintptr_t)out & 7u)) return SPECKV_E_ARG;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SPECKV_E_CUDA;
    ProbeArgs a = {(const uint4 *)src, src_page, out, n_src_pages, n};
    uint32_t grid = (n + kProbeWarps - 1) / kProbeWarps;
    if (grid > (uint32_t)n_sm * 4u) grid = (uint32_t)n_sm * 4u;
    probe_kernel<<<grid, kProbeWarps * 32, 0, (cudaStream_t)stream>>>(a);
    return cudaGetLastError() == cudaSuccess ? 0 : SPECKV_E_CUDA;
}

int speckv_select_scheme(const speckv_probe *p, const speckv_policy *pol, double *objective)
{
    using namespace speckv;
    static const int schemes[SPECKV_N_CANDIDATES] = {
        SPECKV_INT8, SPECKV_INT8_DELTA, SPECKV_INT8_DELTA_RLE, SPECKV_AUTO,
        SPECKV_INT8 | SPECKV_GROUPED, SPECKV_INT8_DELTA | SPECKV_GROUPED, SPECKV_INT8_DELTA_RLE | SPECKV_GROUPED,
        SPECKV_AUTO | SPECKV_GROUPED};
    if (!p || !pol || p->pages == 0) return SPECKV_E_ARG;
    const double quality[2] = {probe_quality(p, 0), probe_quality(p, 1)};
    int best = -1, finest = 0;
    double best_j = 0.0;
    for (int c = 0; c < SPECKV_N_CANDIDATES; ++c) {
        if (p->granules[c] == 0) return SPECKV_E_ARG;
        const double ratio = (double)p->pages * (double)(kPageBytes / kGranule) / (double)p->granules[c];
        const double q = quality[c / 4];
        const double j = pol->w_r * ratio + pol->w_q * q - pol->w_c * pol->cost[c];
        if (objective) objective[c] = j;
        if (q >= pol->q_min && (best < 0 || j > best_j)) { best = c; best_j = j; }
        if (q > quality[finest / 4]) finest = c;
    }
    return schemes[best >= 0 ? best : finest];
}

}  // extern "C"
