// Device twin of kvgen/gen.py: the same function of (seed key, page id, element) evaluated on
// the GPU, so that full-size synthetic KV tensors never cross PCIe.  Input generation only;
// nothing of the codec lives here.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ unsigned long long mix64(unsigned long long z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// one thread = 8 consecutive elements (two 64-bit draws), one 128-bit store
__global__ void __launch_bounds__(256) fill_kernel(uint4 *out, unsigned long long first_pid, unsigned long long n_pages,
                                                   unsigned long long key, const float *__restrict__ table,
                                                   const float *__restrict__ scales, unsigned long long pages_per_layer,
                                                   unsigned int n_kv_heads)
{
    const unsigned long long total = n_pages * 256ull;
    for (unsigned long long t = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (unsigned long long)gridDim.x * blockDim.x) {
        const unsigned long long pid = first_pid + t / 256ull;
        const unsigned int g = (unsigned int)(t % 256ull);            // group of 8 elements inside the page
        const unsigned long long row = (pid / pages_per_layer) * 2ull + (pid / n_kv_heads) % 2ull;
        const float *sc = scales + row * 128ull + (g % 16u) * 8u;
        unsigned int w[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const unsigned long long c = pid * 512ull + g * 2u + h;
            const unsigned long long r = mix64(key + c * 0x9E3779B97F4A7C15ull);
            __half v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                v[j] = __float2half_rn(__fmul_rn(table[(r >> (16 * j)) & 0xFFFFull], sc[h * 4 + j]));
            w[h * 2 + 0] = (unsigned int)__half_as_ushort(v[0]) | ((unsigned int)__half_as_ushort(v[1]) << 16);
            w[h * 2 + 1] = (unsigned int)__half_as_ushort(v[2]) | ((unsigned int)__half_as_ushort(v[3]) << 16);
        }
        out[t] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// piecewise-linear rows (gen.py: runs_pages): one thread = one token row of a page, 128 sequential steps
__global__ void __launch_bounds__(128) fill_runs_kernel(uint4 *out, unsigned long long first_pid, unsigned long long n_pages,
                                                        unsigned long long key, unsigned int p256)
{
    const unsigned long long total = n_pages * 16ull;
    for (unsigned long long t = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (unsigned long long)gridDim.x * blockDim.x) {
        const unsigned long long pid = first_pid + t / 16ull;
        const unsigned int j = (unsigned int)(t % 16ull);
        int u = 0, slope = 0;
        for (unsigned int i0 = 0; i0 < 128u; i0 += 8u) {
            unsigned int w[4];
#pragma unroll
            for (unsigned int e = 0; e < 8u; ++e) {
                const unsigned int i = i0 + e;
                const unsigned long long h = mix64(key + (pid * 2048ull + j * 128u + i) * 0x9E3779B97F4A7C15ull);
                if (i == 0u || (unsigned int)(h & 0xFFull) < p256) slope = (int)((h >> 8) % 5ull) - 2;
                if (i == 0u)
                    u = j == 0u ? 127 : (int)((h >> 16) % 81ull) - 40;
                else
                    u = max(-127, min(127, u + slope));
                const unsigned int bits = __half_as_ushort(__float2half_rn((float)u * 0.0078125f));
                if (e & 1u) w[e >> 1] |= bits << 16; else w[e >> 1] = bits;
            }
            out[t * 16ull + i0 / 8u] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

}  // namespace

extern "C" int kvgen_fill_runs(void *out, unsigned long long first_pid, unsigned long long n_pages, unsigned long long key,
                               unsigned int p256, void *stream)
{
    if (!out) return -1;
    if (n_pages == 0) return 0;
    unsigned long long blocks = (n_pages * 16ull + 127ull) / 128ull;
    if (blocks > 148ull * 64ull) blocks = 148ull * 64ull;
    fill_runs_kernel<<<(unsigned int)blocks, 128, 0, (cudaStream_t)stream>>>((uint4 *)out, first_pid, n_pages, key, p256);
    return cudaGetLastError() == cudaSuccess ? 0 : -2;
}

extern "C" int kvgen_fill(void *out, unsigned long long first_pid, unsigned long long n_pages, unsigned long long key,
                          const float *table_dev, const float *scales_dev, unsigned long long pages_per_layer,
                          unsigned int n_kv_heads, void *stream)
{
    if (!out || !table_dev || !scales_dev || !pages_per_layer || !n_kv_heads) return -1;
    if (n_pages == 0) return 0;
    unsigned long long blocks = (n_pages * 256ull + 255ull) / 256ull;
    if (blocks > 148ull * 32ull) blocks = 148ull * 32ull;
    fill_kernel<<<(unsigned int)blocks, 256, 0, (cudaStream_t)stream>>>((uint4 *)out, first_pid, n_pages, key, table_dev,
                                                                        scales_dev, pages_per_layer, n_kv_heads);
    return cudaGetLastError() == cudaSuccess ? 0 : -2;
}
