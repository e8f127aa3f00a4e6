// Packing, unpacking and dense dequantisation kernels (offline / test aids of
// the weight-only quantised storage; Section 1 of the paper keeps weights in
// INT3/INT4).  One thread produces one packed word (pack) or one code (unpack,
// dequant); all accesses are coalesced along K.
#include "fbq_common.cuh"

namespace fbq {
namespace {

// INT4: word w of a row takes codes 8w .. 8w+7, code e at bits 4e..4e+3.
__global__ void pack4_kernel(const uint8_t *__restrict__ codes, uint32_t *__restrict__ qw, size_t n_words)
{
    size_t w = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (w >= n_words) return;
    const uint2 c8 = *reinterpret_cast<const uint2 *>(codes + 8 * w);   // 8 codes, K % 8 == 0
    uint32_t out = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        out |= ((c8.x >> (8 * e)) & 0xFu) << (4 * e);
        out |= ((c8.y >> (8 * e)) & 0xFu) << (16 + 4 * e);
    }
    qw[w] = out;
}

// INT3: thread (run, i) builds word i of a 32-code run:
//   fields f=0..4 at bits 3f: c[10i+f]; at bits 16+3f: c[10i+5+f];
//   bit 15: bit i of c[30]; bit 31: bit i of c[31].
__global__ void pack3_kernel(const uint8_t *__restrict__ codes, uint32_t *__restrict__ qw, size_t n_words)
{
    size_t w = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (w >= n_words) return;
    const size_t run = w / 3;
    const int i = (int)(w - run * 3);
    const uint8_t *c = codes + run * 32;
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int f = 0; f < 5; ++f) {
        lo |= (uint32_t)(c[10 * i + f] & 7u) << (3 * f);
        hi |= (uint32_t)(c[10 * i + 5 + f] & 7u) << (3 * f);
    }
    lo |= (uint32_t)((c[30] >> i) & 1u) << 15;
    hi |= (uint32_t)((c[31] >> i) & 1u) << 15;
    qw[w] = lo | (hi << 16);
}

__device__ __forceinline__ uint32_t fetch_code(const uint32_t *__restrict__ qw, size_t row_words_base,
                                               int k, int bits)
{
    if (bits == 4) {
        const uint32_t w = qw[row_words_base + (k >> 3)];
        return (w >> ((k & 7) * 4)) & 0xFu;
    }
    const uint32_t *r = qw + row_words_base + (size_t)(k >> 5) * 3;
    const int c = k & 31;
    if (c >= 30) {
        const int sh = (c == 30) ? 15 : 31;
        return ((r[0] >> sh) & 1u) | (((r[1] >> sh) & 1u) << 1) | (((r[2] >> sh) & 1u) << 2);
    }
    const int i = c / 10, f = c - 10 * i;
    const int sh = (f < 5) ? 3 * f : 3 * f + 1;          // 16 + 3(f-5) = 3f + 1
    return (r[i] >> sh) & 7u;
}

__global__ void unpack_kernel(const uint32_t *__restrict__ qw, uint8_t *__restrict__ codes, int N, int K,
                              int bits)
{
    const size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * K) return;
    const int n = (int)(idx / K), k = (int)(idx - (size_t)n * K);
    const size_t row_words = (bits == 4) ? (size_t)(K / 8) : (size_t)(K / 32) * 3;
    codes[idx] = (uint8_t)fetch_code(qw, n * row_words, k, bits);
}

__global__ void dequant_kernel(const uint32_t *__restrict__ qw, const __half *__restrict__ sc,
                               const __half *__restrict__ ze, float *__restrict__ W, int N, int K, int group,
                               int bits)
{
    const size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * K) return;
    const int n = (int)(idx / K), k = (int)(idx - (size_t)n * K);
    const size_t row_words = (bits == 4) ? (size_t)(K / 8) : (size_t)(K / 32) * 3;
    const int G = K / group;
    const float s = __half2float(sc[(size_t)n * G + k / group]);
    const float z = __half2float(ze[(size_t)n * G + k / group]);
    const float q = (float)fetch_code(qw, n * row_words, k, bits);
    W[idx] = __fmul_rn(s, __fsub_rn(q, z));   // exact: 11-bit significand times a 5-bit integer
}

}  // namespace

cudaError_t launch_pack(const uint8_t *codes, uint32_t *qw, int N, int K, int bits, cudaStream_t s)
{
    const size_t n_words = (bits == 4) ? (size_t)N * K / 8 : (size_t)N * K / 32 * 3;
    const int threads = 256;
    const unsigned blocks = (unsigned)((n_words + threads - 1) / threads);
    if (bits == 4)
        pack4_kernel<<<blocks, threads, 0, s>>>(codes, qw, n_words);
    else
        pack3_kernel<<<blocks, threads, 0, s>>>(codes, qw, n_words);
    return cudaGetLastError();
}

cudaError_t launch_unpack(const uint32_t *qw, uint8_t *codes, int N, int K, int bits, cudaStream_t s)
{
    const size_t total = (size_t)N * K;
    const int threads = 256;
    unpack_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, s>>>(qw, codes, N, K, bits);
    return cudaGetLastError();
}

cudaError_t launch_dequant(const uint32_t *qw, const __half *sc, const __half *ze, float *W, int N, int K,
                           int group, int bits, cudaStream_t s)
{
    const size_t total = (size_t)N * K;
    const int threads = 256;
    dequant_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, s>>>(qw, sc, ze, W, N, K, group,
                                                                                  bits);
    return cudaGetLastError();
}

}  // namespace fbq
