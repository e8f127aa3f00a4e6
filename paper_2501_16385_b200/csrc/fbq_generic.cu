// Generic kernel of the FBQuant linear: any well-formed shape, CUDA cores only.
// It is the fallback for shapes outside the decode / prefill kernels' domain
// (odd group sizes such as the 8x8 worked example) and follows the paper's
// two-kernel split of Section 4.3: a small down-projection kernel t = x.A^T,
// then one kernel that dequantises, contracts and adds the up-projection into
// the same output element before the single store.
#include "fbq_common.cuh"

namespace fbq {
namespace {

constexpr int kTokBlock = 8;     // tokens handled per warp pass

template <typename T>
__global__ void gen_down_kernel(const T *__restrict__ x, const T *__restrict__ A, float *__restrict__ t, int K,
                                int rank)
{
    // one block per (j, m): t[m][j] = sum_k x[m][k] * A[j][k], fp32
    const int j = blockIdx.x, m = blockIdx.y;
    const T *xr = x + (size_t)m * K;
    const T *ar = A + (size_t)j * K;
    float acc = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x)
        acc = fmaf(ActTraits<T>::to_float(xr[k]), ActTraits<T>::to_float(ar[k]), acc);
    __shared__ float red[32];
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float v = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) v += red[w];
        t[(size_t)m * rank + j] = v;
    }
}

// Codes of one "unit": 8 consecutive codes of an INT4 word, or the 32 codes of
// an INT3 run (three words).
template <int BITS> struct Unit;
template <> struct Unit<4> {
    static constexpr int kCodes = 8, kWords = 1;
    static __device__ __forceinline__ void decode(const uint32_t *w, int *q)
    {
#pragma unroll
        for (int e = 0; e < 8; ++e) q[e] = (int)((w[0] >> (4 * e)) & 0xFu);
    }
};
template <> struct Unit<3> {
    static constexpr int kCodes = 32, kWords = 3;
    static __device__ __forceinline__ void decode(const uint32_t *w, int *q)
    {
#pragma unroll
        for (int i = 0; i < 3; ++i)
#pragma unroll
            for (int f = 0; f < 5; ++f) {
                q[10 * i + f] = (int)((w[i] >> (3 * f)) & 7u);
                q[10 * i + 5 + f] = (int)((w[i] >> (16 + 3 * f)) & 7u);
            }
        q[30] = (int)(((w[0] >> 15) & 1u) | (((w[1] >> 15) & 1u) << 1) | (((w[2] >> 15) & 1u) << 2));
        q[31] = (int)(((w[0] >> 31) & 1u) | (((w[1] >> 31) & 1u) << 1) | (((w[2] >> 31) & 1u) << 2));
    }
};

template <typename T, int BITS>
__global__ void __launch_bounds__(128)
gen_main_kernel(const T *__restrict__ x, const uint32_t *__restrict__ qw, const __half *__restrict__ sc,
                const __half *__restrict__ ze, const float *__restrict__ t, const T *__restrict__ B,
                T *__restrict__ y, int M, int N, int K, int group, int rank)
{
    using U = Unit<BITS>;
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int m0 = blockIdx.y * kTokBlock;
    if (n >= N) return;
    const int G = K / group;
    const int units = K / U::kCodes;
    const uint32_t *row = qw + (size_t)n * units * U::kWords;
    const int mcount = min(kTokBlock, M - m0);

    float acc[kTokBlock];
#pragma unroll
    for (int i = 0; i < kTokBlock; ++i) acc[i] = 0.f;

    for (int u = lane; u < units; u += 32) {
        uint32_t w[U::kWords];
#pragma unroll
        for (int i = 0; i < U::kWords; ++i) w[i] = row[(size_t)u * U::kWords + i];
        int q[U::kCodes];
        U::decode(w, q);
        const int k0 = u * U::kCodes;
        const int g = k0 / group;                       // a unit never straddles a group
        const float s = __half2float(sc[(size_t)n * G + g]);
        const float z = __half2float(ze[(size_t)n * G + g]);
        float wv[U::kCodes];
#pragma unroll
        for (int e = 0; e < U::kCodes; ++e) wv[e] = __fmul_rn(s, __fsub_rn((float)q[e], z));
        for (int mm = 0; mm < mcount; ++mm) {
            const T *xr = x + (size_t)(m0 + mm) * K + k0;
            float a = 0.f;
#pragma unroll
            for (int e = 0; e < U::kCodes; ++e) a = fmaf(ActTraits<T>::to_float(xr[e]), wv[e], a);
#pragma unroll
            for (int i = 0; i < kTokBlock; ++i)          // keeps acc[] in registers
                if (i == mm) acc[i] += a;
        }
    }
#pragma unroll
    for (int i = 0; i < kTokBlock; ++i)
        for (int o = 16; o > 0; o >>= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);

    // up-projection added into the same output element (Section 4.3: the
    // sub-branch shares the output tensor of the main path)
#pragma unroll
    for (int i = 0; i < kTokBlock; ++i) {
        if (i >= mcount) break;
        float sub = 0.f;
        for (int j = lane; j < rank; j += 32)
            sub = fmaf(t[(size_t)(m0 + i) * rank + j], ActTraits<T>::to_float(B[(size_t)n * rank + j]), sub);
        for (int o = 16; o > 0; o >>= 1) sub += __shfl_xor_sync(0xffffffffu, sub, o);
        if (lane == 0) y[(size_t)(m0 + i) * N + n] = ActTraits<T>::from_float(acc[i] + sub);
    }
}

// The unfused sub-branch of the paper's comparison (Section 3.2, Fig. "kernel-fusion": the low-rank branch as
// separate launches next to the quantised main path).  u = t.B^T, rounded to the activation type and written out ...
template <typename T>
__global__ void gen_up_kernel(const float *__restrict__ t, const T *__restrict__ B, T *__restrict__ u, int N, int rank)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x, m = blockIdx.y;
    if (n >= N) return;
    float acc = 0.f;
    for (int j = 0; j < rank; ++j) acc = fmaf(t[(size_t)m * rank + j], ActTraits<T>::to_float(B[(size_t)n * rank + j]), acc);
    u[(size_t)m * N + n] = ActTraits<T>::from_float(acc);
}
// ... and y += u as a launch of its own (the extra read and write of the layer output that fusion removes).
template <typename T>
__global__ void gen_add_kernel(T *__restrict__ y, const T *__restrict__ u, size_t count)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) y[i] = ActTraits<T>::from_float(ActTraits<T>::to_float(y[i]) + ActTraits<T>::to_float(u[i]));
}

template <typename T>
cudaError_t run_unfused(const void *x, const void *A, const void *B, void *y, float *t, void *u, int M, int N, int K, int rank,
                        cudaStream_t s, int *launches)
{
    gen_down_kernel<T><<<dim3(rank, M), 128, 0, s>>>((const T *)x, (const T *)A, t, K, rank);
    gen_up_kernel<T><<<dim3((N + 127) / 128, M), 128, 0, s>>>(t, (const T *)B, (T *)u, N, rank);
    const size_t count = (size_t)M * N;
    gen_add_kernel<T><<<(unsigned)((count + 255) / 256), 256, 0, s>>>((T *)y, (const T *)u, count);
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) *launches += 3;
    return e;
}

template <typename T>
cudaError_t run_generic(const LinearArgs &a, float *t, cudaStream_t s, int *launches)
{
    if (a.rank > 0) {
        gen_down_kernel<T><<<dim3(a.rank, a.M), 128, 0, s>>>((const T *)a.x, (const T *)a.A, t, a.K, a.rank);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    const dim3 grid((a.N + 3) / 4, (a.M + kTokBlock - 1) / kTokBlock);
    if (a.bits == 4)
        gen_main_kernel<T, 4><<<grid, 128, 0, s>>>((const T *)a.x, a.qw, a.scales, a.zeros, t, (const T *)a.B,
                                                   (T *)a.y, a.M, a.N, a.K, a.group, a.rank);
    else
        gen_main_kernel<T, 3><<<grid, 128, 0, s>>>((const T *)a.x, a.qw, a.scales, a.zeros, t, (const T *)a.B,
                                                   (T *)a.y, a.M, a.N, a.K, a.group, a.rank);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) ++*launches;
    return e;
}

}  // namespace

cudaError_t launch_generic(const LinearArgs &a, Workspace &ws, cudaStream_t s, int *launches)
{
    // ws.t_gen holds M x rank floats (allocated by the caller of this function)
    return a.bf16 ? run_generic<__nv_bfloat16>(a, ws.t_gen, s, launches)
                  : run_generic<__half>(a, ws.t_gen, s, launches);
}

// t (M x rank floats) and u (M x N activation-type values) live in ws.t_gen, sized by the caller.
cudaError_t launch_sub_branch_unfused(const void *x, const void *A, const void *B, void *y, int M, int N, int K, int rank, bool bf16,
                                      Workspace &ws, cudaStream_t s, int *launches)
{
    float *t = ws.t_gen;
    void *u = ws.t_gen + (size_t)M * rank;
    return bf16 ? run_unfused<__nv_bfloat16>(x, A, B, y, t, u, M, N, K, rank, s, launches)
                : run_unfused<__half>(x, A, B, y, t, u, M, N, K, rank, s, launches);
}

}  // namespace fbq
