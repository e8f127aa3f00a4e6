// Feedback quantiser (Section 4.1 of the paper): the main path of FBQuant stores
// Q(W - Sigma), Sigma = B.A, so that  W_F = Q(W - Sigma) + Sigma  stays within s/2 of W
// for a round-to-nearest quantiser (Eq. "diff" and the bound below it).  This is the
// offline step that produces the (codes, s, z) the inference kernels consume.
//
// Reading of "linear quantizer, group size 128, round to nearest with scaling factor s":
// asymmetric min-max per group of `group` consecutive input channels of one output row,
//     r = W - B.A                       s = max((max r - min r)/(2^bits - 1), 2^-14)
//     z = rint(-min r / s)              q = clamp(rint(r/s + z), 0, 2^bits - 1)   (ties to even)
// (constant group c: s = max(|c|, 2^-14), z = 1 if c < 0 else 0), with s and z rounded to
// fp16 first and the STORED values used for the codes, so that dequantisation inverts
// exactly what was coded.  Every rounding decision is taken in IEEE single precision with
// one operation per step (explicit _rn intrinsics: no contraction, no fast division), in
// the order the definition states, so that a CPU check can reproduce the codes bit for bit.
//
// One CTA per (group, row); a thread owns one k: it forms Sigma[n][k] with rank fused
// multiply-adds (A read coalesced across the CTA, B broadcast), the CTA reduces min and max,
// thread 0 fixes (s, z), every thread codes its element.  HBM traffic is W once (4 B per
// weight) plus a byte per code; A is re-read from L2 by every row.  An offline step: it is
// correct and coalesced, not tuned.
#include "fbq_common.cuh"

namespace fbq {
namespace {

template <typename T> __device__ __forceinline__ float ab_to_float(T v) { return ActTraits<T>::to_float(v); }
template <> __device__ __forceinline__ float ab_to_float<float>(float v) { return v; }

// codes, scales/zeros, WF and Delta (= W - W_F, the Delta_F of Section 4.2) are each optional.
template <typename T>
__global__ void quantize_feedback_kernel(const float *__restrict__ W, const T *__restrict__ A, const T *__restrict__ B,
                                         uint8_t *__restrict__ codes, __half *__restrict__ scales,
                                         __half *__restrict__ zeros, float *__restrict__ WF, float *__restrict__ Delta,
                                         int N, int K, int group, int bits, int rank)
{
    __shared__ float s_min[32], s_max[32];
    __shared__ float s_sz[2];
    const int n = blockIdx.x, g = blockIdx.y, i = threadIdx.x;     // rows vary fastest: neighbours share A's columns in L2
    const int G = K / group;
    const bool active = i < group;
    const int k = g * group + (active ? i : 0);
    float sigma = 0.f, r = 0.f;
    if (active) {
        for (int j = 0; j < rank; ++j)
            sigma = __fmaf_rn(ab_to_float<T>(B[(size_t)n * rank + j]), ab_to_float<T>(A[(size_t)j * K + k]), sigma);
        r = __fsub_rn(W[(size_t)n * K + k], sigma);
    }
    float mn = active ? r : INFINITY, mx = active ? r : -INFINITY;
    for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if ((i & 31) == 0) {
        s_min[i >> 5] = mn;
        s_max[i >> 5] = mx;
    }
    __syncthreads();
    if (i == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        for (int w = 1; w < nw; ++w) {
            mn = fminf(mn, s_min[w]);
            mx = fmaxf(mx, s_max[w]);
        }
        const float maxq = (float)((1 << bits) - 1), smin = 6.103515625e-05f;   // 2^-14
        float s, z;
        if (mx > mn) {
            s = fmaxf(__fdiv_rn(__fsub_rn(mx, mn), maxq), smin);
            const float sh = __half2float(__float2half_rn(s));
            z = rintf(__fdiv_rn(-mn, sh));
        } else {
            s = fmaxf(fabsf(mn), smin);
            z = (mn < 0.f) ? 1.f : 0.f;
        }
        const __half s_h = __float2half_rn(s), z_h = __float2half_rn(z);
        if (scales) {
            scales[(size_t)n * G + g] = s_h;
            zeros[(size_t)n * G + g] = z_h;
        }
        s_sz[0] = __half2float(s_h);
        s_sz[1] = __half2float(z_h);
    }
    __syncthreads();
    if (active) {
        const float sh = s_sz[0], zh = s_sz[1], maxq = (float)((1 << bits) - 1);
        float q = rintf(__fadd_rn(__fdiv_rn(r, sh), zh));
        q = fminf(fmaxf(q, 0.f), maxq);
        if (codes) codes[(size_t)n * K + k] = (uint8_t)q;
        const float wf = __fadd_rn(__fmul_rn(sh, __fsub_rn(q, zh)), sigma);
        if (WF) WF[(size_t)n * K + k] = wf;
        if (Delta) Delta[(size_t)n * K + k] = __fsub_rn(W[(size_t)n * K + k], wf);
    }
}

}  // namespace

// ab_kind: 0 = fp16, 1 = bf16, 2 = fp32 sub-branch matrices
cudaError_t launch_quantize_feedback(const float *W, const void *A, const void *B, uint8_t *codes, __half *scales,
                                     __half *zeros, float *WF, float *Delta, int N, int K, int group, int bits, int rank,
                                     int ab_kind, cudaStream_t s)
{
    const dim3 grid((unsigned)N, (unsigned)(K / group));
    const unsigned block = (unsigned)((group + 31) / 32 * 32);
    if (ab_kind == 2)
        quantize_feedback_kernel<float><<<grid, block, 0, s>>>(W, static_cast<const float *>(A), static_cast<const float *>(B),
                                                               codes, scales, zeros, WF, Delta, N, K, group, bits, rank);
    else if (ab_kind == 1)
        quantize_feedback_kernel<__nv_bfloat16><<<grid, block, 0, s>>>(W, static_cast<const __nv_bfloat16 *>(A),
                                                                        static_cast<const __nv_bfloat16 *>(B), codes, scales,
                                                                        zeros, WF, Delta, N, K, group, bits, rank);
    else
        quantize_feedback_kernel<__half><<<grid, block, 0, s>>>(W, static_cast<const __half *>(A),
                                                                static_cast<const __half *>(B), codes, scales, zeros, WF,
                                                                Delta, N, K, group, bits, rank);
    return cudaGetLastError();
}

// ---- reconstruction step helpers (Algorithm 1 lines 7-9) ---------------------------------
// partial[b] = sum over this block's slice of a[i]*b[i]; a second launch with one block adds the
// partials in index order and writes scale * sum.  Fixed order: the result is reproducible.
__global__ void dot_partial_kernel(const float *__restrict__ a, const float *__restrict__ b, size_t n, float *partial)
{
    __shared__ float sh[32];
    float v = 0.f;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) v = fmaf(a[i], b[i], v);
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sh[w];
        partial[blockIdx.x] = t;
    }
}
__global__ void dot_final_kernel(const float *partial, int n, float scale, float *out)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < n; ++i) t += (double)partial[i];
        *out = (float)(t * (double)scale);
    }
}
__global__ void axpy_kernel(float *__restrict__ y, const float *__restrict__ x, float alpha, size_t n)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        y[i] = fmaf(alpha, x[i], y[i]);
}

cudaError_t launch_scaled_dot(const float *a, const float *b, size_t n, float scale, float *partial /*>= 256*/, float *out,
                              cudaStream_t s)
{
    dot_partial_kernel<<<256, 256, 0, s>>>(a, b, n, partial);
    dot_final_kernel<<<1, 32, 0, s>>>(partial, 256, scale, out);
    return cudaGetLastError();
}
cudaError_t launch_axpy(float *y, const float *x, float alpha, size_t n, cudaStream_t s)
{
    const unsigned blocks = (unsigned)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
    axpy_kernel<<<blocks ? blocks : 1, 256, 0, s>>>(y, x, alpha, n);
    return cudaGetLastError();
}

}  // namespace fbq
