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

template <typename T>
__global__ void quantize_feedback_kernel(const float *__restrict__ W, const T *__restrict__ A, const T *__restrict__ B,
                                         uint8_t *__restrict__ codes, __half *__restrict__ scales,
                                         __half *__restrict__ zeros, float *__restrict__ WF, int N, int K, int group,
                                         int bits, int rank)
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
            sigma = __fmaf_rn(ActTraits<T>::to_float(B[(size_t)n * rank + j]), ActTraits<T>::to_float(A[(size_t)j * K + k]), sigma);
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
        scales[(size_t)n * G + g] = s_h;
        zeros[(size_t)n * G + g] = z_h;
        s_sz[0] = __half2float(s_h);
        s_sz[1] = __half2float(z_h);
    }
    __syncthreads();
    if (active) {
        const float sh = s_sz[0], zh = s_sz[1], maxq = (float)((1 << bits) - 1);
        float q = rintf(__fadd_rn(__fdiv_rn(r, sh), zh));
        q = fminf(fmaxf(q, 0.f), maxq);
        codes[(size_t)n * K + k] = (uint8_t)q;
        if (WF) WF[(size_t)n * K + k] = __fadd_rn(__fmul_rn(sh, __fsub_rn(q, zh)), sigma);
    }
}

}  // namespace

cudaError_t launch_quantize_feedback(const float *W, const void *A, const void *B, uint8_t *codes, __half *scales,
                                     __half *zeros, float *WF, int N, int K, int group, int bits, int rank, bool bf16,
                                     cudaStream_t s)
{
    const dim3 grid((unsigned)N, (unsigned)(K / group));
    const unsigned block = (unsigned)((group + 31) / 32 * 32);
    if (bf16)
        quantize_feedback_kernel<__nv_bfloat16><<<grid, block, 0, s>>>(W, static_cast<const __nv_bfloat16 *>(A),
                                                                        static_cast<const __nv_bfloat16 *>(B), codes, scales,
                                                                        zeros, WF, N, K, group, bits, rank);
    else
        quantize_feedback_kernel<__half><<<grid, block, 0, s>>>(W, static_cast<const __half *>(A),
                                                                static_cast<const __half *>(B), codes, scales, zeros, WF, N,
                                                                K, group, bits, rank);
    return cudaGetLastError();
}

}  // namespace fbq
