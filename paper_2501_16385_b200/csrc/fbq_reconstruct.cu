// One iteration of layer-wise reconstruction (Algorithm 1 lines 5-9, Section 4.2 of the paper):
//
//   Delta_F = W - Q(W - B A) - B A                      (feedback quantiser of Section 4.1, detached)
//   L       = tr(Delta_F H Delta_F^T),  H = X^T X        (= ||W X^T - W_F X^T||_F^2)
//   G       = dL/dSigma = -2 Delta_F H
//   dL/dB   = G A^T,   dL/dA = B^T G                     (Sigma = B A)
//   A <- A - lr dL/dA,  B <- B - lr dL/dB                (both gradients from the old A, B)
//
// Delta_F comes from this library's quantiser kernel (fp32 master copies of A and B), the loss
// from a fixed-order reduction kernel, the updates from an axpy kernel; the three dense products
// and the Gram matrix are plain fp32 GEMMs on CUDA cores (64 x 64 tiles through shared memory,
// sums over k in ascending order: results do not depend on the grid).  An offline step: correct,
// not tuned.
#include "fbq_common.cuh"

namespace fbq {
namespace {

constexpr int kGT = 64, kGK = 16;          // output tile, k step

// C[m][n] = alpha * sum_k P(m, k) Q(k, n), C row-major [M x N]; P(m, k) = P[m * pm + k * pk], Q(k, n) = Q[k * qk + n * qn]
// (strides in elements express the transposes).  256 threads, 4 x 4 outputs each.
__global__ void __launch_bounds__(256) sgemm_kernel(const float *__restrict__ P, const float *__restrict__ Q, float *__restrict__ C, int M,
                                                     int N, int K, long long pm, long long pk, long long qk, long long qn, float alpha)
{
    __shared__ float sp[kGK][kGT + 1], sq[kGK][kGT + 1];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * kGT, n0 = blockIdx.x * kGT;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < K; k0 += kGK) {
        for (int e = tid; e < kGT * kGK; e += 256) {
            // along whichever index is contiguous in memory, so that the loads coalesce
            const int a = (pk == 1) ? e / kGK : e % kGT, kk = (pk == 1) ? e % kGK : e / kGT;
            const int m = m0 + a, k = k0 + kk;
            sp[kk][a] = (m < M && k < K) ? P[(long long)m * pm + (long long)k * pk] : 0.f;
            const int c = (qk == 1) ? e / kGK : e % kGT, kq = (qk == 1) ? e % kGK : e / kGT;
            const int n = n0 + c, k2 = k0 + kq;
            sq[kq][c] = (n < N && k2 < K) ? Q[(long long)k2 * qk + (long long)n * qn] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kGK; ++kk) {
            float pv[4], qv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) pv[i] = sp[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) qv[j] = sq[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(pv[i], qv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
            if (m < M && n < N) C[(long long)m * N + n] = alpha * acc[i][j];
        }
}

// Row-major C[m x n] = alpha * op(P)[m x k] . op(Q)[k x n].  P is stored [m x k] (or [k x m] when transposed),
// Q [k x n] (or [n x k]).
bool gemm_rm(cudaStream_t s, bool p_t, bool q_t, int m, int n, int k, float alpha, const float *P, const float *Q, float *C)
{
    const dim3 grid((unsigned)((n + kGT - 1) / kGT), (unsigned)((m + kGT - 1) / kGT));
    sgemm_kernel<<<grid, 256, 0, s>>>(P, Q, C, m, n, k, p_t ? 1 : k, p_t ? m : 1, q_t ? 1 : n, q_t ? k : 1, alpha);
    return cudaGetLastError() == cudaSuccess;
}

}  // namespace

size_t reconstruct_workspace_floats(int N, int K, int rank)
{
    return 2 * (size_t)N * K + (size_t)rank * K + (size_t)N * rank + 256;
}

// H[K x K] = X^T X for X [T x K]
int run_gram(const float *X, float *H, int T, int K, cudaStream_t s)
{
    return gemm_rm(s, true, false, K, K, T, 1.f, X, X, H) ? FBQ_OK : FBQ_ERR_CUDA;
}

int run_reconstruct_step(const float *W, const float *H, float *A, float *B, float lr, float *loss, float *ws, int N, int K,
                         int group, int bits, int rank, cudaStream_t s)
{
    float *Delta = ws, *G = Delta + (size_t)N * K, *gA = G + (size_t)N * K, *gB = gA + (size_t)rank * K,
          *partial = gB + (size_t)N * rank;
    // Delta_F with Q(W - B A) held fixed (nothing else of the quantiser's output is kept)
    if (launch_quantize_feedback(W, A, B, nullptr, nullptr, nullptr, nullptr, Delta, N, K, group, bits, rank, 2, s) != cudaSuccess)
        return FBQ_ERR_CUDA;
    // G = -2 Delta H
    if (!gemm_rm(s, false, false, N, K, K, -2.f, Delta, H, G)) return FBQ_ERR_CUDA;
    // L = tr(Delta H Delta^T) = -1/2 sum G o Delta
    if (loss && launch_scaled_dot(G, Delta, (size_t)N * K, -0.5f, partial, loss, s) != cudaSuccess) return FBQ_ERR_CUDA;
    // dL/dB = G A^T [N x rank],  dL/dA = B^T G [rank x K]
    if (!gemm_rm(s, false, true, N, rank, K, 1.f, G, A, gB)) return FBQ_ERR_CUDA;
    if (!gemm_rm(s, true, false, rank, K, N, 1.f, B, G, gA)) return FBQ_ERR_CUDA;
    if (launch_axpy(A, gA, -lr, (size_t)rank * K, s) != cudaSuccess) return FBQ_ERR_CUDA;
    if (launch_axpy(B, gB, -lr, (size_t)N * rank, s) != cudaSuccess) return FBQ_ERR_CUDA;
    return FBQ_OK;
}

}  // namespace fbq
