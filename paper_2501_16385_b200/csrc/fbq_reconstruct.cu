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
// are plain fp32 GEMMs and go to cuBLAS (pedantic math: no reduced-precision paths).  cuBLAS is
// looked up at run time (dlopen) the first time one of these entry points is called, so that
// the inference library itself has no link-time dependency on it; without it these entries
// return FBQ_ERR_UNSUPPORTED.  An offline step: correct and GEMM-bound, not tuned.
#include <cublas_v2.h>
#include <dlfcn.h>

#include <map>
#include <mutex>

#include "fbq_common.cuh"

namespace fbq {
namespace {

struct Blas {
    void *lib = nullptr;
    cublasStatus_t (*create)(cublasHandle_t *) = nullptr;
    cublasStatus_t (*set_stream)(cublasHandle_t, cudaStream_t) = nullptr;
    cublasStatus_t (*set_math)(cublasHandle_t, cublasMath_t) = nullptr;
    cublasStatus_t (*sgemm)(cublasHandle_t, cublasOperation_t, cublasOperation_t, int, int, int, const float *, const float *,
                            int, const float *, int, const float *, float *, int) = nullptr;
    std::map<int, cublasHandle_t> handles;      // per device
    bool tried = false;
};
Blas g_blas;
std::mutex g_blas_mu;

// Handle for the current device, bound to `s`; nullptr when cuBLAS cannot be had.
cublasHandle_t blas_handle(cudaStream_t s)
{
    std::lock_guard<std::mutex> lk(g_blas_mu);
    if (!g_blas.tried) {
        g_blas.tried = true;
        const char *names[] = {"libcublas.so.12", "libcublas.so", "/usr/local/cuda/lib64/libcublas.so.12"};
        for (const char *n : names) {
            g_blas.lib = dlopen(n, RTLD_NOW | RTLD_GLOBAL);
            if (g_blas.lib) break;
        }
        if (g_blas.lib) {
            g_blas.create = reinterpret_cast<decltype(g_blas.create)>(dlsym(g_blas.lib, "cublasCreate_v2"));
            g_blas.set_stream = reinterpret_cast<decltype(g_blas.set_stream)>(dlsym(g_blas.lib, "cublasSetStream_v2"));
            g_blas.set_math = reinterpret_cast<decltype(g_blas.set_math)>(dlsym(g_blas.lib, "cublasSetMathMode"));
            g_blas.sgemm = reinterpret_cast<decltype(g_blas.sgemm)>(dlsym(g_blas.lib, "cublasSgemm_v2"));
        }
    }
    if (!g_blas.create || !g_blas.set_stream || !g_blas.set_math || !g_blas.sgemm) return nullptr;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    auto it = g_blas.handles.find(dev);
    if (it == g_blas.handles.end()) {
        cublasHandle_t h = nullptr;
        if (g_blas.create(&h) != CUBLAS_STATUS_SUCCESS) return nullptr;
        g_blas.set_math(h, CUBLAS_PEDANTIC_MATH);
        it = g_blas.handles.emplace(dev, h).first;
    }
    if (g_blas.set_stream(it->second, s) != CUBLAS_STATUS_SUCCESS) return nullptr;
    return it->second;
}

// Row-major C[m x n] = alpha * op(P)[m x k] . op(Q)[k x n].  P is stored [m x k] (or [k x m] when
// transposed), Q [k x n] (or [n x k]).  cuBLAS is column-major: a row-major matrix is the
// column-major transpose, so C^T = op(Q)^T . op(P)^T is what is asked for.
bool gemm_rm(cublasHandle_t h, bool p_t, bool q_t, int m, int n, int k, float alpha, const float *P, const float *Q, float *C)
{
    const float beta = 0.f;
    const int ldp = p_t ? m : k, ldq = q_t ? k : n;
    return g_blas.sgemm(h, q_t ? CUBLAS_OP_T : CUBLAS_OP_N, p_t ? CUBLAS_OP_T : CUBLAS_OP_N, n, m, k, &alpha, Q, ldq, P, ldp,
                        &beta, C, n) == CUBLAS_STATUS_SUCCESS;
}

}  // namespace

size_t reconstruct_workspace_floats(int N, int K, int rank)
{
    return 2 * (size_t)N * K + (size_t)rank * K + (size_t)N * rank + 256;
}

// H[K x K] = X^T X for X [T x K]
int run_gram(const float *X, float *H, int T, int K, cudaStream_t s)
{
    cublasHandle_t h = blas_handle(s);
    if (!h) return FBQ_ERR_UNSUPPORTED;
    return gemm_rm(h, true, false, K, K, T, 1.f, X, X, H) ? FBQ_OK : FBQ_ERR_CUDA;
}

int run_reconstruct_step(const float *W, const float *H, float *A, float *B, float lr, float *loss, float *ws, int N, int K,
                         int group, int bits, int rank, cudaStream_t s)
{
    cublasHandle_t h = blas_handle(s);
    if (!h) return FBQ_ERR_UNSUPPORTED;
    float *Delta = ws, *G = Delta + (size_t)N * K, *gA = G + (size_t)N * K, *gB = gA + (size_t)rank * K,
          *partial = gB + (size_t)N * rank;
    // Delta_F with Q(W - B A) held fixed (nothing else of the quantiser's output is kept)
    if (launch_quantize_feedback(W, A, B, nullptr, nullptr, nullptr, nullptr, Delta, N, K, group, bits, rank, 2, s) != cudaSuccess)
        return FBQ_ERR_CUDA;
    // G = -2 Delta H
    if (!gemm_rm(h, false, false, N, K, K, -2.f, Delta, H, G)) return FBQ_ERR_CUDA;
    // L = tr(Delta H Delta^T) = -1/2 sum G o Delta
    if (loss && launch_scaled_dot(G, Delta, (size_t)N * K, -0.5f, partial, loss, s) != cudaSuccess) return FBQ_ERR_CUDA;
    // dL/dB = G A^T [N x rank],  dL/dA = B^T G [rank x K]
    if (!gemm_rm(h, false, true, N, rank, K, 1.f, G, A, gB)) return FBQ_ERR_CUDA;
    if (!gemm_rm(h, true, false, rank, K, N, 1.f, B, G, gA)) return FBQ_ERR_CUDA;
    if (launch_axpy(A, gA, -lr, (size_t)rank * K, s) != cudaSuccess) return FBQ_ERR_CUDA;
    if (launch_axpy(B, gB, -lr, (size_t)N * rank, s) != cudaSuccess) return FBQ_ERR_CUDA;
    return FBQ_OK;
}

}  // namespace fbq
