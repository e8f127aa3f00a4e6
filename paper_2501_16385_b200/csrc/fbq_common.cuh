// Shared declarations of the CUDA sources of libfbq (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fbq.h"

namespace fbq {

constexpr int kGroupFast = 128;   // group size of the decode / prefill kernels (Section 5.1)
constexpr int kMaxRank = 256;
constexpr int kDecodeMaxM = 16, kDecodePreferM = 6;

// Activation-type helpers ---------------------------------------------------
template <typename T> struct ActTraits;
template <> struct ActTraits<__half> {
    using T2 = __half2;
    static __device__ __forceinline__ float to_float(__half v) { return __half2float(v); }
    static __device__ __forceinline__ __half from_float(float v) { return __float2half_rn(v); }
};
template <> struct ActTraits<__nv_bfloat16> {
    using T2 = __nv_bfloat162;
    static __device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
    static __device__ __forceinline__ __nv_bfloat16 from_float(float v) { return __float2bfloat16_rn(v); }
};

// Per-stream scratch space (device memory owned by the library).
struct Workspace {
    float *partial = nullptr;     // split-K partial sums  [SK][M][N]
    size_t partial_floats = 0;
    float *t = nullptr;           // down-projection t = x.A^T, [M][rank] fp32 (kept zero between calls)
    float *t_gen = nullptr;       // t of the generic path (no invariant), grows on demand
    float *tslots = nullptr;      // streaming decode kernel: partial sums of t, one encoded word per entry (all zero between calls)
    size_t tslots_floats = 0;
    size_t t_floats = 0, t_gen_floats = 0;
    int *counters = nullptr;      // [0]=t arrivals [1]=retired tiles [2]=status [3]=t ready [4]=parked; [8..] per tile
    int n_counters = 0;
    void *trace = nullptr;        // optional phase timestamps of the decode kernel (tuning aid)
    void *stage_x = nullptr;      // staging for the host-buffer entry point
    void *stage_y = nullptr;
    size_t stage_x_bytes = 0, stage_y_bytes = 0;
};
constexpr int kCtrT = 0, kCtrDone = 1, kCtrStatus = 2;   // the decode kernel defines the rest

struct LinearArgs {
    const void *x;
    const uint32_t *qw;
    const __half *scales;
    const __half *zeros;
    const void *A;
    const void *B;
    void *y;
    int M, N, K, group, bits, rank;
    bool bf16;
};

// Launchers implemented in the kernel files.  Each returns a cudaError_t from
// the launch and adds the number of kernels it launched to *launches.
cudaError_t launch_pack(const uint8_t *codes, uint32_t *qw, int N, int K, int bits, cudaStream_t s);
cudaError_t launch_unpack(const uint32_t *qw, uint8_t *codes, int N, int K, int bits, cudaStream_t s);
cudaError_t launch_dequant(const uint32_t *qw, const __half *sc, const __half *ze, float *W, int N,
                           int K, int group, int bits, cudaStream_t s);
cudaError_t launch_generic(const LinearArgs &a, Workspace &ws, cudaStream_t s, int *launches);
cudaError_t launch_sub_branch_unfused(const void *x, const void *A, const void *B, void *y, int M, int N, int K, int rank, bool bf16,
                                      Workspace &ws, cudaStream_t s, int *launches);
cudaError_t launch_quantize_feedback(const float *W, const void *A, const void *B, uint8_t *codes, __half *scales,
                                     __half *zeros, float *WF, float *Delta, int N, int K, int group, int bits, int rank,
                                     int ab_kind, cudaStream_t s);
cudaError_t launch_scaled_dot(const float *a, const float *b, size_t n, float scale, float *partial, float *out, cudaStream_t s);
cudaError_t launch_axpy(float *y, const float *x, float alpha, size_t n, cudaStream_t s);
size_t reconstruct_workspace_floats(int N, int K, int rank);
int run_gram(const float *X, float *H, int T, int K, cudaStream_t s);
int run_reconstruct_step(const float *W, const float *H, float *A, float *B, float lr, float *loss, float *ws, int N, int K,
                         int group, int bits, int rank, cudaStream_t s);

struct DecodeTuning {
    int sk = 0, chunk = 0, depth = 0, max_ctas = 0, pdl = 1;
    int t_ctas = 1;  // 1: t = x.A^T comes from a few CTAs at the head of the grid (M <= 4, one K slice)
    int i8 = 1;      // 1: M <= 2 runs the form whose MMAs take the codes and x as 8-bit integers
};
// Returns cudaErrorInvalidConfiguration when no plan fits (caller falls back).
cudaError_t launch_decode(const LinearArgs &a, Workspace &ws, const DecodeTuning &tune,
                          cudaStream_t s, int *launches);
// Scratch the decode kernel needs for a shape (floats of partial sums, ints of counters).
void decode_workspace_need(const LinearArgs &a, const DecodeTuning &tune, size_t *partial_floats,
                           int *counters);

// The streaming decode kernel (fbq_gemv.cu).
struct GemvTuning {
    int max_ctas = 0;          // 0: one main CTA per SM
    int pdl = 1;
    int poll_limit = 0;        // 0: default number of looks at the "t complete" counter
    int test_skip_arrive = 0;  // test switch: the t CTAs do not report their arrival (the wait for t must run out)
};
int gemv_k_slices(int M, int K);      // K slices the streaming decode kernel cuts a shape into (1: x of all K fits)
bool gemv_supported(const LinearArgs &a);
void gemv_workspace_need(const LinearArgs &a, const GemvTuning &tune, size_t *tpart_floats, int *counters, size_t *partial_floats);
cudaError_t launch_gemv(const LinearArgs &a, Workspace &ws, const GemvTuning &tune, cudaStream_t s, int *launches);

int decode_batch_max();
bool decode_batch_need(const LinearArgs *a, int count, const int *ctas, const DecodeTuning &tune, size_t *partial_floats,
                       size_t *t_floats, int *counters);
cudaError_t launch_decode_batch(const LinearArgs *a, int count, const int *ctas, Workspace &ws, const DecodeTuning &tune,
                                cudaStream_t s, int *launches);
bool prefill_supported(const LinearArgs &a);
void prefill_workspace_need(const LinearArgs &a, int *counters, size_t *t_floats, size_t *partial_floats);
cudaError_t launch_prefill(const LinearArgs &a, Workspace &ws, cudaStream_t s, int *launches);

}  // namespace fbq
