// fbq_linear_noalloc: the fused decode layer for callers that must not allocate.
//
// fbq_linear keeps its scratch space (split-K partial tiles, the down-projection
// t, arrival counters) in buffers it cudaMalloc's per stream the first time a
// shape needs them.  Some callers cannot have that happen inside the call: a
// serving process that handed all device memory to its own pool at start-up, so
// that a later cudaMalloc fails; a latency-critical loop that cannot afford the
// device-wide synchronisation cudaMalloc and cudaFree may imply; a plug-in whose
// host forbids driver allocations after initialisation.
// This entry point runs the same decode kernel with its scratch placed in ONE
// fixed array that is part of the library image, so nothing is ever allocated.
//
// The price: the array has a fixed size (requests beyond it are refused), every
// GPU that loads the library holds it until the process exits, and all calls
// share it.
#include <mutex>

#include "fbq_common.cuh"

namespace fbq {
void count_launches(int n);
DecodeTuning decode_tuning_for_noalloc();

namespace {

// Layout of the fixed scratch array (bytes):
//   [0, kCtrBytes)                 arrival counters / flags of the decode kernel (ints)
//   [kCtrBytes, +kTBytes)          t = x.A^T, 16 tokens x 256 ranks fp32
//   [kCtrBytes + kTBytes, end)     partial output tiles, fp32
constexpr size_t kMaxCounters = 8 + 2 * 4096;                 // output tiles: N <= 65536
constexpr size_t kCtrBytes = ((kMaxCounters * sizeof(int) + 255) / 256) * 256;
constexpr size_t kTBytes = (size_t)kDecodeMaxM * kMaxRank * sizeof(float);
constexpr size_t kMaxPartialFloats = 512 * 1024;              // 2 MiB of partial tiles
constexpr size_t kScratchBytes = kCtrBytes + kTBytes + kMaxPartialFloats * sizeof(float);

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char *g_base[kMaxDevices] = {};      // device address of the array, per device

// In host code `g_noalloc_scratch` is only a handle for the symbol, not a device
// address; the address each device gave the array has to be asked for, with that
// device current, once.
cudaError_t scratch_base(unsigned char **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_base[dev]) {
        unsigned char *ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_base[dev] = ptr;
    }
    *out = g_base[dev];
    return cudaSuccess;
}

}  // namespace

// Status word of the fixed array on device `dev` (FBQ_OK when the array was never used there).  A word
// that is set is returned once: reading clears it and resets the array's counters and t, which a kernel
// that gave up has left unfinished.  Called by fbq_poll_status after it has synchronised the stream.
int noalloc_poll_status(int dev)
{
    unsigned char *base = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (dev < 0 || dev >= kMaxDevices || !g_base[dev]) return FBQ_OK;
        base = g_base[dev];
    }
    int st = 0;
    if (cudaMemcpy(&st, base + kCtrStatus * sizeof(int), sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return FBQ_ERR_CUDA;
    if (st != 0 && cudaMemset(base, 0, kCtrBytes + kTBytes) != cudaSuccess) return FBQ_ERR_CUDA;
    return st;
}
}  // namespace fbq

using namespace fbq;

extern "C" int fbq_linear_noalloc(const void *x, const uint32_t *qweight, const void *scales, const void *zeros,
                                  const void *A, const void *B, void *y, int M, int N, int K, int group, int bits,
                                  int rank, int act_is_bf16, void *stream)
{
    // the decode kernel's domain, checked before anything touches CUDA
    if (M < 0 || N < 1 || K < 1 || rank < 0 || (bits != 3 && bits != 4)) return FBQ_ERR_BADARG;
    if (group != kGroupFast || K % kGroupFast != 0 || rank % 8 != 0 || rank > kMaxRank || M > kDecodeMaxM)
        return FBQ_ERR_UNSUPPORTED;
    if (M == 0) return FBQ_OK;
    if (!x || !qweight || !scales || !zeros || !y || (rank > 0 && (!A || !B))) return FBQ_ERR_BADARG;
    auto mis16 = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (mis16(x) || mis16(qweight) || mis16(y) || (rank > 0 && (mis16(A) || mis16(B)))) return FBQ_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(scales) & 1u) || (reinterpret_cast<uintptr_t>(zeros) & 1u)) return FBQ_ERR_ALIGN;

    LinearArgs a{};
    a.x = x;
    a.qw = qweight;
    a.scales = static_cast<const __half *>(scales);
    a.zeros = static_cast<const __half *>(zeros);
    a.A = rank > 0 ? A : nullptr;
    a.B = rank > 0 ? B : nullptr;
    a.y = y;
    a.M = M; a.N = N; a.K = K; a.group = group; a.bits = bits; a.rank = rank;
    a.bf16 = act_is_bf16 != 0;

    const DecodeTuning tune = decode_tuning_for_noalloc();     // the process-wide options; scratch-sizing ones automatic
    size_t partial_floats = 0;
    int counters = 0;
    decode_workspace_need(a, tune, &partial_floats, &counters);
    if (partial_floats > kMaxPartialFloats || (size_t)counters > kMaxCounters)
        return FBQ_ERR_UNSUPPORTED;            // beyond the fixed array: use fbq_linear

    unsigned char *base = nullptr;
    if (scratch_base(&base) != cudaSuccess) return FBQ_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Counters, flags and t must be zero when the kernel starts.  The kernel leaves them
    // zero, but the array is shared with every other call, so do not rely on it.
    // The status word (counter slot kCtrStatus) is left alone: a time-out of an earlier call stays readable
    // through fbq_poll_status until it is read.
    constexpr size_t kHead = (size_t)kCtrStatus * sizeof(int), kTail = ((size_t)kCtrStatus + 1) * sizeof(int);
    if (cudaMemsetAsync(base, 0, kHead, s) != cudaSuccess) return FBQ_ERR_CUDA;
    if (cudaMemsetAsync(base + kTail, 0, kCtrBytes + kTBytes - kTail, s) != cudaSuccess) return FBQ_ERR_CUDA;

    Workspace ws{};
    ws.counters = reinterpret_cast<int *>(base);
    ws.n_counters = (int)kMaxCounters;
    ws.t = reinterpret_cast<float *>(base + kCtrBytes);
    ws.t_floats = kTBytes / sizeof(float);
    ws.partial = reinterpret_cast<float *>(base + kCtrBytes + kTBytes);
    ws.partial_floats = kMaxPartialFloats;
    int launches = 0;
    const cudaError_t e = launch_decode(a, ws, tune, s, &launches);
    if (e == cudaErrorInvalidConfiguration) {
        (void)cudaGetLastError();
        return FBQ_ERR_UNSUPPORTED;
    }
    if (e != cudaSuccess) return FBQ_ERR_CUDA;
    count_launches(launches);
    return FBQ_OK;
}
